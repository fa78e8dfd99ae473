"""Sequence-parallel attention (Section 3.2 of the paper): every rank holds a contiguous range of the flat token
axis with all heads; attention runs head-sharded between two exchanges.

Plumbing only: `torch.distributed` carries the two all-to-alls (NCCL on GPUs), every byte that moves on the
device is moved by the library's kernels (stride-aware QKV pack, attention, inverse head merge).  One
collective each way, as in the paper; the packed QKV receive buffer is consumed by the attention through strides,
and the attention's own output buffer is the send buffer of the return path, so neither side makes a layout copy
beyond the pack and the merge.

Transport "peer" (optional, one node): the pack kernel stores straight into the owners' receive buffers and the
attention epilogue stores each output row straight into its token owner's merged buffer, so the only
collectives left are barriers.  Where the buffers come from is a separate object (`PeerBuffers`):
`symmetric_memory_buffers` maps every rank's buffers into this process with
`torch.distributed._symmetric_memory`; `local_peer_buffers` puts all ranks' buffers on one device, which is how
the transport's own code runs in single-GPU tests (the ranks then take turns phase by phase).
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B


def shard_ranges(total: int, n_ranks: int) -> List[Tuple[int, int]]:
    """Contiguous token ranges per rank: ceil(total / n_ranks) tokens each, trailing ranks shorter or empty."""
    per = (total + n_ranks - 1) // n_ranks
    return [(min(g * per, total), min((g + 1) * per, total)) for g in range(n_ranks)]


class ExchangePlan:
    """Host-side description of the two all-to-alls for one rank (pure Python, no device work)."""

    def __init__(self, total_tokens: int, heads: int, head_dim: int, n_ranks: int, rank: int, out_record_bytes: int,
                 qkv_record_elems: int = 0, out_record_elems: int = 0):
        """qkv_record_elems / out_record_elems: elements of the exchanged tensors per (token, head) record
        (default: 3*head_dim and head_dim, the unquantised layouts; the block-INT8 records are 400 / 144 bytes)."""
        if n_ranks < 1 or n_ranks > B.MAX_RANKS:
            raise ValueError(f"1 <= n_ranks <= {B.MAX_RANKS}")
        if heads % n_ranks:
            raise ValueError("heads must be divisible by the number of ranks")
        if not 0 <= rank < n_ranks:
            raise ValueError("rank out of range")
        self.total, self.heads, self.head_dim, self.n_ranks, self.rank = total_tokens, heads, head_dim, n_ranks, rank
        self.hl = heads // n_ranks
        self.ranges = shard_ranges(total_tokens, n_ranks)
        self.tok_begin = [a for a, _ in self.ranges] + [total_tokens]
        self.n_local = self.ranges[rank][1] - self.ranges[rank][0]
        self.first_token = self.ranges[rank][0]
        self.qkv_record_elems = qkv_record_elems or 3 * head_dim
        self.out_record_elems = out_record_elems or head_dim
        self.out_record_bytes = out_record_bytes               # bytes of one (token, head) record on the wire
        (self.qkv_send_splits, self.qkv_recv_splits, self.out_send_splits, self.out_recv_splits) = self.splits(self.hl)

    def splits(self, group_heads: int):
        """Split sizes, in ELEMENTS of the exchanged tensors, when `group_heads` heads of every rank's shard travel:
        (qkv send, qkv receive, output send, output receive).  QKV: this rank sends its n_local rows to everyone
        and receives n_s rows from rank s.  Output: it owes rows [a_g, b_g) to rank g and receives its own
        n_local rows from everyone."""
        qkv_row = group_heads * self.qkv_record_elems
        out_row = group_heads * self.out_record_elems
        return ([self.n_local * qkv_row] * self.n_ranks, [(b - a) * qkv_row for a, b in self.ranges],
                [(b - a) * out_row for a, b in self.ranges], [self.n_local * out_row] * self.n_ranks)


class PeerBuffers:
    """Memory of the peer transport as one rank sees it: its own receive buffers and every rank's addresses.

    qkv          this rank's packed QKV receive buffer [total, 3, heads/G, D] bf16
    merged       this rank's output rows [largest shard, heads, D]
    qkv_peers    device addresses of every rank's `qkv`, by rank (this rank's own included)
    merged_peers the same for `merged`
    barrier      callable: orders the phases across ranks (stream-ordered; a no-op where one stream runs all ranks)
    """

    def __init__(self, rank, n_ranks, qkv, merged, qkv_peers, merged_peers, barrier, keep=None):
        self.rank, self.n_ranks = rank, n_ranks
        self.qkv, self.merged = qkv, merged
        self.qkv_peers, self.merged_peers = [int(x) for x in qkv_peers], [int(x) for x in merged_peers]
        self.barrier = barrier
        self.keep = keep                                   # whatever must stay alive with the buffers (handles)


def peer_buffer_shapes(total: int, heads: int, head_dim: int, n_ranks: int, qkv_record_bytes: int = 0,
                       out_record_bytes: int = 0):
    """Shapes of the two buffers every rank of the peer transport owns: the QKV receive buffer, [total, 3, heads/G, D]
    bf16 or [total, heads/G, record] bytes for the block-INT8 wire format, and the output rows, [largest shard, heads,
    D] or [largest shard, heads, record] bytes."""
    per = shard_ranges(total, n_ranks)[0]
    n_max, hl = max(per[1] - per[0], 1), heads // n_ranks
    qkv = (total, hl, qkv_record_bytes) if qkv_record_bytes else (total, 3, hl, head_dim)
    merged = (n_max, heads, out_record_bytes) if out_record_bytes else (n_max, heads, head_dim)
    return qkv, merged


def symmetric_memory_buffers(total, heads, head_dim, out_dtype, device, group=None, qkv_record_bytes: int = 0,
                             out_record_bytes: int = 0) -> PeerBuffers:
    """Buffers in symmetric memory, every rank's mapped into this process (plain peer addresses; no multicast is
    used by the kernels that store through them).  Collective: every rank of `group` must call it."""
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm
    n_ranks, rank = dist.get_world_size(group), dist.get_rank(group)
    qkv_shape, merged_shape = peer_buffer_shapes(total, heads, head_dim, n_ranks, qkv_record_bytes, out_record_bytes)
    qkv = symm.empty(qkv_shape, dtype=torch.uint8 if qkv_record_bytes else torch.bfloat16, device=device)
    merged = symm.empty(merged_shape, dtype=torch.uint8 if out_record_bytes else out_dtype, device=device)
    gname = (group or dist.group.WORLD).group_name
    hq, hm = symm.rendezvous(qkv, gname), symm.rendezvous(merged, gname)
    token = torch.zeros(1, dtype=torch.int32, device=device)

    def barrier():
        # stream-ordered: every rank's earlier kernels on this stream are complete when the reduction returns
        dist.all_reduce(token, group=group)

    return PeerBuffers(rank, n_ranks, qkv, merged, hq.buffer_ptrs, hm.buffer_ptrs, barrier, keep=(hq, hm, token))


def local_peer_buffers(total, heads, head_dim, n_ranks, out_dtype, device, qkv_record_bytes: int = 0,
                       out_record_bytes: int = 0) -> List[PeerBuffers]:
    """All ranks' buffers on one device (one PeerBuffers per rank, sharing the address lists).  The ranks' phases
    are then run one after another on one stream, which orders them: the barrier is a no-op."""
    qkv_shape, merged_shape = peer_buffer_shapes(total, heads, head_dim, n_ranks, qkv_record_bytes, out_record_bytes)
    qkvs = [torch.empty(qkv_shape, dtype=torch.uint8 if qkv_record_bytes else torch.bfloat16, device=device)
            for _ in range(n_ranks)]
    mergeds = [torch.empty(merged_shape, dtype=torch.uint8 if out_record_bytes else out_dtype, device=device)
               for _ in range(n_ranks)]
    qp, mp = [t.data_ptr() for t in qkvs], [t.data_ptr() for t in mergeds]
    return [PeerBuffers(r, n_ranks, qkvs[r], mergeds[r], qp, mp, lambda: None) for r in range(n_ranks)]


class _HeadGroup:
    """Buffers and plan of one head group of this rank's shard (collective transport)."""

    def __init__(self, sp, seqs, begin: int, count: int, rope_dims, theta, device):
        xp, D, G, n_local, total = sp.xp, sp.head_dim, sp.n_ranks, sp.xp.n_local, sp.xp.total
        self.begin, self.count = begin, count
        self.qkv_send_splits, self.qkv_recv_splits, self.out_send_splits, self.out_recv_splits = xp.splits(count)
        st = (3 * count * D, D)
        self.attn = B.Attn3d(seqs, count, D, rope_dims, theta, device, q_strides=st, k_strides=st, v_strides=st)
        if sp.qkv_int8:
            # records arrive and feed the attention as they are: the rotary producer dequantises (Q~, K~ into the plan's
            # workspace, V into this scratch); no packed bf16 QKV tensor exists on this side
            self.send = torch.empty((G, n_local, count, sp.rb_in), dtype=torch.uint8, device=device)
            self.qkv_records = torch.empty((total, count, sp.rb_in), dtype=torch.uint8, device=device)
            self.v_scratch = torch.empty((total, count, D), dtype=torch.bfloat16, device=device)
        else:
            self.qkv = torch.empty((total, 3, count, D), dtype=torch.bfloat16, device=device)
            self.send = torch.empty((G, n_local, 3, count, D), dtype=torch.bfloat16, device=device)
        if sp.out_int8:
            # the attention epilogue writes the records that travel back
            self.out_shard = torch.empty((total, count, sp.rb_out), dtype=torch.uint8, device=device)
            self.recv_out = torch.empty((G, n_local, count, sp.rb_out), dtype=torch.uint8, device=device)
        else:
            self.out_shard = torch.empty((total, count, D), dtype=sp.out_dtype, device=device)
            self.recv_out = torch.empty((G, n_local, count, D), dtype=sp.out_dtype, device=device)
        self.ev_in = torch.cuda.Event()
        self.ev_out = torch.cuda.Event()


class SequenceParallelAttn3d:
    """One DiT-block attention over a sequence-sharded Q, K, V.  forward() returns this rank's token rows."""

    def __init__(self, seqs: Sequence[Tuple[int, int, int, int]], heads: int, head_dim: int, rope_dims, theta: float = 10000.0,
                 group=None, device="cuda", out_format: str = "bf16", transport: str = "collective", qkv_wire: str = "bf16",
                 n_groups: int = 1, peer_buffers: Optional[PeerBuffers] = None):
        """out_format: what travels back and is returned -- "bf16", "e4m3" (raw bytes, returned as uint8) or "int8"
        (block-INT8 records on the wire, dequantised to bf16 on arrival).  qkv_wire: "bf16" or "int8" (block-INT8
        records on the wire, dequantised to bf16 before the attention).  The quantised formats are approximate.
        n_groups (collective transport): this rank's head shard is served in that many head groups; the exchanges
        of one group run on side streams under the attention of another (heads are independent).
        peer_buffers (peer transport): where the buffers live and who the ranks are; default: symmetric memory over
        `group`.  With buffers from local_peer_buffers no process group is needed."""
        if peer_buffers is not None:
            if transport != "peer":
                raise ValueError("peer_buffers belong to transport 'peer'")
            self.dist, self.group = None, None
            self.n_ranks, self.rank = peer_buffers.n_ranks, peer_buffers.rank
        else:
            import torch.distributed as dist
            self.dist = dist
            self.group = group
            self.n_ranks = dist.get_world_size(group)
            self.rank = dist.get_rank(group)
        if out_format not in ("bf16", "e4m3", "int8"):
            raise ValueError("out_format: 'bf16', 'e4m3' or 'int8'")
        if qkv_wire not in ("bf16", "int8"):
            raise ValueError("qkv_wire: 'bf16' or 'int8'")
        if transport not in ("collective", "peer"):
            raise ValueError("transport: 'collective' or 'peer'")
        if transport == "peer" and n_groups != 1:
            raise ValueError("transport 'peer' works in one head group")
        self.fp8 = out_format == "e4m3"
        self.out_int8 = out_format == "int8"
        self.qkv_int8 = qkv_wire == "int8"
        self.transport = transport
        self.heads, self.head_dim = heads, head_dim
        total = sum(L + T * H * W for (L, T, H, W) in seqs)
        D = head_dim
        self.rb_in = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D) if self.qkv_int8 else 3 * D * 2
        self.rb_out = B.sol_attn3d_exchange_record_bytes(
            B.WIRE_OUT_INT8 if self.out_int8 else B.WIRE_OUT_E4M3 if self.fp8 else B.WIRE_OUT_BF16, D)
        self.xp = ExchangePlan(total, heads, D, self.n_ranks, self.rank, self.rb_out,
                               qkv_record_elems=self.rb_in if self.qkv_int8 else 0,
                               out_record_elems=self.rb_out if self.out_int8 else 0)
        hl = self.xp.hl
        self.out_dtype = torch.uint8 if self.fp8 else torch.bfloat16
        if transport == "collective":
            n_groups = max(1, min(int(n_groups), hl))
            bounds = [hl * j // n_groups for j in range(n_groups + 1)]
            self.groups = [_HeadGroup(self, seqs, bounds[j], bounds[j + 1] - bounds[j], rope_dims, theta, device)
                           for j in range(n_groups)]
            self.s_in = torch.cuda.Stream(device=device)       # QKV pack + exchange (+ dequantisation)
            self.s_out = torch.cuda.Stream(device=device)      # output exchange + merge (+ dequantisation)
        else:
            qkv_strides = (3 * hl * D, D)
            self.attn = B.Attn3d(seqs, hl, D, rope_dims, theta, device, q_strides=qkv_strides, k_strides=qkv_strides,
                                 v_strides=qkv_strides)
            rb_q = self.rb_in if self.qkv_int8 else 0
            rb_o = self.rb_out if self.out_int8 else 0
            self.pb = peer_buffers if peer_buffers is not None else symmetric_memory_buffers(
                total, heads, D, self.out_dtype, device, group, rb_q, rb_o)
            qkv_shape, merged_shape = peer_buffer_shapes(total, heads, D, self.n_ranks, rb_q, rb_o)
            if tuple(self.pb.qkv.shape) != qkv_shape or tuple(self.pb.merged.shape) != merged_shape or \
                    self.pb.merged.dtype != (torch.uint8 if rb_o else self.out_dtype) or \
                    len(self.pb.qkv_peers) != self.n_ranks or len(self.pb.merged_peers) != self.n_ranks:
                raise ValueError("peer buffers do not fit this problem")

    # ---- peer transport, phase by phase (forward() runs them with barriers in between)
    def peer_pack(self, q, k, v):
        """Phase 1: this rank's Q, K, V rows go straight into every owner's receive buffer (as bf16 rows, or quantised to
        block-INT8 records on the way)."""
        pack = B.sol_attn3d_exchange_pack_qkv_int8 if self.qkv_int8 else B.sol_attn3d_exchange_pack_qkv
        pack(q, k, v, self.n_ranks, self.pb.qkv_peers, self.xp.first_token)

    def peer_attend(self, key_mask=None):
        """Phase 2 (after every rank's phase 1): attention over this rank's head shard; the epilogue stores each
        output row into its token owner's merged buffer, at this shard's head offset."""
        qkv = self.pb.qkv
        fmt = B.OUT_INT8 if self.out_int8 else B.OUT_E4M3 if self.fp8 else B.OUT_BF16
        if self.qkv_int8:
            # the scatter entry point takes bf16 views: dequantise the records this rank received (its own buffer) first
            bf = torch.empty((self.xp.total, 3, self.xp.hl, self.head_dim), dtype=torch.bfloat16, device=qkv.device)
            B.sol_attn3d_exchange_unpack_qkv_int8(qkv, bf, self.xp.total, self.xp.hl, self.head_dim)
            qkv = bf
        B.sol_attn3d_forward_scatter(self.attn.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], key_mask, self.pb.merged_peers,
                                     self.xp.tok_begin, self.heads, self.rank * self.xp.hl, fmt)

    def peer_result(self):
        """Phase 3 (after every rank's phase 2): this rank's token rows, all heads (block-INT8 records are dequantised
        to bf16 rows here, on arrival)."""
        rows = self.pb.merged[:self.xp.n_local]
        if not self.out_int8:
            return rows
        out = torch.empty((self.xp.n_local, self.heads, self.head_dim), dtype=torch.bfloat16, device=rows.device)
        if self.xp.n_local:
            B.sol_attn3d_exchange_dequantize_out_int8(rows.contiguous(), out)
        return out

    def forward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, key_mask: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q, k, v: [n_local, heads, D] bf16 (any strides, e.g. views into packed QKV); key_mask: uint8 [total] or None."""
        xp = self.xp
        if tuple(q.shape) != (xp.n_local, self.heads, self.head_dim):
            raise ValueError(f"expected [{xp.n_local}, {self.heads}, {self.head_dim}] on rank {self.rank}")
        if self.transport == "collective":
            return self._forward_collective(q, k, v, key_mask)
        # peer transport: stores into the owners' buffers, barriers instead of payload collectives
        self.pb.barrier()                                     # everyone is done reading last call's buffers
        self.peer_pack(q, k, v)
        self.pb.barrier()
        self.peer_attend(key_mask)
        self.pb.barrier()
        return self.peer_result()

    def _forward_collective(self, q, k, v, key_mask):
        xp, D, G = self.xp, self.head_dim, self.n_ranks
        cur = torch.cuda.current_stream()
        out = torch.empty((xp.n_local, self.heads, D), dtype=self.out_dtype, device=q.device)
        out.record_stream(self.s_out)
        merged = None
        if self.out_int8:
            merged = torch.empty((xp.n_local, self.heads, self.rb_out), dtype=torch.uint8, device=q.device)
            merged.record_stream(self.s_out)
        # (1) every group's QKV exchange is queued up front on the input stream: pack -> all-to-all (-> dequantise)
        self.s_in.wait_stream(cur)                            # q, k, v are ready; last call's readers are done
        self.s_out.wait_stream(cur)
        with torch.cuda.stream(self.s_in):
            for gr in self.groups:
                dsts = [gr.send[r].data_ptr() for r in range(G)]
                if self.qkv_int8:
                    B.sol_attn3d_exchange_pack_qkv_int8(q, k, v, G, dsts, 0, group_begin=gr.begin, group_heads=gr.count)
                    self.dist.all_to_all_single(gr.qkv_records.view(-1), gr.send.view(-1), gr.qkv_recv_splits,
                                                gr.qkv_send_splits, group=self.group)
                else:
                    B.sol_attn3d_exchange_pack_qkv(q, k, v, G, dsts, 0, group_begin=gr.begin, group_heads=gr.count)
                    self.dist.all_to_all_single(gr.qkv.view(-1), gr.send.view(-1), gr.qkv_recv_splits, gr.qkv_send_splits,
                                                group=self.group)
                gr.ev_in.record(self.s_in)
        # (2) attention group by group on the caller's stream; (3) each group's output returns on the output stream
        for gr in self.groups:
            cur.wait_event(gr.ev_in)
            fmt = B.OUT_INT8 if self.out_int8 else B.OUT_E4M3 if self.fp8 else B.OUT_BF16
            if self.qkv_int8:
                B.sol_attn3d_forward_qkv_int8(gr.attn.plan, gr.qkv_records, gr.v_scratch, gr.out_shard, key_mask, fmt)
            else:
                qv, kv, vv = gr.qkv[:, 0], gr.qkv[:, 1], gr.qkv[:, 2]
                if self.out_int8:
                    B.sol_attn3d_forward_int8(gr.attn.plan, qv, kv, vv, gr.out_shard, key_mask)
                elif self.fp8:
                    B.sol_attn3d_forward_e4m3(gr.attn.plan, qv, kv, vv, gr.out_shard, key_mask)
                else:
                    B.sol_attn3d_forward(gr.attn.plan, qv, kv, vv, gr.out_shard, key_mask)
            wire = gr.out_shard
            gr.ev_out.record(cur)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(gr.ev_out)
                self.dist.all_to_all_single(gr.recv_out.view(-1), wire.view(-1), gr.out_recv_splits, gr.out_send_splits,
                                            group=self.group)
                # the group's heads land in their place in the full rows: rank stride = the whole shard
                target = merged if self.out_int8 else out
                rec = self.rb_out
                B.sol_attn3d_exchange_merge_heads(gr.recv_out, target.data_ptr() + gr.begin * rec, xp.n_local, G * gr.count, rec, G,
                                                  self.heads * rec, out_rank_stride_bytes=xp.hl * rec)
        with torch.cuda.stream(self.s_out):
            if self.out_int8:
                B.sol_attn3d_exchange_dequantize_out_int8(merged, out)
        cur.wait_stream(self.s_out)
        return out

    def close(self):
        if self.transport == "collective":
            for gr in self.groups:
                gr.attn.close()
        else:
            self.attn.close()
