/*
 * sol_attn3d -- 3D-RoPE joint self-attention of a video DiT block on NVIDIA B200 (sm_100a).
 *
 * The operation (per sequence, per head):
 *
 *     q~_i = RoPE3D(q_i, pos_i),  k~_j = RoPE3D(k_j, pos_j)        (video tokens only)
 *     out_i = sum_j softmax_j( <q~_i, k~_j> / sqrt(head_dim) ) v_j   over valid keys j
 *
 * This is the dense attention ("SDPA") that Section 3.2 of the paper ("Optimized attention
 * collectives") reports as the dominant cost of a denoising step, combined with the rotary
 * embedding of fusion group (2) in Section 3.5 ("QK normalization with partial RoPE"), on the
 * prefix-first packed token order of Section 3.4 ("Safety rails and the exact prefix KV sink")
 * and the flat (total, heads, head_dim) activation layout of Section 3.2.
 *
 * Conventions (the paper prints no formula; these are the definitions this library implements):
 *   - a sequence is text_len prefix tokens followed by T*H*W video tokens, t slowest, w fastest;
 *   - prefix tokens carry no rotary embedding; V is never rotated;
 *   - rope_dims = {d_T, d_H, d_W}: head dims [0,d_T) rotate with t, [d_T,d_T+d_H) with h, the next
 *     d_W with w; dims beyond d_T+d_H+d_W pass through ("partial" RoPE).  Inside an axis of width
 *     d_a the ADJACENT pair (2j, 2j+1) rotates by pos_a * theta^(-2j/d_a), counter-clockwise;
 *   - non-causal; the only masks are the key-padding mask and the block-diagonal structure of a
 *     packed batch (a query attends to the keys of its own sequence only);
 *   - a query row whose sequence has no valid key returns zeros.
 *
 * All tensors are bf16.  Math: rotation in fp32 from fp64-built tables, QK^T and PV on tcgen05
 * tensor cores (bf16 operands, fp32 accumulation in tensor memory), softmax in fp32.
 *
 * Every function returns 0 on success or a negative sol_attn3d_error.  No function throws, aborts
 * or synchronises the device unless stated.  There is no CPU fallback: without a B200 the device
 * calls fail with SOL_ATTN3D_ERR_NO_DEVICE / SOL_ATTN3D_ERR_UNSUPPORTED_ARCH.
 */
#ifndef SOL_ATTN3D_H_
#define SOL_ATTN3D_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sol_attn3d_plan_s* sol_attn3d_plan_t;
/* A cudaStream_t, passed as an opaque pointer so this header needs no CUDA include. */
typedef void* sol_attn3d_stream_t;

typedef enum {
  SOL_ATTN3D_OK = 0,
  SOL_ATTN3D_ERR_INVALID_ARG = -1,      /* NULL where a pointer is required, non-positive size, odd rope dim ... */
  SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE = -2,/* head_dim not 64/128, strides not 16-byte multiples, size overflow */
  SOL_ATTN3D_ERR_NO_WORKSPACE = -3,     /* forward before set_workspace, or workspace too small / misaligned */
  SOL_ATTN3D_ERR_NO_DEVICE = -4,        /* no CUDA device / driver */
  SOL_ATTN3D_ERR_UNSUPPORTED_ARCH = -5, /* current device is not compute capability 10.x */
  SOL_ATTN3D_ERR_CUDA = -6,             /* a CUDA call failed; sol_attn3d_last_cuda_error() has the code */
  SOL_ATTN3D_ERR_DEVICE_TIMEOUT = -7,   /* a bounded wait inside a kernel ran out (status word) */
  SOL_ATTN3D_ERR_NO_MEMORY = -8,        /* host allocation failed */
  SOL_ATTN3D_ERR_SCRATCH_LIMIT = -9,    /* sol_attn3d_forward_noalloc: the plan needs more than the built-in scratch */
  SOL_ATTN3D_ERR_DEVICE_ASSERT = -10    /* debug build: a device-side index check failed (status word) */
} sol_attn3d_error;

/*
 * Extended problem description (packed / ragged batches, strided tensors).
 *   size       sizeof(sol_attn3d_desc), for versioning.
 *   n_seqs     number of packed sequences (>= 1).
 *   grids      n_seqs x 3 ints {T, H, W}, each >= 1 ... or T*H*W may be 0 only via T=0 (prefix-only sequence).
 *   text_lens  n_seqs prefix lengths (>= 0).  Sequence s holds text_lens[s] + T*H*W tokens and starts
 *              where sequence s-1 ends (cu_seqlens is derived; see sol_attn3d_cu_seqlens).
 *   theta      rotary base (> 1); the benchmark configurations use 10000.
 *   *_strides  element strides {token, head} of q, k, v, out; {0,0} means contiguous
 *              {heads*head_dim, head_dim}.  head_dim is always contiguous.  Strides let Q, K and V be
 *              views into one packed QKV buffer (Section 3.2).  Byte strides must be multiples of 16.
 */
typedef struct {
  uint32_t size;
  int32_t n_seqs;
  const int32_t* grids;
  const int32_t* text_lens;
  int32_t heads;
  int32_t head_dim;
  int32_t rope_dims[3];
  double theta;
  int64_t q_strides[2];
  int64_t k_strides[2];
  int64_t v_strides[2];
  int64_t out_strides[2];
} sol_attn3d_desc;

/*
 * Plan for B equal sequences (Section 3.2's attention over [prefix | T*H*W video tokens]).
 * Host-only: validates, derives the token layout, the tile schedule and the fp64-computed cos/sin
 * tables.  Allocates no device memory.  theta = 10000.  Tensors are [B, N, heads, head_dim] with
 * N = text_len + T*H*W, contiguous.  *plan is written only on success; free with sol_attn3d_destroy.
 */
int sol_attn3d_plan(sol_attn3d_plan_t* plan, int B, int heads, int head_dim, int T, int H, int W,
                    int text_len, const int rope_dims[3]);

/* Same for a packed ragged batch and/or strided tensors ([total_tokens, heads, head_dim]). */
int sol_attn3d_plan_ex(sol_attn3d_plan_t* plan, const sol_attn3d_desc* desc);

/* Derived token offsets: *cu points at n_seqs+1 int64 values owned by the plan (host memory). */
int sol_attn3d_cu_seqlens(sol_attn3d_plan_t plan, const int64_t** cu, int* n_seqs);

/*
 * Device scratch the caller must provide (the library never allocates device memory).  Holds the
 * rotated Q and K (the rotary prologue writes them once per forward), the rotary tables, the
 * per-128-key-tile validity bits and a status word.
 */
size_t sol_attn3d_workspace_bytes(sol_attn3d_plan_t plan);

/*
 * Binds caller-owned device memory (256-byte aligned, >= workspace_bytes) to the plan and uploads
 * the plan's tables into it on the current device (synchronous copy; checks that the device is
 * compute capability 10.x).  The workspace must stay alive and untouched until the plan is
 * destroyed or rebound.  One plan supports one forward in flight at a time.
 */
int sol_attn3d_set_workspace(sol_attn3d_plan_t plan, void* device_ptr, size_t bytes);

/*
 * out = attention(q, k, v) as defined at the top of this file.  Steps, all enqueued on `stream`
 * without host synchronisation: key-validity bits per 128-key tile (Section 3.2 layout; only when
 * the mask may have changed), rotary prologue on Q and K (Section 3.5 group (2)), attention main
 * kernel (Section 3.2 "SDPA").
 *
 *   q, k, v, out  DEVICE pointers, bf16, [total_tokens, heads, head_dim] with the plan's strides,
 *                 16-byte aligned; q and k are UN-rotated.  out must not alias q, k or v.
 *   key_mask      DEVICE pointer, uint8 [total_tokens] (i.e. [B, N]), nonzero = attend; applies to
 *                 keys only, broadcast over heads and queries; NULL = all keys valid.
 *   K and V values at masked positions must be finite (0 * inf inside the tensor core is NaN).
 * The call only enqueues kernels (no allocation, no synchronisation, no host-device copy), so it may be
 * stream-captured into a CUDA graph and replayed (profiling off).
 * Results are deterministic: the same plan on the same inputs gives the same bits, whichever entry point or head
 * range is used.  Plans that differ in their number of heads walk the key tiles of a (head, query block) in
 * possibly different order at sizes beyond one wave of CTAs, so their results agree to rounding, not to the bit.
 * Errors: INVALID_ARG (NULL / misaligned pointer), NO_WORKSPACE, CUDA.  Device-side time-outs are
 * reported by sol_attn3d_status after the caller has synchronised the stream.
 */
int sol_attn3d_forward(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out,
                       const uint8_t* key_mask, sol_attn3d_stream_t stream);

/*
 * sol_attn3d_forward with the QK normalisation of the paper's fusion group (2) ("QK normalization with
 * partial RoPE", Section 3.5) done by the library's producer kernel: every (token, head) row of q and k is
 * RMS-normalised over head_dim in fp32,  y = x / sqrt(mean(x^2) + eps) * gain,  then rotated, and rounded
 * to bf16 once.  The paper prints no formula; per-head normalisation with one gain vector per tensor is
 * the reading taken.  V is not normalised.
 *   q_gain, k_gain  DEVICE pointers to head_dim fp32 values each (4-byte aligned), both required.
 *   eps             >= 0.
 * Everything else as for sol_attn3d_forward.  Errors: as sol_attn3d_forward, plus INVALID_ARG for a NULL gain.
 */
int sol_attn3d_forward_qknorm(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out,
                              const uint8_t* key_mask, const float* q_gain, const float* k_gain, float eps,
                              sol_attn3d_stream_t stream);

/*
 * The producer alone (fusion group (2) of Section 3.5: QK normalisation + partial RoPE): q_out / k_out
 * receive the normalised, rotated bf16 tensors, contiguous [total_tokens, heads, head_dim].  Either tensor
 * may be NULL together with its output; a tensor that is given needs its gain.  Needs a bound workspace
 * (tables).  Asynchronous on `stream`.
 */
int sol_attn3d_qknorm_rope(sol_attn3d_plan_t plan, const void* q, const void* k, const float* q_gain,
                           const float* k_gain, float eps, void* q_out, void* k_out, sol_attn3d_stream_t stream);

/*
 * Rectangular attention: fewer queries than keys.  Serves the reference-KV caching of the paper (section
 * "Caching Reference Tokens for Reference to Video Generation", paragraph "Reference KV caching mechanism":
 * after the first step the reference query rows are skipped, text and generated tokens attend to the cached
 * reference K/V and to each other): every token of the sequence is a key, but only the rows with
 * query_mask != 0 are computed and written.
 *   query_mask  DEVICE pointer, uint8 [total_tokens], nonzero = compute this query row.  Rows with 0 are
 *               not written (`out` keeps what it held); 256-row query blocks without any wanted row cost nothing.
 * Everything else as for sol_attn3d_forward; wanted rows get bit-identical results.  One extra tiny kernel per call.
 */
int sol_attn3d_forward_rect(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out,
                            const uint8_t* key_mask, const uint8_t* query_mask, sol_attn3d_stream_t stream);

/*
 * sol_attn3d_forward with the FP8 output format of Section 3.2 ("Quantized communication": the FP8
 * alternative transmits 128 raw E4M3 bytes per token/head, without scale metadata or padding; Section 3.3, "Joint
 * optimization with quantized communication": the raw E4M3 values returned by attention feed the quantized
 * output projection with unit scales).  The epilogue converts O/l from fp32 straight to E4M3 (round to
 * nearest even, magnitudes above 448 saturate, no bf16 step in between).
 *   out_e4m3   DEVICE pointer, uint8 [total_tokens, heads, head_dim] with the plan's out strides (counted
 *              in elements = bytes here), 16-byte aligned; rows of head_dim bytes.
 * Everything else as for sol_attn3d_forward.
 */
int sol_attn3d_forward_e4m3(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out_e4m3,
                            const uint8_t* key_mask, sol_attn3d_stream_t stream);

/*
 * Sequence-parallel exchange around the attention (Section 3.2, "Optimized attention collectives"): ranks
 * hold contiguous ranges of the flat token axis with all heads; attention needs every token for a shard of
 * the heads.  The paper's path is pack -> all-to-all -> attention -> all-to-all -> head merge with ONE
 * collective each way; the two layout kernels below are bit-exact copies of 16-byte chunks.
 */
#define SOL_ATTN3D_MAX_RANKS 8
#define SOL_ATTN3D_OUT_BF16 0
#define SOL_ATTN3D_OUT_E4M3 1
#define SOL_ATTN3D_OUT_INT8 2

/*
 * Sender's side, one pass: reads this rank's Q, K, V [n_local, heads, head_dim] (bf16, DEVICE) through their
 * element strides {token, head} ({0,0} = contiguous; views into a packed QKV buffer are fine) and writes, for
 * every destination g < n_ranks, heads [g*heads/n_ranks, (g+1)*heads/n_ranks) as rows
 *   dst[g][dst_row0 + t][which = q,k,v][heads/n_ranks][head_dim].
 *   dst        HOST array of n_ranks DEVICE pointers, 16-byte aligned, caller-owned.  Either slices of one
 *              local send buffer with dst_row0 = 0 (then one all-to-all follows), or the ranks' receive
 *              buffers mapped into this process (peer memory) with dst_row0 = this rank's first token: the
 *              pack and the transfer are then the same pass of plain peer stores, and the caller needs a
 *              barrier across ranks before the attention reads the buffer.
 * After the exchange rank g holds [total_tokens][3][heads/n_ranks][head_dim]; its Q, K, V are views with
 * token stride 3*heads/n_ranks*head_dim that sol_attn3d_plan_ex takes as they are.
 *   group_begin, group_heads   send only heads [group_begin, group_begin + group_heads) of every rank's shard (a head
 *              group; rows then hold group_heads heads), so that the exchange of one group can run under the
 *              attention of another; 0, 0 = the whole shard.
 * n_local = 0 is a no-op (pointers are not looked at).
 * Errors: INVALID_ARG (NULL / misaligned pointer, heads not divisible, n_ranks > SOL_ATTN3D_MAX_RANKS), CUDA.
 */
int sol_attn3d_exchange_pack_qkv(const void* q, const void* k, const void* v, const int64_t q_strides[2],
                                 const int64_t k_strides[2], const int64_t v_strides[2], int64_t n_local, int heads,
                                 int head_dim, int n_ranks, int group_begin, int group_heads, void* const* dst,
                                 int64_t dst_row0, sol_attn3d_stream_t stream);

/*
 * Receiver's side of the output return (the paper's "inverse head merge"): recv [n_ranks][n_local]
 * [heads/n_ranks][record_bytes] (DEVICE; slice g = what rank g computed for this rank's tokens) ->
 * out [n_local][heads][record_bytes] with head = g*heads/n_ranks + local head, the row-major input of the
 * output projection.  record_bytes is the size of one (token, head) record on the wire, a multiple of 16:
 * 2*head_dim for bf16, head_dim for raw E4M3.  out_tok_stride_bytes: 0 = dense.  recv and out must not alias.
 * out_rank_stride_bytes: distance between rank g's and rank g+1's heads inside an output row; 0 = adjacent
 * (heads/n_ranks * record_bytes).  When recv holds one head group of every rank, pass the full shard's size here
 * and point `out` at the group's first head: the group lands in its place in the full row.
 */
int sol_attn3d_exchange_merge_heads(const void* recv, void* out, int64_t n_local, int heads, int record_bytes,
                                    int n_ranks, int64_t out_tok_stride_bytes, int64_t out_rank_stride_bytes,
                                    sol_attn3d_stream_t stream);

/*
 * Quantized wire formats of the exchange (Section 3.2, "Quantized communication").  One record per (token,
 * head); head_dim 64 or 128:
 *   QKV block-INT8   [q int8 x D | k int8 x D | v int8 x D | D/32 q scale codes | D/32 k codes | D/32 v codes |
 *                    zeros to a multiple of 16 bytes]                      D = 128: 384 + 12 + 4 = 400 bytes
 *   out block-INT8   [o int8 x D | D/32 scale codes | zeros to a multiple of 16 bytes]   D = 128: 144 bytes
 *   out E4M3         D raw bytes (sol_attn3d_forward_e4m3 writes them; no kernel here)
 * Scale code: unsigned 8-bit float, 5 exponent bits (bias 15), 3 mantissa bits (value (8+m) * 2^(e-18), or
 * m * 2^-17 for e = 0), one per group of 32 values; only finite positive codes 0x01..0xf7 are written.  The
 * paper fixes the record sizes and the scale format; the rule is this library's: scale = smallest value s with
 * 127 * s >= max|x| of the group (nothing clips; all-zero group -> 0x01), q = clamp(rint(x * (1/s)), -127, 127)
 * with the reciprocal and the product rounded to fp32 (round to nearest even), value = q * s.  All padding
 * bytes are written.  Both formats are approximate.
 */
#define SOL_ATTN3D_WIRE_QKV_BF16 0
#define SOL_ATTN3D_WIRE_QKV_INT8 1
#define SOL_ATTN3D_WIRE_OUT_BF16 2
#define SOL_ATTN3D_WIRE_OUT_E4M3 3
#define SOL_ATTN3D_WIRE_OUT_INT8 4
/* Bytes of one (token, head) record of the given kind; 0 for an unknown kind or head_dim. */
size_t sol_attn3d_exchange_record_bytes(int kind, int head_dim);

/*
 * sol_attn3d_exchange_pack_qkv that quantises on the way: same arguments and destinations, but destination g
 * receives records  dst[g][dst_row0 + t][heads/n_ranks][record_bytes(QKV_INT8)]  (one pass: bf16 in, records out).
 */
int sol_attn3d_exchange_pack_qkv_int8(const void* q, const void* k, const void* v, const int64_t q_strides[2],
                                      const int64_t k_strides[2], const int64_t v_strides[2], int64_t n_local, int heads,
                                      int head_dim, int n_ranks, int group_begin, int group_heads, void* const* dst,
                                      int64_t dst_row0, sol_attn3d_stream_t stream);

/*
 * Receiver's side: records [n_rows][heads][record_bytes(QKV_INT8)] (DEVICE; heads = this rank's shard) -> qkv
 * bf16 [n_rows][3][heads][head_dim] (DEVICE, 16-byte aligned, caller-owned), the packed tensor whose three
 * strided views feed sol_attn3d_forward.  q * s is exact in fp32 and rounded once to bf16.
 */
int sol_attn3d_exchange_unpack_qkv_int8(const void* records, void* qkv, int64_t n_rows, int heads, int head_dim,
                                        sol_attn3d_stream_t stream);

/*
 * Output rows bf16 [n_rows][heads][head_dim] (element strides {token, head}, {0,0} = dense) -> records
 * [n_rows][heads][record_bytes(OUT_INT8)]; and back to dense bf16 rows.  Records travel through
 * sol_attn3d_exchange_merge_heads like any other record (record_bytes = 144 for head_dim 128).
 */
int sol_attn3d_exchange_quantize_out_int8(const void* out_rows, const int64_t out_strides[2], int64_t n_rows, int heads,
                                          int head_dim, void* records, sol_attn3d_stream_t stream);
int sol_attn3d_exchange_dequantize_out_int8(const void* records, void* out_rows, int64_t n_rows, int heads, int head_dim,
                                            sol_attn3d_stream_t stream);

/*
 * sol_attn3d_forward with the block-INT8 output format of Section 3.2 ("Quantized communication": a 144-byte record
 * per token and head at head_dim 128) written by the attention epilogue itself, the kind of fusion that Section 3.3
 * ("Joint optimization with quantized communication") aims at: the bf16 rows are never written or re-read.  The values are
 * rounded to bf16 and quantised by the rule stated above, so the records are byte for byte those of
 * sol_attn3d_forward followed by sol_attn3d_exchange_quantize_out_int8.
 *   out_records  DEVICE pointer, dense [total_tokens][heads][sol_attn3d_exchange_record_bytes(OUT_INT8, head_dim)]
 *                bytes, 16-byte aligned (the plan's output strides, which describe bf16 rows, do not apply).
 * Everything else as for sol_attn3d_forward.  Rows of a sequence without any valid key become records of zeros.
 */
int sol_attn3d_forward_int8(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out_records,
                            const uint8_t* key_mask, sol_attn3d_stream_t stream);

/*
 * sol_attn3d_forward fed by the block-INT8 QKV records of the exchange (Section 3.2, "Quantized communication"): the
 * receiver's dequantisation is fused into the rotary producer (Section 3.3, "Joint optimization with quantized communication"),
 * so the packed bf16 QKV tensor is never written or re-read.  Each value is q * s rounded to bf16, exactly what
 * sol_attn3d_exchange_unpack_qkv_int8 would have stored, and Q, K are rotated from there: the result is bit for bit
 * that of unpack followed by sol_attn3d_forward on the unpacked views.
 *   qkv_records  DEVICE pointer, dense [total_tokens][heads][record_bytes(QKV_INT8, head_dim)], 16-byte aligned
 *                (heads = this plan's heads, e.g. a rank's shard after the all-to-all).
 *   v_scratch    DEVICE pointer, caller-owned bf16 [total_tokens][heads][head_dim], 16-byte aligned: the producer
 *                writes the dequantised V there and the attention kernel reads it (rotated Q and K go to the plan's
 *                workspace as always).  Undefined afterwards.
 *   out          as the output of sol_attn3d_forward (out_format BF16, plan's output strides),
 *                sol_attn3d_forward_e4m3 (E4M3) or sol_attn3d_forward_int8 (INT8).
 * The plan's q / k / v strides do not apply.  Everything else as for sol_attn3d_forward.
 */
int sol_attn3d_forward_qkv_int8(sol_attn3d_plan_t plan, const void* qkv_records, void* v_scratch, void* out,
                                const uint8_t* key_mask, int out_format, sol_attn3d_stream_t stream);

/*
 * sol_attn3d_forward whose epilogue delivers each output row to the owner of its token: the output return
 * of the exchange and the head merge fused into the attention kernel (no counterpart kernel in the paper,
 * which returns the output with a collective; same result).  The plan describes this rank's head shard
 * over all tokens.  Destination g owns flat tokens [tok_begin[g], tok_begin[g+1]) and receives them as rows
 *   dst[g][token - tok_begin[g]][head_offset + h][head_dim],   row stride dst_heads * head_dim elements.
 *   n_dst       1 .. SOL_ATTN3D_MAX_RANKS.
 *   dst         HOST array of n_dst DEVICE pointers (this GPU's memory or a peer's mapped into this process;
 *               plain stores, whole 16-byte chunks of contiguous rows), 16-byte aligned; may be NULL for an
 *               owner without tokens.
 *   tok_begin   HOST array of n_dst+1 ascending token offsets, tok_begin[0] = 0, tok_begin[n_dst] = total.
 *   dst_heads   heads per row in the destinations (all ranks' shards); head_offset = this shard's first head.
 *   out_format  SOL_ATTN3D_OUT_BF16, SOL_ATTN3D_OUT_E4M3 (see sol_attn3d_forward_e4m3) or SOL_ATTN3D_OUT_INT8 (see
 *               sol_attn3d_forward_int8; a destination row then holds dst_heads records instead of dst_heads * head_dim
 *               elements).
 * The arrays are read during the call only.  The caller needs a barrier across ranks before the owners
 * read their rows.  Everything else as for sol_attn3d_forward.
 */
int sol_attn3d_forward_scatter(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v,
                               const uint8_t* key_mask, int n_dst, void* const* dst, const int64_t* tok_begin,
                               int dst_heads, int head_offset, int out_format, sol_attn3d_stream_t stream);

/*
 * sol_attn3d_forward on HOST buffers: q, k, v are read from and out is written to host memory (pinned, or the
 * copies will not overlap), through caller-owned device staging memory.  The heads are served in n_groups
 * groups (heads are independent): the host-to-device copy of group g+1 and the device-to-host copy of group
 * g-1 run on two internal streams while the kernels of group g run, so that only the first group's inputs and
 * the last group's outputs are exposed.  The kernels of even groups run on `stream`, those of odd groups on a
 * third internal stream, so that a group's kernels fill the SMs that the last wave of its predecessor leaves
 * idle.  On return everything is enqueued; `stream` has been made to wait for the last device-to-host copy, so
 * synchronising `stream` is enough before reading out.
 *   q_host, k_host, v_host, out_host   HOST pointers, bf16, dense [total_tokens, heads, head_dim] (the plan must use
 *                  the default strides); key_mask_host HOST uint8 [total_tokens] or NULL.
 *   staging        DEVICE memory, 256-byte aligned, >= sol_attn3d_host_staging_bytes(plan) (four tensors and the
 *                  mask), caller-owned, must stay untouched until `stream` has passed this call.
 *   n_groups       1 .. 8 equal groups (clamped to the number of heads); 0 = default: eight groups of growing and then
 *                  shrinking size (a small first group, whose inputs are exposed, and a small last one, whose outputs are).
 * The first call creates three streams and a few events (no device memory); sol_attn3d_destroy releases them.
 * Result: bit-identical to sol_attn3d_forward on device copies of the same tensors.
 * Errors: INVALID_ARG, NO_WORKSPACE (plan workspace or staging), UNSUPPORTED_SHAPE (strided plan), CUDA.
 */
size_t sol_attn3d_host_staging_bytes(sol_attn3d_plan_t plan);
int sol_attn3d_forward_host(sol_attn3d_plan_t plan, const void* q_host, const void* k_host, const void* v_host,
                            void* out_host, const uint8_t* key_mask_host, void* staging, size_t staging_bytes,
                            int n_groups, sol_attn3d_stream_t stream);

/*
 * Block-sparse variant of sol_attn3d_forward: the per-step dynamic sparsity of Section 3.4 ("Sparse
 * Attention") with its safety rails.  An approximation of dense attention.
 *   Query blocks of 256 tokens, KV blocks of 128 tokens, per sequence and head.  Block-level score =
 *   <mean of rotated q over the query block, mean of rotated k over the KV block> / sqrt(head_dim) (the
 *   paper does not print the block statistic: mean-pooled logits of the bf16 operands are the reading
 *   taken).  Per query block, mu and sigma are the mean and (population) standard deviation of its scores
 *   over all KV blocks; a KV block is attended iff score > mu + tau * sigma.  Rails: KV blocks holding a
 *   prefix token are always attended (exact prefix sink); query blocks holding a prefix token attend
 *   densely; the best-scoring block is always kept.  The softmax runs over the valid keys of the
 *   attended blocks only.  The paper's schedule uses tau = 1.0, 1.25, 1.5 for its three refinement steps
 *   and keeps the first two layers dense (call sol_attn3d_forward for those).
 *   sparse_ws  caller-owned DEVICE scratch of sol_attn3d_sparse_workspace_bytes(plan) bytes, 256-byte
 *              aligned (pooled operands, per-CTA key-tile lists, counters); one forward in flight per buffer.
 * Everything else as for sol_attn3d_forward (the plan's workspace must be bound).  Extra kernels per call:
 * two pooling kernels and one selection kernel per sequence.
 */
size_t sol_attn3d_sparse_workspace_bytes(sol_attn3d_plan_t plan);
int sol_attn3d_forward_sparse(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out,
                              const uint8_t* key_mask, float tau, void* sparse_ws, size_t sparse_ws_bytes,
                              sol_attn3d_stream_t stream);
/* After the stream has drained: attended / total (query block, KV block) pairs of the last sparse forward
 * on this scratch (synchronous 16-byte copy). */
int sol_attn3d_sparse_stats(sol_attn3d_plan_t plan, const void* sparse_ws, long long* selected_tiles,
                            long long* all_tiles);
/* After the stream has drained: the ascending KV-block list of one (sequence, head, query block) of the last
 * sparse forward (synchronous copies; for inspection and tests).  *count receives the full length. */
int sol_attn3d_sparse_selection(sol_attn3d_plan_t plan, const void* sparse_ws, int seq, int head, int query_block,
                                int* kv_blocks, int capacity, int* count);

/*
 * sol_attn3d_forward for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a deployment variant of the call above, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- an inference plugin whose host
 * framework owns all device memory and forbids allocation inside its enqueue hook, a real-time loop
 * that may not touch the allocator after start-up, a process whose memory has been handed over
 * completely to another pool.  Such a caller cannot provide the workspace that sol_attn3d_forward wants.
 * Here the scratch (rotated Q and K, rotary tables, sequence table, key-validity bits) is a 32 MiB
 * array built into the library image, so the caller passes only inputs and outputs.  Every GPU context
 * that loads the library holds those 32 MiB until the process ends, whether this function is used or not.
 *
 *   plan           any plan with sol_attn3d_workspace_bytes(plan) <= 32 MiB (33,554,432 bytes); larger
 *                  plans are refused with SOL_ATTN3D_ERR_SCRATCH_LIMIT before anything is enqueued.
 *                  No workspace needs to be bound.
 *   q, k, v, out, key_mask, stream   exactly as for sol_attn3d_forward.
 *   device_status  optional DEVICE pointer to one 4-byte word (4-byte aligned) that receives the status
 *                  word of this call: zeroed on `stream` first, nonzero after the stream has drained if
 *                  a bounded wait inside a kernel ran out (then `out` is undefined).  With NULL the
 *                  word stays inside the built-in array and cannot be read; sol_attn3d_status does not
 *                  see this path.
 *
 * The function calls no cudaMalloc, cudaFree or other allocating routine, neither directly nor through
 * a library.  The first call on each device looks up the device address of the built-in array
 * (cudaGetSymbolAddress), raises the kernels' shared-memory limit and resolves one driver entry
 * point; do that first call with the device current and before any stream capture begins.  If the CUDA
 * runtime loads modules lazily, that first call is also where the driver places the library's code and
 * the 32 MiB array on the device; later calls find device memory unchanged.  Later calls only enqueue
 * work: a 4-byte memset, two small host-to-device copies of the plan's tables (a few KB to a few hundred
 * KB, read from ordinary pageable host memory owned by the plan), and three kernels.  Keep the plan alive
 * until `stream` has passed the call.
 *
 * All calls on a device share the one array and it keeps the previous call's contents.  Everything a
 * call reads from it is rewritten by that call first (the status word is cleared, tables are copied
 * in again, rotated Q/K and key bits are recomputed), so calls that follow one another on a stream,
 * also with different plans, are independent.  Calls that OVERLAP on the GPU (different streams, or
 * host threads racing on the same device) corrupt each other's scratch: serialise them.
 * Errors: INVALID_ARG, SCRATCH_LIMIT, NO_DEVICE, UNSUPPORTED_ARCH, CUDA.
 */
int sol_attn3d_forward_noalloc(sol_attn3d_plan_t plan, const void* q, const void* k, const void* v, void* out,
                               const uint8_t* key_mask, unsigned int* device_status, sol_attn3d_stream_t stream);

/*
 * The rotary prologue alone (Section 3.5 group (2), rotation part): q_rot / k_rot receive the rotated
 * bf16 tensors, contiguous [total_tokens, heads, head_dim].  DEVICE pointers, 16-byte aligned; either
 * input may be NULL together with its output.  Needs a bound workspace (tables).  Asynchronous.
 */
int sol_attn3d_rope_qk(sol_attn3d_plan_t plan, const void* q, const void* k, void* q_rot, void* k_rot,
                       sol_attn3d_stream_t stream);

/*
 * Reads the device status word (synchronous 4-byte copy; call after synchronising the stream).
 * 0 = no fault; SOL_ATTN3D_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up, in which
 * case `out` is undefined.  The word is cleared by the next sol_attn3d_set_workspace.
 */
int sol_attn3d_status(sol_attn3d_plan_t plan);

/*
 * The raw status word behind sol_attn3d_status (same synchronous copy).  Low byte: 0 = fine, 1..3 = a bounded wait
 * of the producer / MMA issuer / softmax warps ran out, 5 = a device-side index check failed; for 5 the upper 24
 * bits name the check.  The checks exist only in the debug build of the library (compiled with
 * -DSOL_ATTN3D_DEBUG=1; sol_attn3d_debug_build() returns 1 there): work-item decoding, key-tile numbers and counts
 * taken from the lists, output-row addresses, the token -> sequence lookup of the rotary producer (the layout of
 * Section 3.2 / 3.4 is where an indexing mistake would show).  A failing check records itself and execution goes
 * on: nothing traps, the kernel returns.  SOL_ATTN3D_ERR_DEVICE_ASSERT is what sol_attn3d_status then returns.
 */
int sol_attn3d_status_word(sol_attn3d_plan_t plan, unsigned int* word);
int sol_attn3d_debug_build(void);

/*
 * Per-kernel timing for roofline accounting (Section 3.2 times "SDPA" apart from the layout work
 * around it).  enable != 0 creates four CUDA events owned by the plan; every later forward records
 * them on its stream around its three steps.  sol_attn3d_last_forward_ms blocks on the last event
 * (cudaEventSynchronize) and writes ms[0..2] = {key-validity bits, rotary prologue, attention kernel}
 * of the most recent forward (0 for a step that was skipped).  Returns INVALID_ARG if profiling is
 * off or no forward ran.  enable == 0 destroys the events.
 */
int sol_attn3d_set_profiling(sol_attn3d_plan_t plan, int enable);
int sol_attn3d_last_forward_ms(sol_attn3d_plan_t plan, float ms[3]);

/*
 * Number of kernels the most recent forward-type call on this plan enqueued (any sol_attn3d_forward* entry point,
 * sol_attn3d_rope_qk, sol_attn3d_qknorm_rope), counted as they were launched: the dense forward launches 2 (rotary
 * prologue, attention) plus 1 when the key-validity bits are rebuilt; the block-sparse forward adds 3 per sequence,
 * the rectangular one 1, and sol_attn3d_forward_host launches one such set per head group.  Host-side counter, no
 * device access.  For launch accounting in benchmarks (Section 3.2 counts launches around "SDPA").
 */
int sol_attn3d_last_launch_count(sol_attn3d_plan_t plan);

/*
 * Diagnostic for the online softmax (the running-maximum form of the softmax in Section 3.2's "SDPA"; the paper does
 * not describe it): the attention kernel exponentiates each 128-key tile against a reference maximum per query
 * row and moves that reference only when a tile's row maximum exceeds it by more than 2^8 (then the partial
 * output and row sum are rescaled).  *count receives how often that happened, in (warp of 32 query rows, key
 * tile) events, since the workspace was bound (sol_attn3d_set_workspace resets it).  Synchronous 4-byte copy;
 * call after synchronising the stream.  Tests use it to prove that inputs built to move the maximum did so.
 */
int sol_attn3d_softmax_rescale_count(sol_attn3d_plan_t plan, unsigned long long* count);

/* cudaError_t of the last failing CUDA call made on behalf of this plan (0 if none). */
int sol_attn3d_last_cuda_error(sol_attn3d_plan_t plan);

/* Static string for an error code. */
const char* sol_attn3d_strerror(int code);

/* Frees host state.  Never frees caller memory.  NULL is a no-op.  Does not synchronise. */
int sol_attn3d_destroy(sol_attn3d_plan_t plan);

#ifdef __cplusplus
}
#endif
#endif /* SOL_ATTN3D_H_ */
