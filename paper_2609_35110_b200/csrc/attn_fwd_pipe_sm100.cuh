// Attention main kernel, "pipelined" form: ONE 128-row query tile per CTA, two score buffers and two P buffers in
// tensor memory.
//
// The two-tile kernel (attn_fwd_sm100.cuh) keeps one score buffer per query tile and writes P over it, so the QK^T
// of a tile's next key block can only start after the softmax of the current one has finished and its P has been
// consumed: every key block pays the whole chain  S -> softmax -> P -> PV -> QK  in sequence.  Here P has buffers of
// its own, so a score buffer is free again as soon as the softmax has read it into registers: the tensor core
// computes S(j+2) while the softmax works on S(j) and S(j+1), the softmax warps do not wait for the tensor core
// and the hand-over latencies are off the critical path.  The price is that a K / V tile serves 128 query rows
// instead of 256; CTA pairs (kCtas = 2) buy that back: the two CTAs of a cluster take the two 128-row tiles of a
// 256-row query block, each loads HALF of every K / V tile, and one tcgen05.mma.cta_group::2 of M = 256 works on
// both (issued by the even CTA, completion multicast to both).  Nothing is loaded with multicast.
//
// Work item = (sequence, head, 256-row query block), exactly as in the two-tile kernel; CTA 2u and 2u+1 of the
// grid take its two tiles (as a cluster when kCtas = 2, independently otherwise).
//
// Warp roles (384 threads):
//   warps 0-3  softmax of the EVEN key blocks of the tile (thread = one query row), and the epilogue
//   warps 4-7  softmax of the ODD key blocks (warp w + 4 owns the same 32 rows as warp w and sits on the same
//              scheduler: while one of the two waits for tensor memory or a barrier, the other keeps the
//              special-function unit busy)
//   warp  8    TMA producer (lane 0)
//   warp  9    tcgen05.mma issuer (whole warp convergent, one elected lane issues); owns the TMEM allocation
//   warps 10-11 idle (complete the third warpgroup)
// Tensor memory (512 columns): S0 | S1 (128 columns each, fp32) | P0 | P1 (64 columns each, bf16 pairs) | O (D
// columns).  Key block i uses S[i % 2] and P[i % 2].
//
// Online softmax over two warpgroups.  Both exponentiate against a per-row reference maximum that only ever grows
// (lazily: by more than 2^8 or not at all, see the two-tile kernel).  The key blocks are FINALISED in order: the
// warp that owns block i hands its P over only after its partner has finalised block i-1 and published the
// reference it ended with.  If that reference differs from the one block i was exponentiated against (rare), the
// block is redone from the scores still in registers; if block i itself needs a larger reference (rare), its
// owner rescales O (after PV(i-1)) and publishes the new one.  Each warpgroup keeps the row sum of its own blocks;
// the two are brought to the final reference and added in the epilogue.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "attn_fwd_sm100.cuh"

namespace sol {

// SOL_PIPE_PROF=1 (experiments only): per-role wait cycles summed over all CTAs into 64-bit words after the
// counters word: [1] softmax wait for S, [2] softmax loop, [3] MMA wait V, [4] MMA wait P, [5] MMA wait K,
// [6] MMA loop, [7] producer wait for a free stage, [8] producer loop, [9] CTAs counted.
#ifndef SOL_PIPE_PROF
#define SOL_PIPE_PROF 0
#endif
#if SOL_PIPE_PROF
#define SOL_PROF_T(var) const long long var = clock64()
#define SOL_PROF_ADD(acc, t0) acc += clock64() - (t0)
#define SOL_PROF_OUT(idx, v) atomicAdd(reinterpret_cast<unsigned long long*>(p.counters) + (idx), (unsigned long long)(v))
#else
#define SOL_PROF_T(var)
#define SOL_PROF_ADD(acc, t0)
#define SOL_PROF_OUT(idx, v)
#endif

constexpr int kPipeThreads = 384;
constexpr int kPipeBufs = 2;

template <int D, int kCtas>
struct PipeSmem {
  static constexpr int kTile = 128 * D * 2;               // bytes of one 128 x D bf16 tile
  static constexpr int kHalves = D / 64;                  // 64-column (128-byte) swizzle boxes per row
  static constexpr int kHalfBytes = 128 * 128;            // one box: 128 rows x 128 bytes
  static constexpr int kStageBytes = kTile / kCtas;       // what one CTA holds of a K or V tile
  static constexpr int kKBoxBytes = kHalfBytes / kCtas;   // one K box: (128 / kCtas) keys x 128 bytes
  static constexpr int kStages = (D == 128 ? 6 : 12) * (kCtas == 2 ? 10 : 6) / 6;   // K/V ring
  static constexpr int kOffQ = 0;
  static constexpr int kOffKV = kTile;
  static constexpr int kOffBars = kOffKV + kStages * kStageBytes;
  // q_full, kv_full/empty, s_full[2], p_full[2], o_done[2], s_free[2], drain, fin[4 row groups][2 warpgroups]
  static constexpr int kNumBars = 1 + 2 * kStages + 4 * kPipeBufs + 1 + 8;
  static constexpr int kOffTmemPtr = kOffBars + kNumBars * 8;
  static constexpr int kOffRef = kOffTmemPtr + 16;        // float[128]: reference maximum per row as of the last finalised block
  static constexpr int kOffSum = kOffRef + 128 * 4;       // float2[128]: (row sum, its reference) of the odd-block warpgroup
  static constexpr int kBytes = kOffSum + 128 * 8;
  static constexpr int kDynBytes = kBytes + 1024;         // slack to align the base to 1024 bytes
};

template <int D, int kCtas>
__global__ void __launch_bounds__(kPipeThreads, 1)
attn_fwd_pipe_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
  static_assert(kCtas == 1 || (kCtas == 2 && D == 128), "CTA pairs are built for head_dim 128");
  using L = PipeSmem<D, kCtas>;
  constexpr bool kPair = kCtas == 2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t sbase = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (sbase - raw_addr);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // which of the block's two 128-row tiles; in a pair, rank 0 is the leader (issues the MMAs, owns the barriers the
  // other CTA reports to)
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const bool leader = rank == 0;
  const int half = kPair ? (int)rank : ((int)blockIdx.x & 1);

  const uint32_t sQ = sbase + L::kOffQ;
  const uint32_t sKV = sbase + L::kOffKV;
  const uint32_t bars = sbase + L::kOffBars;
  const uint32_t bar_q_full = bars;
  auto bar_kv_full = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_kv_empty = [&](int s) { return bars + 8u * (1 + L::kStages + s); };
  auto bar_s_full = [&](int b) { return bars + 8u * (1 + 2 * L::kStages + b); };
  auto bar_p_full = [&](int b) { return bars + 8u * (1 + 2 * L::kStages + kPipeBufs + b); };
  // "PV of a key block that used P buffer b has completed" (P[b] may be overwritten, O holds that block).  One
  // barrier per buffer, not one for all: a waiter may be two PVs behind the tensor core, and an mbarrier phase can
  // only be told from its neighbour.
  auto bar_o_done = [&](int b) { return bars + 8u * (1 + 2 * L::kStages + 2 * kPipeBufs + b); };
  // "the softmax has read S[b] into registers": the tensor core may overwrite it
  auto bar_s_free = [&](int b) { return bars + 8u * (1 + 2 * L::kStages + 3 * kPipeBufs + b); };
  const uint32_t bar_drain = bars + 8u * (1 + 2 * L::kStages + 4 * kPipeBufs);
  // "warp (g, q) has finalised its latest key block": waited on by its partner warp (1 - g, q)
  auto bar_fin = [&](int q, int g) { return bars + 8u * (2 + 2 * L::kStages + 4 * kPipeBufs + 2 * q + g); };
  volatile float* ref_smem = reinterpret_cast<volatile float*>(smem + L::kOffRef);
  volatile float* sum_smem = reinterpret_cast<volatile float*>(smem + L::kOffSum);   // [2 * row] sum, [2 * row + 1] its reference
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + L::kOffTmemPtr);

  // ---- which work item
  const int unit = (int)blockIdx.x / 2 + p.cta_offset;
  int si = 0;
  while (si + 1 < p.n_seqs && unit >= p.seqs[si + 1].work_start) ++si;
  const SeqDev sq = p.seqs[si];
  const int local = unit - sq.work_start;
  const int head = local / sq.n_qpairs;
  const int blk = local - head * sq.n_qpairs;           // 256-row query block
  // a launch may serve a range of heads only (uniform over the block's two CTAs, before any set-up)
  if (head < p.head_begin || head >= p.head_end) return;
  // rectangular mode: a query block without a wanted row has nothing to do (uniform, before any set-up)
  if (p.pair_needed != nullptr && p.pair_needed[sq.pair_start + blk] == 0) return;
  const int q_row0 = blk * 256 + half * 128;            // first local query row of this CTA
  // an independent CTA whose tile lies wholly beyond the sequence has nothing to do (in a pair it must stay: the
  // leader's MMAs cover both CTAs)
  if (!kPair && q_row0 >= sq.n_tokens) return;
  // dense: every CTA of a sequence walks the same list of key tiles; block-sparse: one list per 256-row query block
  const bool sparse = p.cta_list != nullptr;
  const int n_proc = sparse ? p.cta_count[unit] : p.ktile_count[si];
  const int* __restrict__ ktiles =
      sparse ? p.cta_list + sq.sparse_list_start + (long long)local * sq.n_ktiles : p.ktile_list + sq.ktile_start;
  const uint4* __restrict__ keybits = p.keybits + sq.ktile_start;
  // Successive waves of CTAs walk the key tiles in opposite directions (the softmax does not care about the order):
  // a wave then starts on the tiles its predecessor touched last, which are still in L2.
  const bool backwards = ((unit / max(1, p.wave_ctas / 2)) & 1) != 0;
  auto tile_at = [&](int i) { return __ldg(&ktiles[backwards ? n_proc - 1 - i : i]); };
  const int tok0 = (int)sq.tok_start;                   // TMA token coordinate of the sequence start
  const unsigned long long limit = p.wait_limit_ns;

  if (warp == 8 && lane == 0) {
    mbar_init(bar_q_full, 1);
    for (int s = 0; s < L::kStages; ++s) {
      mbar_init(bar_kv_full(s), 1);
      mbar_init(bar_kv_empty(s), 1);
    }
    for (int b = 0; b < kPipeBufs; ++b) {
      mbar_init(bar_s_full(b), 1);
      mbar_init(bar_p_full(b), 4 * kCtas);              // one arrival per softmax warp of the block, from every CTA of the pair
      mbar_init(bar_s_free(b), 4 * kCtas);
      mbar_init(bar_o_done(b), 1);
    }
    mbar_init(bar_drain, 1);
    for (int q = 0; q < 4; ++q)
      for (int g = 0; g < 2; ++g) mbar_init(bar_fin(q, g), 1);
    fence_mbar_init();
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_k);
    prefetch_tensormap(&tm_v);
  }
  // A fault recorded by an earlier CTA stops later ones at the door (read once; made uniform over the pair below).
  if (threadIdx.x == 0) tmem_ptr_smem[1] = *reinterpret_cast<volatile unsigned int*>(p.status);
  if (warp == 9) {
    if (kPair) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), 512); tmem_relinquish_pair(); }
    else       { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), 512); tmem_relinquish(); }
  }
  tc_fence_before();
  if (kPair) cluster_sync_all(); else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_ptr_smem[0];
  {
    uint32_t stop = tmem_ptr_smem[1];
    if (kPair) {
      // both CTAs must take the same decision: each looks at both flags, and nobody leaves before the other has looked
      stop |= ld_shared_cluster_u32(mapa_shared(smem_u32(const_cast<uint32_t*>(&tmem_ptr_smem[1])), rank ^ 1u));
      cluster_sync_all();
    }
    if (stop != 0) {
      if (warp == 9) {
        if (kPair) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512);
      }
      return;
    }
  }
  const uint32_t tP_base = tmem_base + kPipeBufs * 128;   // P0 | P1, 64 columns each
  const uint32_t tO_base = tP_base + kPipeBufs * 64;

  if (warp < 8) {
    // =========================================================== softmax / correction / epilogue
    setmaxnreg_inc<SOL_REGS_SOFTMAX>();
    const int g = warp >> 2;                             // warpgroup: key blocks g, g + 2, g + 4, ...
    const int q = warp & 3;                              // row group: rows 32 q .. 32 q + 31 (tensor-memory lanes)
    const int row = q * 32 + lane;
    const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
    const uint32_t tO = tO_base + lane_off;
    const float c = p.scale_log2;
    float m_ref = -CUDART_INF_F;
    float l = 0.f;
    bool ok = true;
    long long prof_wait = 0, prof_a = 0, prof_b = 0, prof_c = 0, prof_d = 0, prof_e = 0;
    SOL_PROF_T(prof_t0);

    // Validity bits of this warpgroup's blocks are fetched one block ahead and their tile numbers two blocks ahead,
    // so that neither load (the second depends on the first) is waited for inside a block.
    uint4 kb_next = g < n_proc ? __ldg(&keybits[tile_at(g)]) : make_uint4(0u, 0u, 0u, 0u);
    int jt_next = g + 2 < n_proc ? tile_at(g + 2) : 0;
    for (int i = g; i < n_proc; i += 2) {
      const int b = i % kPipeBufs;                       // score buffer of key block i
      const uint32_t use = (uint32_t)(i / kPipeBufs);    // how often that buffer has been used before
      const uint4 kb = kb_next;
      if (i + 2 < n_proc) kb_next = __ldg(&keybits[jt_next]);
      if (i + 4 < n_proc) jt_next = tile_at(i + 4);
      const uint32_t tS = tmem_base + lane_off + b * 128;
      const uint32_t tP = tP_base + lane_off + b * 64;
      if (i == 1) {
        // the odd warpgroup's first block: exponentiate against the reference that block 0 ended with
        ok = __all_sync(0xffffffffu, mbar_wait(bar_fin(q, 0), 0u, limit));
        if (!ok) break;
        m_ref = ref_smem[row];
      }
      SOL_PROF_T(prof_w0);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full(b), use & 1u, limit));
      SOL_PROF_ADD(prof_wait, prof_w0);
      if (!ok) break;
      tc_fence_after();

      const bool mixed = (kb.x & kb.y & kb.z & kb.w) != 0xffffffffu;
      uint32_t r[128];
      uint32_t pk[64];
      float tile_sum;
      bool first_half_stored = false;
      SOL_PROF_T(prof_s1);
      // the whole row of scores into registers, then S[b] goes back to the tensor core at once: S(i+2) is computed
      // while this block is exponentiated (the partner warp on this scheduler covers the load latency)
#pragma unroll
      for (int cch = 0; cch < 4; ++cch) tmem_ld32(tS + cch * 32, *reinterpret_cast<uint32_t(*)[32]>(&r[cch * 32]));
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_cluster(mapa_shared(bar_s_free(b), 0)); else mbar_arrive(bar_s_free(b));
      }
      SOL_PROF_ADD(prof_a, prof_s1);
      // P[b] still feeds PV(i-2) until that has completed: checked right before the first store into it
      auto p_buffer_free = [&]() {
        return i < 2 || __all_sync(0xffffffffu, mbar_wait(bar_o_done(b), (uint32_t)((i - 2) >> 1) & 1u, limit));
      };
      SOL_PROF_T(prof_s3);
      if (!mixed && i > 0) {
        // Common case, in two halves: the first half of P is on its way to tensor memory while the second is computed
        uint32_t (&r_lo)[64] = *reinterpret_cast<uint32_t(*)[64]>(&r[0]);
        uint32_t (&r_hi)[64] = *reinterpret_cast<uint32_t(*)[64]>(&r[64]);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const float mc = m_ref * c;
        softmax_half(r_lo, c, mc, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]), acc);
        SOL_PROF_T(prof_s2);
        ok = p_buffer_free();
        SOL_PROF_ADD(prof_b, prof_s2);
        if (!ok) break;
        tmem_st32(tP, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
        first_half_stored = true;
        softmax_half(r_hi, c, mc, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]), acc);
        tile_sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      } else {
        if (mixed) {
          // masked or out-of-range keys get -inf
#pragma unroll
          for (int cc = 0; cc < 128; ++cc) {
            const uint32_t w = cc < 32 ? kb.x : cc < 64 ? kb.y : cc < 96 ? kb.z : kb.w;
            if (((w >> (cc & 31)) & 1u) == 0) r[cc] = __float_as_uint(-CUDART_INF_F);
          }
        }
        if (i == 0) m_ref = row_max128(r);
        if (mixed) softmax_pass<false>(r, c, m_ref * c, pk, tile_sum);
        else       softmax_pass<true>(r, c, m_ref * c, pk, tile_sum);
        ok = p_buffer_free();
        if (!ok) break;
      }
      SOL_PROF_ADD(prof_c, prof_s3);

      // ---- finalise block i, in block order.  (1) The partner has finalised block i-1: adopt its reference.
      if (i > 0) {
        SOL_PROF_T(prof_s4);
        ok = __all_sync(0xffffffffu, mbar_wait(bar_fin(q, 1 - g), (uint32_t)((i - 1) >> 1) & 1u, limit));
        SOL_PROF_ADD(prof_d, prof_s4);
        if (!ok) break;
        const float r_prev = ref_smem[row];
        const bool moved = r_prev != m_ref;              // it can only have grown
        if (__any_sync(0xffffffffu, moved)) {
          if (moved) { l *= ex2_approx((m_ref - r_prev) * c); m_ref = r_prev; }
          softmax_pass<false>(r, c, m_ref * c, pk, tile_sum);
          if (first_half_stored) tmem_wait_st();                         // the stale first half lands before its replacement
          first_half_stored = false;
        }
      }
      // (2) Lazy reference: the pass ran against the current reference.  All terms are positive, so a row sum
      // <= 2^8 proves every term <= 2^8 and the reference still good.  Otherwise the row maximum is taken; if it
      // grew by more than 2^8 (exp2 domain) the reference moves, l and O are rescaled and the block is redone.
      bool published = i == 0;
      if (__any_sync(0xffffffffu, !(tile_sum <= 256.0f))) {
        const float mx = row_max128(r);
        const bool grow = (mx - m_ref) * c > 8.0f;
        if (__any_sync(0xffffffffu, grow)) {
          if (lane == 0) atomicAdd(p.counters, 1u);                      // rare path: counted for the tests
          const float f = grow ? ex2_approx((m_ref - mx) * c) : 1.0f;
          if (grow) m_ref = mx;
          l *= f;
          // O holds the sum over key blocks 0 .. i-1 once PV(i-1) has completed (PV(i) cannot start before this P).
          // PV(i-3), the previous user of that barrier, completed before the partner stored P(i-1).
          ok = __all_sync(0xffffffffu, mbar_wait(bar_o_done((i - 1) % kPipeBufs), (uint32_t)((i - 1) / kPipeBufs) & 1u, limit));
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int cch = 0; cch < D / 32; ++cch) {
            uint32_t o[32];
            tmem_ld32(tO + cch * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int cc = 0; cc < 32; ++cc) o[cc] = __float_as_uint(__uint_as_float(o[cc]) * f);
            tmem_st32(tO + cch * 32, o);
          }
          softmax_pass<false>(r, c, m_ref * c, pk, tile_sum);
          if (first_half_stored) tmem_wait_st();
          first_half_stored = false;
          published = true;
        }
      }
      // (3) publish the reference this block ended with (only when it changed), then hand P over
      if (published) ref_smem[row] = m_ref;
      l += tile_sum;
      SOL_PROF_T(prof_s5);
      if (!first_half_stored) tmem_st32(tP, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
      tmem_st32(tP + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]));
      tmem_wait_st();
      tc_fence_before();
      // one arrival per warp: on the leader's barrier for P (the MMA over both CTAs' rows starts when all have
      // come), and on this warp's own "finalised" barrier for the partner
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_cluster(mapa_shared(bar_p_full(b), 0)); else mbar_arrive(bar_p_full(b));
        mbar_arrive(bar_fin(q, g));
      }
      SOL_PROF_ADD(prof_e, prof_s5);
    }
#if SOL_PIPE_PROF
    if (warp == 0 && lane == 0) {
      SOL_PROF_OUT(1, prof_wait); SOL_PROF_OUT(2, clock64() - prof_t0); SOL_PROF_OUT(9, 1);
      SOL_PROF_OUT(10, prof_a); SOL_PROF_OUT(11, prof_b); SOL_PROF_OUT(12, prof_c); SOL_PROF_OUT(13, prof_d); SOL_PROF_OUT(14, prof_e);
    }
#endif
    (void)prof_wait; (void)prof_a; (void)prof_b; (void)prof_c; (void)prof_d; (void)prof_e;

    // ---- the two warpgroups' row sums meet: the odd one leaves (sum, reference), the even one does the epilogue
    if (g == 1) { sum_smem[2 * row] = l; sum_smem[2 * row + 1] = m_ref; }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (g == 0) {
      // ---- epilogue: O / l in the output format, staged through shared memory, coalesced 16-byte stores
      if (ok && n_proc > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_o_done((n_proc - 1) % kPipeBufs), (uint32_t)((n_proc - 1) / kPipeBufs) & 1u, limit));
        if (ok) tc_fence_after();
      }
      if (ok && n_proc > 0) {
        // both sums at the reference O ended with: that of the last block's owner
        const float lo = sum_smem[2 * row], mo = sum_smem[2 * row + 1];
        const float m_fin = fmaxf(m_ref, mo);            // references only grow: the later one is the larger one
        float l_tot = l * ex2_approx((m_ref - m_fin) * c);
        if (n_proc > 1) l_tot += lo * ex2_approx((mo - m_fin) * c);
        const float inv = 1.0f / l_tot;
        uint8_t* stage = smem + L::kOffQ + q * 32 * (D * 2);
        if (p.sink.fmt == kOutE4M3) store_rows<D, true>(p, sq, head, q_row0 + q * 32, lane, tO, inv, stage);
        else                        store_rows<D, false>(p, sq, head, q_row0 + q * 32, lane, tO, inv, stage);
      } else if (ok) {
        // no key tile at all (every key of the sequence masked): the row is defined as zero
        const int qrow = q_row0 + row;
        bool store = qrow < sq.n_tokens;
        if (store && p.query_mask != nullptr) store = p.query_mask[sq.tok_start + qrow] != 0;
        if (store) {
          const int row_bytes = p.sink.fmt == kOutE4M3 ? D : D * 2;
          uint8_t* dst = out_row_ptr(p, sq.tok_start + qrow, head, row_bytes / D);
          for (int c16 = 0; c16 < row_bytes / 16; ++c16) *reinterpret_cast<uint4*>(dst + c16 * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    if (!ok && lane == 0) atomicCAS(p.status, 0u, kStatusTimeoutSoftmax);
  } else {
    setmaxnreg_dec<SOL_REGS_OTHER>();
  }
  if (warp == 8) {
    // =========================================================== TMA producer
    if (lane == 0) {
      bool ok = true;
      // Q tiles are read once: first to go from L2, so that they do not push out the head's K / V
      const uint64_t pol_once = l2_policy_evict_first();
      const uint32_t lead_q_full = kPair ? mapa_shared(bar_q_full, 0) : bar_q_full;
      // the leader's barrier counts the bytes of both CTAs' loads
      if (leader) mbar_arrive_expect_tx(bar_q_full, kCtas * L::kTile);
#pragma unroll
      for (int hf = 0; hf < L::kHalves; ++hf) {
        const uint32_t dst = sQ + hf * L::kHalfBytes;
        if (kPair) tma_load_3d_pair_hint(dst, &tm_q, lead_q_full, hf * 64, head, tok0 + q_row0, pol_once);
        else       tma_load_3d_hint(dst, &tm_q, bar_q_full, hf * 64, head, tok0 + q_row0, pol_once);
      }
      uint32_t it = 0, stage = 0, par = 0;
      // one K or V tile (this CTA's half of it, in a pair) into the next ring stage
      long long prof_wait = 0;
      SOL_PROF_T(prof_t0);
      auto load = [&](int jt, bool is_v) {
        SOL_PROF_T(prof_w0);
        const bool free_stage = mbar_wait(bar_kv_empty(stage), par ^ 1u, limit);
        SOL_PROF_ADD(prof_wait, prof_w0);
        if (!free_stage) return false;
        if (leader) mbar_arrive_expect_tx(bar_kv_full(stage), L::kTile);
        const uint32_t dst = sKV + stage * L::kStageBytes;
        if (kPair) {
          // K = this CTA's 64 keys (all head dims, two boxes), V = its 64 head dims (all keys)
          const uint32_t full = mapa_shared(bar_kv_full(stage), 0);
          if (!is_v) {
#pragma unroll
            for (int hf = 0; hf < L::kHalves; ++hf)
              tma_load_3d_pair(dst + hf * L::kKBoxBytes, &tm_k, full, hf * 64, head, tok0 + jt * 128 + (int)rank * 64);
          } else {
            tma_load_3d_pair(dst, &tm_v, full, (int)rank * 64, head, tok0 + jt * 128);
          }
        } else {
          const CUtensorMap* tm = is_v ? &tm_v : &tm_k;
#pragma unroll
          for (int hf = 0; hf < L::kHalves; ++hf)
            tma_load_3d(dst + hf * L::kHalfBytes, tm, bar_kv_full(stage), hf * 64, head, tok0 + jt * 128);
        }
        ++it;
        if (++stage == (uint32_t)L::kStages) { stage = 0; par ^= 1u; }
        return true;
      };
      // in the order the MMA issuer consumes them: K(0), K(1), then K(i+2), V(i)
      const int pre = n_proc < kPipeBufs ? n_proc : kPipeBufs;
      for (int i = 0; i < pre && ok; ++i) ok = load(tile_at(i), false);
      for (int i = 0; i < n_proc && ok; ++i) {
        if (i + kPipeBufs < n_proc) ok = load(tile_at(i + kPipeBufs), false);
        if (ok) ok = load(tile_at(i), true);
      }
#if SOL_PIPE_PROF
      SOL_PROF_OUT(7, prof_wait); SOL_PROF_OUT(8, clock64() - prof_t0);
#endif
      (void)prof_wait;
      if (!ok) {
        atomicCAS(p.status, 0u, kStatusTimeoutProducer);
        // Let the copies already in flight land before the CTA gives its shared memory back.  A single CTA (and the
        // leader of a pair) can see them on its own barriers; the other CTA of a pair reports to the leader's
        // barriers and cannot, but the wait that just ran out lasted `limit`, far longer than any copy takes.
        if (leader) {
          mbar_wait(bar_q_full, 0, limit);
          const uint32_t first = it > (uint32_t)L::kStages ? it - L::kStages : 0u;
          for (uint32_t j = first; j < it; ++j) mbar_wait(bar_kv_full(j % L::kStages), (j / L::kStages) & 1u, limit);
        }
      }
    }
    __syncwarp();
  } else if (warp == 9 && leader) {
    // =========================================================== MMA issuer
    // The whole warp runs this loop (convergent); one elected lane issues each tcgen05 instruction.
    constexpr uint32_t idesc_qk = idesc_bf16_f32(128 * kCtas, 128, false);
    constexpr uint32_t idesc_pv = idesc_bf16_f32(128 * kCtas, D, true);
    bool ok = true;
    const uint32_t v_lbo = p.v_lbo, v_sbo = p.v_sbo;
    // descriptor words: only the low word (address) moves inside the loop
    const uint32_t hi_k = smem_desc_hi_sw128(1024);
    const uint32_t hi_v = smem_desc_hi_sw128(v_sbo);
    const uint32_t q_lo = smem_desc_lo(sQ, 16);
    const uint32_t k_lo_base = smem_desc_lo(sKV, 16);
    const uint32_t v_lo_base = smem_desc_lo(sKV, v_lbo);
    constexpr uint32_t kStageStep = L::kStageBytes >> 4;
    auto commit = [&](uint32_t bar) { if (kPair) tc_commit_elect_pair(bar); else tc_commit_elect(bar); };
    auto wait_full = [&](uint32_t bar, uint32_t parity) { return mbar_wait_warp(bar, parity, limit); };
    auto issue_qk = [&](uint32_t d_tmem, uint32_t stage) {
      const uint32_t k_lo = k_lo_base + stage * kStageStep;
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const uint32_t q_off = ((k >> 2) * L::kHalfBytes + (k & 3) * 32) >> 4;
        const uint32_t k_off = ((k >> 2) * L::kKBoxBytes + (k & 3) * 32) >> 4;
        if (kPair) {
          if (k == 0) mma_ss_elect_pair<false>(d_tmem, q_lo + q_off, k_lo + k_off, hi_k, idesc_qk, 0u);
          else        mma_ss_elect_pair<true>(d_tmem, q_lo + q_off, k_lo + k_off, hi_k, idesc_qk, 1u);
        } else {
          if (k == 0) mma_ss_elect<false>(d_tmem, q_lo + q_off, k_lo + k_off, hi_k, idesc_qk, 0u);
          else        mma_ss_elect<true>(d_tmem, q_lo + q_off, k_lo + k_off, hi_k, idesc_qk, 1u);
        }
      }
    };
    auto issue_pv = [&](uint32_t d_tmem, uint32_t p_tmem, uint32_t stage, bool acc) {
      const uint32_t v_lo = v_lo_base + stage * kStageStep;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (kPair) {
          if (k == 0) mma_ts_elect_pair<false>(d_tmem, p_tmem, v_lo, hi_v, idesc_pv, acc ? 1u : 0u);
          else        mma_ts_elect_pair<true>(d_tmem, p_tmem + k * 8, v_lo + k * (2048 >> 4), hi_v, idesc_pv, 1u);
        } else {
          if (k == 0) mma_ts_elect<false>(d_tmem, p_tmem, v_lo, hi_v, idesc_pv, acc ? 1u : 0u);
          else        mma_ts_elect<true>(d_tmem, p_tmem + k * 8, v_lo + k * (2048 >> 4), hi_v, idesc_pv, 1u);
        }
      }
    };
    // consumer position in the K/V ring
    uint32_t st = 0, ph = 0;
    auto advance = [&]() { if (++st == (uint32_t)L::kStages) { st = 0; ph ^= 1u; } };

    if (n_proc > 0) {
      ok = wait_full(bar_q_full, 0);
      // fill the score pipeline: S(0), S(1)
      const int pre = n_proc < kPipeBufs ? n_proc : kPipeBufs;
      for (int b = 0; b < pre && ok; ++b) {
        if (!wait_full(bar_kv_full(st), ph)) { ok = false; break; }
        tc_fence_after();
        issue_qk(tmem_base + b * 128, st);
        // (test hook: work item 0 withholds this signal so that the waits downstream run into their limit)
        if (!(p.fault_inject == 1u && unit == 0 && b == 1)) commit(bar_s_full(b));
        commit(bar_kv_empty(st));
        advance();
      }
      long long prof_v = 0, prof_p = 0, prof_k = 0;
      SOL_PROF_T(prof_t0);
      for (int i = 0; i < n_proc && ok; ++i) {
        const int b = i & 1;
        const uint32_t use = (uint32_t)(i >> 1);
        if (i + kPipeBufs < n_proc) {
          // S(i+2) goes into S[b] as soon as the softmax has read S(i) out of it
          const uint32_t k_st = st, k_ph = ph;
          advance();
          SOL_PROF_T(prof_w2);
          if (!wait_full(bar_kv_full(k_st), k_ph)) { ok = false; break; }
          if (!wait_full(bar_s_free(b), use & 1u)) { ok = false; break; }
          SOL_PROF_ADD(prof_k, prof_w2);
          tc_fence_after();
          issue_qk(tmem_base + b * 128, k_st);
          commit(bar_s_full(b));
          commit(bar_kv_empty(k_st));
        }
        const uint32_t v_st = st, v_ph = ph;
        advance();
        SOL_PROF_T(prof_w0);
        if (!wait_full(bar_kv_full(v_st), v_ph)) { ok = false; break; }
        SOL_PROF_ADD(prof_v, prof_w0);
        SOL_PROF_T(prof_w1);
        if (!wait_full(bar_p_full(b), use & 1u)) { ok = false; break; }
        SOL_PROF_ADD(prof_p, prof_w1);
        tc_fence_after();
        issue_pv(tO_base, tP_base + b * 64, v_st, i > 0);
        commit(bar_o_done(b));
        commit(bar_kv_empty(v_st));
      }
#if SOL_PIPE_PROF
      if (lane == 0) { SOL_PROF_OUT(3, prof_v); SOL_PROF_OUT(4, prof_p); SOL_PROF_OUT(5, prof_k); SOL_PROF_OUT(6, clock64() - prof_t0); }
#endif
      (void)prof_v; (void)prof_p; (void)prof_k;
    }
    if (!ok) {
      if (lane == 0) atomicCAS(p.status, 0u, kStatusTimeoutMma);
      // tensor-core work already issued must finish before tensor memory is released (in both CTAs of a pair:
      // the other one learns of it at the cluster barrier below)
      commit(bar_drain);
      mbar_wait_warp(bar_drain, 0, limit);
    }
    __syncwarp();
  }

  // ---- teardown: everyone (of both CTAs) is done with tensor memory and shared memory before they are released
  tc_fence_before();
  if (kPair) cluster_sync_all(); else __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    if (kPair) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace sol
