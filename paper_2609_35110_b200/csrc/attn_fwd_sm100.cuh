// Attention main kernel for sm_100a: S = Q~ K~^T and O += P V on tcgen05 tensor cores with the
// accumulators in tensor memory, TMA-fed shared-memory ring, online softmax in registers.
//
// One CTA = one (sequence, head, pair of 128-row query tiles).  With kCtas = 2 two such CTAs on neighbouring SMs
// form a cluster that covers 512 consecutive query rows of one (sequence, head) and shares every K / V tile:
// each CTA loads HALF of the tile (K: 64 of the 128 keys; V: 64 of the 128 head dims) with its own TMA loads and
// one tcgen05.mma.cta_group::2 of M = 256 works on both CTAs' query rows, which halves the shared-memory reads of
// the B operand and the L2 -> SM traffic per flop.  The even CTA (the leader) issues all MMAs; completion goes to
// both CTAs with a multicast commit.  Nothing is loaded with multicast.
// Warp roles (per CTA):
//   warps 0-3   softmax / correction / epilogue of query tile 0 (thread = one query row)
//   warps 4-7   the same for query tile 1
//   warp  8     TMA producer (lane 0)
//   warp  9     tcgen05.mma issuer: the whole warp runs the loop convergently, one elected lane issues each
//               instruction (descriptors then stay in uniform registers); owns the TMEM allocation
//   warps 10-11 idle (complete the third warpgroup)
// The two query tiles ping-pong: while the softmax of one tile runs on the ALUs, the tensor core
// works on the other tile's QK^T / PV.
//
// Tensor memory (512 columns x 128 lanes x 32 bit):
//   [0,128)    S0  (fp32 scores of tile 0);  P0 (bf16, 64 columns) overwrites its first half
//   [128,256)  S1 / P1
//   [256,256+D)       O0 (fp32)
//   [256+D,256+2D)    O1
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "device_types.cuh"
#include "exchange_kernels.cuh"
#include "ptx_sm100.cuh"

namespace sol {

// Register split after launch (384 threads x 168): the softmax warpgroups take what the third
// warpgroup (producer, MMA issuer, two idle warps) gives back: (168 - other) * 128 >= (softmax - 168) * 256.
#ifndef SOL_REGS_SOFTMAX
#define SOL_REGS_SOFTMAX 216
#endif
#ifndef SOL_REGS_OTHER
#define SOL_REGS_OTHER 64
#endif
constexpr int kAttnThreads = 384;   // 8 softmax warps + producer + MMA issuer + 2 idle warps (a full third warpgroup)

__device__ __forceinline__ float row_max128(const uint32_t (&r)[128]) {
  float m0 = max3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
  float m1 = max3(__uint_as_float(r[3]), __uint_as_float(r[4]), __uint_as_float(r[5]));
#pragma unroll
  for (int cc = 6; cc + 3 < 128; cc += 4) {
    m0 = max3(m0, __uint_as_float(r[cc]), __uint_as_float(r[cc + 1]));
    m1 = max3(m1, __uint_as_float(r[cc + 2]), __uint_as_float(r[cc + 3]));
  }
  return max3(m0, m1, fmaxf(__uint_as_float(r[126]), __uint_as_float(r[127])));
}

// One pass over a 128-column score row held in registers: p = 2^(s*c - mc) packed to bf16 and the fp32
// row sum of the un-rounded p.  Every exponential goes to the special-function unit: evaluating a share of them
// with a polynomial on the FMA pipes was measured more than once (scalar and packed fp32x2 arithmetic, 1/8 to 1/2
// of the elements) and lost every time: the polynomial costs 12 to 16 issue cycles per element against 8
// special-function cycles, and the thread-per-row layout has no registers left to interleave enough of them.
__device__ __forceinline__ void softmax_pass(const uint32_t (&r)[128], float c, float mc, uint32_t (&pk)[64],
                                             float& sum) {
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int cc = 0; cc < 64; ++cc) {
    const float p_lo = ex2_approx(fmaf(__uint_as_float(r[2 * cc]), c, -mc));
    const float p_hi = ex2_approx(fmaf(__uint_as_float(r[2 * cc + 1]), c, -mc));
    acc[(2 * cc) & 3] += p_lo;
    acc[(2 * cc + 1) & 3] += p_hi;
    pk[cc] = pack_bf16x2(p_lo, p_hi);
  }
  sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

// Address of output row (flat token, head) in the destination that owns the token.
__device__ __forceinline__ uint8_t* out_row_ptr(const AttnParams& p, long long tok, int head, int elem_bytes) {
  int g = 0;
  while (g + 1 < p.sink.n_dst && tok >= p.sink.tok_begin[g + 1]) ++g;
  return static_cast<uint8_t*>(p.sink.base[g]) +
         ((tok - p.sink.tok_begin[g]) * p.o_tok_stride + (long long)head * p.o_head_stride) * elem_bytes;
}

// Epilogue of one warp: its 32 accumulator rows O * inv -> bf16 (or raw E4M3 bytes) -> staged in the part of
// the query tile's shared memory that belongs to those rows (every MMA that read it has completed; 16-byte
// chunks XOR-swizzled by row) -> written out with one 16-byte chunk per lane, so every store instruction
// covers whole contiguous rows.  Rows beyond the sequence, or not wanted by the query mask, are not stored.
template <int D, bool kFp8>
__device__ __forceinline__ void store_rows(const AttnParams& p, const SeqDev& sq, int head, int first_row, int lane,
                                           uint32_t tO, float inv, uint8_t* stage) {
  constexpr int kRowBytes = kFp8 ? D : D * 2;
  constexpr int kLanesPerRow = kRowBytes / 16;
#pragma unroll
  for (int cch = 0; cch < D / 32; ++cch) {
    uint32_t o[32];
    tmem_ld32(tO + cch * 32, o);
    tmem_wait_ld();
    if (kFp8) {
#pragma unroll
      for (int v4 = 0; v4 < 2; ++v4) {
        uint4 w;
        w.x = pack_e4m3x4(__uint_as_float(o[16 * v4 + 0]) * inv, __uint_as_float(o[16 * v4 + 1]) * inv,
                          __uint_as_float(o[16 * v4 + 2]) * inv, __uint_as_float(o[16 * v4 + 3]) * inv);
        w.y = pack_e4m3x4(__uint_as_float(o[16 * v4 + 4]) * inv, __uint_as_float(o[16 * v4 + 5]) * inv,
                          __uint_as_float(o[16 * v4 + 6]) * inv, __uint_as_float(o[16 * v4 + 7]) * inv);
        w.z = pack_e4m3x4(__uint_as_float(o[16 * v4 + 8]) * inv, __uint_as_float(o[16 * v4 + 9]) * inv,
                          __uint_as_float(o[16 * v4 + 10]) * inv, __uint_as_float(o[16 * v4 + 11]) * inv);
        w.w = pack_e4m3x4(__uint_as_float(o[16 * v4 + 12]) * inv, __uint_as_float(o[16 * v4 + 13]) * inv,
                          __uint_as_float(o[16 * v4 + 14]) * inv, __uint_as_float(o[16 * v4 + 15]) * inv);
        const int ch = cch * 2 + v4;
        *reinterpret_cast<uint4*>(stage + lane * kRowBytes + ((ch ^ (lane & (kLanesPerRow - 1))) << 4)) = w;
      }
    } else {
#pragma unroll
      for (int v4 = 0; v4 < 4; ++v4) {
        uint4 w;
        w.x = pack_bf16x2(__uint_as_float(o[8 * v4 + 0]) * inv, __uint_as_float(o[8 * v4 + 1]) * inv);
        w.y = pack_bf16x2(__uint_as_float(o[8 * v4 + 2]) * inv, __uint_as_float(o[8 * v4 + 3]) * inv);
        w.z = pack_bf16x2(__uint_as_float(o[8 * v4 + 4]) * inv, __uint_as_float(o[8 * v4 + 5]) * inv);
        w.w = pack_bf16x2(__uint_as_float(o[8 * v4 + 6]) * inv, __uint_as_float(o[8 * v4 + 7]) * inv);
        const int ch = cch * 4 + v4;
        *reinterpret_cast<uint4*>(stage + lane * kRowBytes + ((ch ^ (lane & (kLanesPerRow - 1))) << 4)) = w;
      }
    }
  }
  __syncwarp();
  const uint64_t pol_once = l2_policy_evict_first();            // output rows are written once, never read here
  const int ch = lane % kLanesPerRow;
#pragma unroll 4
  for (int r0 = 0; r0 < 32; r0 += 32 / kLanesPerRow) {
    const int rr = r0 + lane / kLanesPerRow;
    const int qrow = first_row + rr;
    bool store = qrow < sq.n_tokens;
    if (store && p.query_mask != nullptr) store = p.query_mask[sq.tok_start + qrow] != 0;
    SOL_DEVICE_CHECK(p.status, !store || (sq.tok_start + qrow >= 0 && sq.tok_start + qrow < p.sink.tok_begin[p.sink.n_dst]),
                     kCheckOutputRow);
    const uint4 w = *reinterpret_cast<const uint4*>(stage + rr * kRowBytes + ((ch ^ (rr & (kLanesPerRow - 1))) << 4));
    if (store) st_global_evict_first(out_row_ptr(p, sq.tok_start + qrow, head, kFp8 ? 1 : 2) + ch * 16, w, pol_once);
  }
}

// Epilogue in the block-INT8 wire format of the exchange (Section 3.2, "Quantized communication"): the thread that owns
// an accumulator row writes that row's record, [D int8 | D/32 scale codes | zeros to a multiple of 16 bytes], straight
// from tensor memory.  A group of 32 values is exactly one 32-column load.  The values are first rounded to bf16 and
// then quantised by the rule of quantize_records_kernel, so the bytes equal those of the bf16 epilogue followed by that
// kernel; what is saved is a write and a read of the bf16 rows.  A record is contiguous (144 bytes at D = 128), so
// every thread writes whole 16-byte chunks of its own record; nothing is staged.
template <int D>
__device__ __forceinline__ void store_rows_int8(const AttnParams& p, const SeqDev& sq, int head, int qrow, uint32_t tO, float inv) {
  constexpr int kGroups = D / 32;
  constexpr int kRecBytes = (D + kGroups + 15) / 16 * 16;
  bool store = qrow < sq.n_tokens;
  if (store && p.query_mask != nullptr) store = p.query_mask[sq.tok_start + qrow] != 0;
  SOL_DEVICE_CHECK(p.status, !store || sq.tok_start + qrow < p.sink.tok_begin[p.sink.n_dst], kCheckOutputRow);
  uint8_t* rec = out_row_ptr(p, sq.tok_start + (store ? qrow : 0), head, 1);
  uint32_t codes = 0;
#pragma unroll
  for (int grp = 0; grp < kGroups; ++grp) {
    uint32_t o[32];
    tmem_ld32(tO + grp * 32, o);                  // warp-collective: every lane loads, whether or not its row is stored
    tmem_wait_ld();
    float f[32];
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      f[e] = __bfloat162float(__float2bfloat16_rn(__uint_as_float(o[e]) * inv));
      amax = fmaxf(amax, fabsf(f[e]));
    }
    const int code = ue5m3_smallest_cover(amax);
    const float rs = __frcp_rn(ue5m3_value(code));
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      w[j] = pack_low_bytes(rint_sat_s8(__fmul_rn(f[4 * j], rs)), rint_sat_s8(__fmul_rn(f[4 * j + 1], rs)),
                            rint_sat_s8(__fmul_rn(f[4 * j + 2], rs)), rint_sat_s8(__fmul_rn(f[4 * j + 3], rs)));
    codes |= (uint32_t)code << (8 * grp);
    if (store) {
      uint4* dst = reinterpret_cast<uint4*>(rec + grp * 32);
      dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
  // tail: the scale codes, then zeros up to the record size (D = 128: one chunk; D = 64: 2 codes + 14 zeros)
  if (store) {
#pragma unroll
    for (int b = D; b < kRecBytes; b += 16)
      *reinterpret_cast<uint4*>(rec + b) = make_uint4(b == D ? codes : 0u, 0u, 0u, 0u);
  }
}

// Half of softmax_pass: 64 columns -> 32 packed pairs, partial sums kept in acc.
__device__ __forceinline__ void softmax_half(const uint32_t (&r)[64], float c, float mc, uint32_t (&pk)[32], float (&acc)[4]) {
#pragma unroll
  for (int cc = 0; cc < 32; ++cc) {
    const float p_lo = ex2_approx(fmaf(__uint_as_float(r[2 * cc]), c, -mc));
    const float p_hi = ex2_approx(fmaf(__uint_as_float(r[2 * cc + 1]), c, -mc));
    acc[(2 * cc) & 3] += p_lo;
    acc[(2 * cc + 1) & 3] += p_hi;
    pk[cc] = pack_bf16x2(p_lo, p_hi);
  }
}

template <int D, int kCtas = 1>
struct AttnSmem {
  static constexpr int kTile = 128 * D * 2;               // bytes of one 128 x D bf16 tile
  static constexpr int kHalves = D / 64;                  // 64-column (128-byte) swizzle boxes per row
  static constexpr int kHalfBytes = 128 * 128;            // one box: 128 rows x 128 bytes
  static constexpr int kStageBytes = kTile / kCtas;       // what one CTA holds of a K or V tile
  static constexpr int kKBoxBytes = kHalfBytes / kCtas;   // one K box: (128 / kCtas) keys x 128 bytes
  static constexpr int kStages = ((D == 128) ? 5 : 10) * (kCtas == 2 ? 8 : 5) / 5;   // K/V ring (K and V tiles alternate)
  static constexpr int kOffQ = 0;
  static constexpr int kOffKV = 2 * kTile;
  static constexpr int kOffBars = kOffKV + kStages * kStageBytes;
  static constexpr int kNumBars = 1 + 2 * kStages + 7;  // q_full, kv_full/empty, s_full[2], p_full[2], o_done[2], drain
  static constexpr int kOffTmemPtr = kOffBars + kNumBars * 8;
  static constexpr int kBytes = kOffTmemPtr + 16;
  static constexpr int kDynBytes = kBytes + 1024;         // slack to align the base to 1024 bytes
};

template <int D, int kCtas>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
  static_assert(kCtas == 1 || (kCtas == 2 && D == 128), "CTA pairs are built for head_dim 128");
  using L = AttnSmem<D, kCtas>;
  constexpr bool kPair = kCtas == 2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t sbase = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (sbase - raw_addr);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // CTA pairs: rank 0 is the leader (issues the MMAs, owns the barriers the other CTA reports to)
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const bool leader = rank == 0;

  const uint32_t sQ = sbase + L::kOffQ;
  const uint32_t sKV = sbase + L::kOffKV;
  const uint32_t bars = sbase + L::kOffBars;
  const uint32_t bar_q_full = bars;
  auto bar_kv_full = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_kv_empty = [&](int s) { return bars + 8u * (1 + L::kStages + s); };
  auto bar_s_full = [&](int t) { return bars + 8u * (1 + 2 * L::kStages + t); };
  auto bar_p_full = [&](int t) { return bars + 8u * (3 + 2 * L::kStages + t); };
  auto bar_o_done = [&](int t) { return bars + 8u * (5 + 2 * L::kStages + t); };
  const uint32_t bar_drain = bars + 8u * (7 + 2 * L::kStages);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + L::kOffTmemPtr);

  // ---- which work item (one per CTA, or one per CTA pair)
  const int unit = (int)blockIdx.x / kCtas + p.cta_offset;
  int si = 0;
  if (kPair) { while (si + 1 < p.n_seqs && unit >= p.seqs[si + 1].quad_work_start) ++si; }
  else       { while (si + 1 < p.n_seqs && unit >= p.seqs[si + 1].work_start) ++si; }
  const SeqDev sq = p.seqs[si];
  const int units_per_head = kPair ? (sq.n_qpairs + 1) / 2 : sq.n_qpairs;
  const int local = unit - (kPair ? sq.quad_work_start : sq.work_start);
  const int head = local / units_per_head;
  const int blk = local - head * units_per_head;        // query pair (256 rows) or query quad (512 rows)
  SOL_DEVICE_CHECK(p.status, si < p.n_seqs && local >= 0 && head < p.heads && blk >= 0 && blk < units_per_head, kCheckWorkItem);
  SOL_DEVICE_CHECK(p.status, !(p.fault_inject == 2u && unit == 0), kCheckInjected);
  // a launch may serve a range of heads only (uniform over the CTA / the pair, before any set-up)
  if (head < p.head_begin || head >= p.head_end) return;
  // rectangular mode: a query block without a wanted row has nothing to do (uniform, before any set-up)
  if (p.pair_needed != nullptr) {
    const uint8_t* need = p.pair_needed + sq.pair_start;
    bool any = need[kCtas * blk] != 0;
    if (kPair && 2 * blk + 1 < sq.n_qpairs) any = any || need[2 * blk + 1] != 0;
    if (!any) return;
  }
  // dense: every CTA of a sequence walks the same list of key tiles; block-sparse (single CTAs only): each CTA has its own
  const bool sparse = !kPair && p.cta_list != nullptr;
  const int n_proc = sparse ? p.cta_count[unit] : p.ktile_count[si];
  const int* __restrict__ ktiles =
      sparse ? p.cta_list + sq.sparse_list_start + (long long)local * sq.n_ktiles : p.ktile_list + sq.ktile_start;
  const uint4* __restrict__ keybits = p.keybits + sq.ktile_start;
  SOL_DEVICE_CHECK(p.status, n_proc >= 0 && n_proc <= sq.n_ktiles, kCheckTileCount);
  // Successive waves of CTAs walk the key tiles in opposite directions (the softmax does not care about the
  // order): a wave then starts on the tiles its predecessor touched last, which are still in L2, instead of
  // on the ones it touched first, which a long sequence has pushed out by then.
  const bool backwards = ((unit / max(1, p.wave_ctas / kCtas)) & 1) != 0;
  const int q_row0 = blk * (256 * kCtas) + (int)rank * 256;   // first local query row of this CTA
  const int tok0 = (int)sq.tok_start;                  // TMA token coordinate of the sequence start
  const unsigned long long limit = p.wait_limit_ns;

  if (warp == 8 && lane == 0) {
    mbar_init(bar_q_full, 1);
    for (int s = 0; s < L::kStages; ++s) {
      mbar_init(bar_kv_full(s), 1);
      mbar_init(bar_kv_empty(s), 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(bar_s_full(t), 1);
      mbar_init(bar_p_full(t), 4 * kCtas);              // one arrival per softmax warp of the tile, from every CTA
      mbar_init(bar_o_done(t), 1);
    }
    mbar_init(bar_drain, 1);
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
  // barriers of the leader that this CTA reports to (its own when it is the leader)
  const uint32_t lead_q_full = kPair ? mapa_shared(bar_q_full, 0) : bar_q_full;

  if (warp < 8) {
    // =========================================================== softmax / correction / epilogue
    setmaxnreg_inc<SOL_REGS_SOFTMAX>();
    const int t = warp >> 2;
    const int wq = warp & 3;
    const int row = wq * 32 + lane;
    const uint32_t lane_off = static_cast<uint32_t>(wq * 32) << 16;
    const uint32_t tS = tmem_base + lane_off + t * 128;
    const uint32_t tO = tmem_base + lane_off + 256 + t * D;
    const uint32_t lead_p_full = kPair ? mapa_shared(bar_p_full(t), 0) : bar_p_full(t);
    const float c = p.scale_log2;
    float m_ref = -CUDART_INF_F;
    float l = 0.f;
    bool ok = true;

    for (int i = 0; i < n_proc; ++i) {
      const int jt = __ldg(&ktiles[backwards ? n_proc - 1 - i : i]);
      SOL_DEVICE_CHECK(p.status, jt >= 0 && jt < sq.n_ktiles, kCheckKeyTile);
      const uint4 kb = __ldg(&keybits[jt]);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full(t), i & 1, limit));
      if (!ok) break;
      tc_fence_after();

      const bool mixed = (kb.x & kb.y & kb.z & kb.w) != 0xffffffffu;
      uint32_t r[128];
      uint32_t pk[64];
      float tile_sum;
      bool first_half_stored = false;
      if (!mixed && i > 0) {
        // Common case, in two halves: the second half of S is still on its way while the first is exponentiated, and
        // the first half of P is on its way to tensor memory while the second is.
        uint32_t (&r_lo)[64] = *reinterpret_cast<uint32_t(*)[64]>(&r[0]);
        uint32_t (&r_hi)[64] = *reinterpret_cast<uint32_t(*)[64]>(&r[64]);
        tmem_ld32(tS, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        tmem_ld32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
        tmem_wait_ld_dep64(r_lo);
        tmem_ld32(tS + 64, *reinterpret_cast<uint32_t(*)[32]>(&r[64]));
        tmem_ld32(tS + 96, *reinterpret_cast<uint32_t(*)[32]>(&r[96]));
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const float mc = m_ref * c;
        softmax_half(r_lo, c, mc, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]), acc);
        tmem_wait_ld_dep64(r_hi);
        tmem_st32(tS, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));       // columns [0,32): their scores are in registers
        first_half_stored = true;
        softmax_half(r_hi, c, mc, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]), acc);
        tile_sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      } else {
#pragma unroll
        for (int cch = 0; cch < 4; ++cch) tmem_ld32(tS + cch * 32, *reinterpret_cast<uint32_t(*)[32]>(&r[cch * 32]));
        tmem_wait_ld();
        if (mixed) {
          // masked or out-of-range keys get -inf
#pragma unroll
          for (int cc = 0; cc < 128; ++cc) {
            const uint32_t w = cc < 32 ? kb.x : cc < 64 ? kb.y : cc < 96 ? kb.z : kb.w;
            if (((w >> (cc & 31)) & 1u) == 0) r[cc] = __float_as_uint(-CUDART_INF_F);
          }
        }
        if (i == 0) m_ref = row_max128(r);
        softmax_pass(r, c, m_ref * c, pk, tile_sum);
      }
      // The pass ran against the current reference maximum, no row maximum taken.
      // All terms are positive, so a row sum <= 2^8 proves that every term is <= 2^8: the reference
      // is still good enough (the result does not depend on which reference is used, only overflow
      // does).  Only when the sum is larger (or not finite) is the row maximum computed; if it has grown
      // by more than 2^8 in the exp2 domain the reference moves, l and O are rescaled and the tile is
      // redone from the scores still held in registers, before any of its P is released.  Rare.
      if (__any_sync(0xffffffffu, !(tile_sum <= 256.0f))) {
        const float mx = row_max128(r);
        const bool grow = (mx - m_ref) * c > 8.0f;
        if (__any_sync(0xffffffffu, grow)) {
          if (lane == 0) atomicAdd(p.counters, 1u);                      // rare path: counted for the tests
          const float f = grow ? ex2_approx((m_ref - mx) * c) : 1.0f;
          if (grow) m_ref = mx;
          l *= f;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_o_done(t), (i - 1) & 1, limit));
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
          softmax_pass(r, c, m_ref * c, pk, tile_sum);
          if (first_half_stored) tmem_wait_st();                         // the stale first half lands before its replacement
          first_half_stored = false;
        }
      }
      l += tile_sum;
      if (!first_half_stored) tmem_st32(tS, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
      tmem_st32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]));
      tmem_wait_st();
      tc_fence_before();
      // one arrival per warp, on the leader's barrier (the MMA over both CTAs' rows starts when all eight have come)
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_cluster(lead_p_full); else mbar_arrive(lead_p_full);
      }
    }

    // ---- epilogue: O / l in the output format, staged through shared memory, coalesced 16-byte stores
    if (ok && n_proc > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(bar_o_done(t), (n_proc - 1) & 1, limit));
      if (ok) tc_fence_after();
    }
    if (ok && n_proc > 0) {
      const float inv = 1.0f / l;
      uint8_t* stage = smem + L::kOffQ + t * L::kTile + wq * 32 * (D * 2);
      if (p.sink.fmt == kOutInt8)      store_rows_int8<D>(p, sq, head, q_row0 + t * 128 + row, tO, inv);
      else if (p.sink.fmt == kOutE4M3) store_rows<D, true>(p, sq, head, q_row0 + t * 128 + wq * 32, lane, tO, inv, stage);
      else                             store_rows<D, false>(p, sq, head, q_row0 + t * 128 + wq * 32, lane, tO, inv, stage);
    } else if (ok) {
      // no key tile at all (every key of the sequence masked): the row is defined as zero
      const int qrow = q_row0 + t * 128 + row;
      bool store = qrow < sq.n_tokens;
      if (store && p.query_mask != nullptr) store = p.query_mask[sq.tok_start + qrow] != 0;
      if (store && p.sink.fmt == kOutInt8) {
        // a record of zeros: every group's scale code is the smallest one (0x01), as the quantiser writes it
        constexpr int kRecBytes = (D + D / 32 + 15) / 16 * 16;
        uint8_t* dst = out_row_ptr(p, sq.tok_start + qrow, head, 1);
        for (int b = 0; b < kRecBytes; b += 16)
          *reinterpret_cast<uint4*>(dst + b) = make_uint4(b == D ? (D == 128 ? 0x01010101u : 0x00000101u) : 0u, 0u, 0u, 0u);
      } else if (store) {
        const int row_bytes = p.sink.fmt == kOutE4M3 ? D : D * 2;
        uint8_t* dst = out_row_ptr(p, sq.tok_start + qrow, head, row_bytes / D);
        for (int c16 = 0; c16 < row_bytes / 16; ++c16) *reinterpret_cast<uint4*>(dst + c16 * 16) = make_uint4(0u, 0u, 0u, 0u);
      }
    } else if (lane == 0) {
      atomicCAS(p.status, 0u, kStatusTimeoutSoftmax);
    }
  } else {
    setmaxnreg_dec<SOL_REGS_OTHER>();
  }
  if (warp == 8) {
    // =========================================================== TMA producer
    if (lane == 0) {
      bool ok = true;
      // Q tiles are read once: first to go from L2, so that they do not push out the head's K / V, which every CTA of the
      // head streams.  K / V of a CTA pair are loaded with an evict-last hint on half of the lines: at the high-resolution
      // size that took the DRAM reads of a launch from 6.9 to 5.6 GB (any share from 0.3 to 1.0 did; evict-first on the rest
      // instead of the default: 38-48 GB).  Single CTAs keep the default: there the hint was measured to raise the reads,
      // because the previous heads' tiles then linger.
      const uint64_t pol_once = l2_policy_evict_first();
      const uint64_t pol_kv = l2_policy_evict_last_half();
      // the leader's barrier counts the bytes of both CTAs' loads
      if (leader) mbar_arrive_expect_tx(bar_q_full, kCtas * 2 * L::kTile);
#pragma unroll
      for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int hf = 0; hf < L::kHalves; ++hf) {
          const uint32_t dst = sQ + t * L::kTile + hf * L::kHalfBytes;
          if (kPair) tma_load_3d_pair_hint(dst, &tm_q, lead_q_full, hf * 64, head, tok0 + q_row0 + t * 128, pol_once);
          else       tma_load_3d_hint(dst, &tm_q, bar_q_full, hf * 64, head, tok0 + q_row0 + t * 128, pol_once);
        }
      uint32_t it = 0, stage = 0, par = 0;
      for (int i = 0; i < n_proc && ok; ++i) {
        const int jt = __ldg(&ktiles[backwards ? n_proc - 1 - i : i]);
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
          if (!mbar_wait(bar_kv_empty(stage), par ^ 1u, limit)) { ok = false; break; }
          if (leader) mbar_arrive_expect_tx(bar_kv_full(stage), L::kTile);
          const uint32_t dst = sKV + stage * L::kStageBytes;
          if (kPair) {
            // this CTA's half of the tile: K = its 64 keys (all head dims, two boxes), V = its 64 head dims (all keys)
            const uint32_t full = mapa_shared(bar_kv_full(stage), 0);
            if (kv == 0) {
#pragma unroll
              for (int hf = 0; hf < L::kHalves; ++hf)
                tma_load_3d_pair_hint(dst + hf * L::kKBoxBytes, &tm_k, full, hf * 64, head, tok0 + jt * 128 + (int)rank * 64, pol_kv);
            } else {
              tma_load_3d_pair_hint(dst, &tm_v, full, (int)rank * 64, head, tok0 + jt * 128, pol_kv);
            }
          } else {
            const CUtensorMap* tm = kv ? &tm_v : &tm_k;
#pragma unroll
            for (int hf = 0; hf < L::kHalves; ++hf)
              tma_load_3d(dst + hf * L::kHalfBytes, tm, bar_kv_full(stage), hf * 64, head, tok0 + jt * 128);
          }
          ++it;
          if (++stage == (uint32_t)L::kStages) { stage = 0; par ^= 1u; }
        }
      }
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
    {
      // The whole warp runs this loop (convergent); one elected lane issues each tcgen05 instruction.
      constexpr uint32_t idesc_qk = idesc_bf16_f32(128 * kCtas, 128, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128 * kCtas, D, true);
      bool ok = true;
      const uint32_t v_lbo = p.v_lbo, v_sbo = p.v_sbo;
      // descriptor words: only the low word (address) moves inside the loop
      const uint32_t hi_k = smem_desc_hi_sw128(1024);
      const uint32_t hi_v = smem_desc_hi_sw128(v_sbo);
      const uint32_t q_lo0 = smem_desc_lo(sQ, 16), q_lo1 = smem_desc_lo(sQ + L::kTile, 16);
      const uint32_t k_lo_base = smem_desc_lo(sKV, 16);
      const uint32_t v_lo_base = smem_desc_lo(sKV, v_lbo);
      constexpr uint32_t kStageStep = L::kStageBytes >> 4;
      const uint32_t tS0 = tmem_base, tS1 = tmem_base + 128;
      const uint32_t tO0 = tmem_base + 256, tO1 = tmem_base + 256 + D;
      auto commit = [&](uint32_t bar) { if (kPair) tc_commit_elect_pair(bar); else tc_commit_elect(bar); };
      auto wait_full = [&](uint32_t bar, uint32_t parity) { return mbar_wait_warp(bar, parity, limit); };
      auto issue_qk = [&](uint32_t d_tmem, uint32_t q_lo, uint32_t stage) {
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
        ok = wait_full(bar_q_full, 0) && wait_full(bar_kv_full(st), ph);
        if (ok) {
          tc_fence_after();
          issue_qk(tS0, q_lo0, st);
          commit(bar_s_full(0));
          issue_qk(tS1, q_lo1, st);
          // (test hook: work item 0 withholds this signal so that the waits downstream run into their limit)
          if (!(p.fault_inject == 1u && unit == 0)) commit(bar_s_full(1));
          commit(bar_kv_empty(st));
          advance();
        }
        for (int i = 0; i < n_proc && ok; ++i) {
          const uint32_t v_st = st, v_ph = ph;
          advance();
          const bool more = i + 1 < n_proc;
          const uint32_t k_st = st, k_ph = ph;
          if (more) advance();
          if (!wait_full(bar_kv_full(v_st), v_ph)) { ok = false; break; }
          if (!wait_full(bar_p_full(0), i & 1)) { ok = false; break; }
          tc_fence_after();
          issue_pv(tO0, tS0, v_st, i > 0);
          commit(bar_o_done(0));
          if (more) {
            if (!wait_full(bar_kv_full(k_st), k_ph)) { ok = false; break; }
            tc_fence_after();
            issue_qk(tS0, q_lo0, k_st);
            commit(bar_s_full(0));
          }
          if (!wait_full(bar_p_full(1), i & 1)) { ok = false; break; }
          tc_fence_after();
          issue_pv(tO1, tS1, v_st, i > 0);
          commit(bar_o_done(1));
          commit(bar_kv_empty(v_st));
          if (more) {
            issue_qk(tS1, q_lo1, k_st);
            commit(bar_s_full(1));
            commit(bar_kv_empty(k_st));
          }
        }
      }
      if (!ok) {
        if (lane == 0) atomicCAS(p.status, 0u, kStatusTimeoutMma);
        // tensor-core work already issued must finish before tensor memory is released (in both CTAs of a pair:
        // the other one learns of it at the cluster barrier below)
        commit(bar_drain);
        mbar_wait_warp(bar_drain, 0, limit);
      }
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
