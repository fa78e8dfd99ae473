// Block-sparse selection (the per-step dynamic sparsity of Section 3.4 of the paper): pooled block
// operands, block-level logits, per-query-block threshold mu + tau * sigma, safety rails, and the
// per-CTA list of key tiles the attention kernel then walks.
//   query block = 256 tokens (one CTA of the attention kernel), KV block = 128 tokens (one key tile).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "device_types.cuh"

namespace sol {

// ---------------------------------------------------------------------------------------------
// Mean of the rotated operand over a block of tokens, per head (fp32).
// x: rotated bf16 [token][head][D] contiguous.  One CTA of 256 threads per (sequence, head, block): D/8 lanes
// cover a token row with 16-byte loads, the other 256 / (D/8) lanes take every 16th (32nd) token; partial sums
// meet in shared memory and are added in a fixed order.
// Output layout: out[head][block][d], or transposed out[head][d][block] (so that the selection kernel
// reads the pooled keys with consecutive threads on consecutive blocks).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pool_blocks_kernel(const __nv_bfloat16* __restrict__ x,
                                                          const SeqDev* __restrict__ seqs, int heads, int head_dim,
                                                          int block_tokens, int seq_index, int n_blocks, int transposed,
                                                          float* __restrict__ out) {
  __shared__ float part[32][129];                  // [token lane][d], padded against bank conflicts
  const SeqDev sq = seqs[seq_index];
  const int blk = blockIdx.x % n_blocks;
  const int head = blockIdx.x / n_blocks;
  const int chunks = head_dim >> 3;
  const int tlanes = blockDim.x / chunks;           // 16 for D = 128, 32 for D = 64
  const int c = threadIdx.x % chunks, tl = threadIdx.x / chunks;
  const int t0 = blk * block_tokens;
  const int t1 = min(sq.n_tokens, t0 + block_tokens);
  const long long row = (long long)heads * head_dim;
  const __nv_bfloat16* src = x + ((sq.tok_start + t0 + tl) * heads + head) * (long long)head_dim + c * 8;
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  for (int t = t0 + tl; t < t1; t += tlanes, src += row * tlanes) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      acc[2 * u] += __uint_as_float(w[u] << 16);
      acc[2 * u + 1] += __uint_as_float(w[u] & 0xffff0000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) part[tl][c * 8 + e] = acc[e];
  __syncthreads();
  for (int d = threadIdx.x; d < head_dim; d += blockDim.x) {
    float sum = 0.f;
    for (int j = 0; j < tlanes; ++j) sum += part[j][d];
    const float mean = sum / (float)(t1 - t0);
    if (transposed) out[((long long)head * head_dim + d) * n_blocks + blk] = mean;
    else            out[((long long)head * n_blocks + blk) * head_dim + d] = mean;
  }
}

// ---------------------------------------------------------------------------------------------
// One CTA per (sequence, head, group of 8 query blocks): block logits of the 8 query blocks against
// every KV block (the pooled keys are read once per group), then one warp per query block: mean and
// standard deviation, threshold, rails, ascending list of selected key tiles.
// Key tiles without any valid key (key-padding mask, see keybits) are never listed.
// qbar: [head][query block][d]; kbar_t: [head][d][KV block].  blockDim = 256 (8 warps).
// ---------------------------------------------------------------------------------------------
constexpr int kSelectRows = 8;

__global__ void __launch_bounds__(256) select_blocks_kernel(const SeqDev* __restrict__ seqs, int seq_index, int heads,
                                                            int head_dim, float tau, const float* __restrict__ qbar,
                                                            const float* __restrict__ kbar_t,
                                                            const uint4* __restrict__ keybits, int* __restrict__ cta_list,
                                                            int* __restrict__ cta_count,
                                                            unsigned long long* __restrict__ stats) {
  extern __shared__ float sm[];                     // [8][head_dim] pooled queries + [8][n_ktiles] scores
  const SeqDev sq = seqs[seq_index];
  const int groups = (sq.n_qpairs + kSelectRows - 1) / kSelectRows;
  const int head = blockIdx.x / groups;
  const int qb0 = (blockIdx.x - head * groups) * kSelectRows;
  const int rows = min(kSelectRows, sq.n_qpairs - qb0);
  const int nk = sq.n_ktiles;
  float* q_s = sm;
  float* sc = sm + kSelectRows * head_dim;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  for (int idx = tid; idx < kSelectRows * head_dim; idx += blockDim.x) {
    const int r = idx / head_dim, d = idx - r * head_dim;
    q_s[idx] = r < rows ? qbar[((long long)head * sq.n_qpairs + qb0 + r) * head_dim + d] : 0.f;
  }
  __syncthreads();
  const float inv_sqrt_d = rsqrtf((float)head_dim);
  const float* kt = kbar_t + (long long)head * head_dim * nk;
  for (int kb = tid; kb < nk; kb += blockDim.x) {
    float acc[kSelectRows];
#pragma unroll
    for (int r = 0; r < kSelectRows; ++r) acc[r] = 0.f;
    for (int d = 0; d < head_dim; ++d) {
      const float kv = __ldg(kt + (long long)d * nk + kb);
#pragma unroll
      for (int r = 0; r < kSelectRows; ++r) acc[r] = fmaf(q_s[r * head_dim + d], kv, acc[r]);
    }
#pragma unroll
    for (int r = 0; r < kSelectRows; ++r) sc[r * nk + kb] = acc[r] * inv_sqrt_d;
  }
  __syncthreads();

  // ---- warp `wid` owns query block qb0 + wid
  if (wid >= rows) return;
  const int qb = qb0 + wid;
  const float* row = sc + wid * nk;
  auto warp_sum = [&](float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
  };
  float part = 0.f;
  for (int kb = lane; kb < nk; kb += 32) part += row[kb];
  const float mu = warp_sum(part) / (float)nk;
  part = 0.f;
  for (int kb = lane; kb < nk; kb += 32) { const float dlt = row[kb] - mu; part = fmaf(dlt, dlt, part); }
  const float sigma = sqrtf(warp_sum(part) / (float)nk);
  const float thr = mu + tau * sigma;
  // arg-max (first one on ties) is always kept
  float best = -CUDART_INF_F;
  int best_i = 0x7fffffff;
  for (int kb = lane; kb < nk; kb += 32)
    if (row[kb] > best) { best = row[kb]; best_i = kb; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
    if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
  }

  const int prefix_kblocks = (sq.text_len + 127) / 128;
  const bool dense_row = qb < (sq.text_len + 255) / 256;
  const uint4* kbits = keybits + sq.ktile_start;
  const long long local = (long long)head * sq.n_qpairs + qb;   // CTA order of the attention kernel
  int* list = cta_list + sq.sparse_list_start + local * nk;
  int count = 0;
  for (int base = 0; base < nk; base += 32) {
    const int kb = base + lane;
    bool on = false;
    if (kb < nk) {
      on = dense_row || kb < prefix_kblocks || kb == best_i || row[kb] > thr;
      const uint4 b = kbits[kb];
      on = on && ((b.x | b.y | b.z | b.w) != 0u);
    }
    const unsigned ballot = __ballot_sync(0xffffffffu, on);
    if (on) list[count + __popc(ballot & ((1u << lane) - 1u))] = kb;
    count += __popc(ballot);
  }
  if (lane == 0) {
    cta_count[sq.work_start + local] = count;
    atomicAdd(stats, (unsigned long long)count);
    atomicAdd(stats + 1, (unsigned long long)nk);
  }
}

}  // namespace sol
