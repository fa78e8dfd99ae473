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
// Mean of the rotated operand over a block of tokens, per head: out[head][block][d] (fp32).
// x: rotated bf16 [token][head][D] contiguous.  One CTA per (sequence, head, block); thread d sums
// column d over the block's tokens in order.  blockDim = D.
// ---------------------------------------------------------------------------------------------
__global__ void pool_blocks_kernel(const __nv_bfloat16* __restrict__ x, const SeqDev* __restrict__ seqs, int heads,
                                   int head_dim, int block_tokens, int seq_index, int n_blocks, float* __restrict__ out) {
  const SeqDev sq = seqs[seq_index];
  const int blk = blockIdx.x % n_blocks;
  const int head = blockIdx.x / n_blocks;
  const int d = threadIdx.x;
  const int t0 = blk * block_tokens;
  const int t1 = min(sq.n_tokens, t0 + block_tokens);
  const __nv_bfloat16* src = x + ((sq.tok_start + t0) * heads + head) * (long long)head_dim + d;
  float acc = 0.f;
  for (int t = t0; t < t1; ++t, src += (long long)heads * head_dim) acc += __bfloat162float(*src);
  out[((long long)head * n_blocks + blk) * head_dim + d] = acc / (float)(t1 - t0);
}

// ---------------------------------------------------------------------------------------------
// One CTA per attention work item (sequence, head, query block): block logits against every KV
// block, mean and standard deviation, threshold, rails, ascending list of selected key tiles.
// Key tiles without any valid key (key-padding mask, see keybits) are never listed.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) select_blocks_kernel(const SeqDev* __restrict__ seqs, int seq_index, int heads,
                                                            int head_dim, float tau, const float* __restrict__ qbar,
                                                            const float* __restrict__ kbar,
                                                            const uint4* __restrict__ keybits, int* __restrict__ cta_list,
                                                            int* __restrict__ cta_count,
                                                            unsigned long long* __restrict__ stats) {
  extern __shared__ float sm[];                     // [head_dim] pooled query + [n_ktiles] scores + reduction scratch
  const SeqDev sq = seqs[seq_index];
  const int local = blockIdx.x;                     // head-major, query block fastest (= CTA order of the attention kernel)
  const int head = local / sq.n_qpairs;
  const int qb = local - head * sq.n_qpairs;
  const int nk = sq.n_ktiles;
  float* q_s = sm;
  float* sc = sm + head_dim;
  float* red = sc + nk;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  for (int d = tid; d < head_dim; d += blockDim.x) q_s[d] = qbar[((long long)head * sq.n_qpairs + qb) * head_dim + d];
  __syncthreads();
  const float inv_sqrt_d = rsqrtf((float)head_dim);
  for (int kb = tid; kb < nk; kb += blockDim.x) {
    const float* kr = kbar + ((long long)head * nk + kb) * head_dim;
    float acc = 0.f;
    for (int d = 0; d < head_dim; ++d) acc = fmaf(q_s[d], __ldg(kr + d), acc);
    sc[kb] = acc * inv_sqrt_d;
  }
  __syncthreads();

  auto block_sum = [&](float v) -> float {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red[wid] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    __syncthreads();
    return t;
  };
  float part = 0.f;
  for (int kb = tid; kb < nk; kb += blockDim.x) part += sc[kb];
  const float mu = block_sum(part) / (float)nk;
  part = 0.f;
  for (int kb = tid; kb < nk; kb += blockDim.x) { const float dlt = sc[kb] - mu; part = fmaf(dlt, dlt, part); }
  const float sigma = sqrtf(block_sum(part) / (float)nk);
  const float thr = mu + tau * sigma;
  // arg-max (first one on ties) is always kept
  float best = -CUDART_INF_F;
  int best_i = 0x7fffffff;
  for (int kb = tid; kb < nk; kb += blockDim.x)
    if (sc[kb] > best) { best = sc[kb]; best_i = kb; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
    if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
  }
  float* red_v = red;
  int* red_i = reinterpret_cast<int*>(red + 8);
  if (lane == 0) { red_v[wid] = best; red_i[wid] = best_i; }
  __syncthreads();
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w)
    if (red_v[w] > best || (red_v[w] == best && red_i[w] < best_i)) { best = red_v[w]; best_i = red_i[w]; }
  __syncthreads();

  const int prefix_kblocks = (sq.text_len + 127) / 128;
  const bool dense_row = qb < (sq.text_len + 255) / 256;
  const uint4* kbits = keybits + sq.ktile_start;
  int* list = cta_list + sq.sparse_list_start + (long long)local * nk;
  if (wid == 0) {
    int count = 0;
    for (int base = 0; base < nk; base += 32) {
      const int kb = base + lane;
      bool on = false;
      if (kb < nk) {
        on = dense_row || kb < prefix_kblocks || kb == best_i || sc[kb] > thr;
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
}

}  // namespace sol
