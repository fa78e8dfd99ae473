// Prologue kernels: key-validity bits per 128-key tile, and the 3D rotary embedding of Q and K.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "device_types.cuh"

namespace sol {

// ---------------------------------------------------------------------------------------------
// Key-padding mask + ragged tail -> 128 validity bits per key tile, plus the ascending list of
// tiles that contain at least one valid key (fully masked tiles are skipped by the main kernel).
// One CTA per sequence.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) keybits_kernel(const SeqDev* __restrict__ seqs,
                                                      const uint8_t* __restrict__ key_mask,
                                                      uint32_t* __restrict__ keybits_words,
                                                      int* __restrict__ ktile_list, int* __restrict__ ktile_count) {
  const SeqDev sq = seqs[blockIdx.x];
  const int n_words = sq.n_ktiles * 4;
  for (int idx = threadIdx.x; idx < n_words; idx += blockDim.x) {
    const int key0 = idx * 32;
    uint32_t bits = 0;
#pragma unroll 4
    for (int b = 0; b < 32; ++b) {
      const int key = key0 + b;
      bool valid = key < sq.n_tokens;
      if (valid && key_mask != nullptr) valid = key_mask[sq.tok_start + key] != 0;
      bits |= (valid ? 1u : 0u) << b;
    }
    keybits_words[(size_t)sq.ktile_start * 4 + idx] = bits;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int count = 0;
    for (int base = 0; base < sq.n_ktiles; base += 32) {
      const int tile = base + lane;
      bool nz = false;
      if (tile < sq.n_ktiles) {
        const uint32_t* w = keybits_words + ((size_t)sq.ktile_start + tile) * 4;
        nz = (w[0] | w[1] | w[2] | w[3]) != 0;
      }
      const unsigned ballot = __ballot_sync(0xffffffffu, nz);
      if (nz) ktile_list[sq.ktile_start + count + __popc(ballot & ((1u << lane) - 1u))] = tile;
      count += __popc(ballot);
    }
    if (lane == 0) ktile_count[blockIdx.x] = count;
  }
}

// ---------------------------------------------------------------------------------------------
// 3D rotary embedding of Q and K.  A thread owns one 16-byte chunk (8 head dims = 4 adjacent
// pairs) of a token, fetches the four (cos, sin) once and walks over the heads, so the angle
// lookups are amortised over all heads.  Prefix tokens are copied.  fp32 math, bf16 RNE out.
// Layout in: [token][head][D] with element strides (tok, head); out: contiguous.
// Block: (D/8) x HEADS_PER_PASS threads handle one token per iteration.
// ---------------------------------------------------------------------------------------------
struct RopeArgs {
  const __nv_bfloat16* x[2];
  __nv_bfloat16* y[2];
  long long x_tok_stride[2], x_head_stride[2];
  const SeqDev* seqs;
  int n_seqs;
  long long total_tokens;
  const float2* tables;
  RopeGeom g;
};

__device__ __forceinline__ uint32_t rotate_pair(uint32_t xy, float2 cs) {
  const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(&xy);
  const float xe = __low2float(v), xo = __high2float(v);
  const float re = xe * cs.x - xo * cs.y;
  const float ro = xe * cs.y + xo * cs.x;
  const __nv_bfloat162 r = __floats2bfloat162_rn(re, ro);
  return *reinterpret_cast<const uint32_t*>(&r);
}

__global__ void __launch_bounds__(256) rope_qk_kernel(const RopeArgs a) {
  const int chunks = a.g.head_dim >> 3;          // 16-byte chunks per head row
  const int heads_per_pass = blockDim.x / chunks;
  const int chunk = threadIdx.x % chunks;
  const int hsub = threadIdx.x / chunks;
  const int d1 = a.g.rope[0], d2 = d1 + a.g.rope[1], d3 = d2 + a.g.rope[2];

  for (long long tok = blockIdx.x; tok < a.total_tokens; tok += gridDim.x) {
    // which sequence, which grid position
    int s = 0;
    while (s + 1 < a.n_seqs && !(tok >= a.seqs[s].tok_start && tok < a.seqs[s].tok_start + a.seqs[s].n_tokens)) ++s;
    const SeqDev sq = a.seqs[s];
    const int local = (int)(tok - sq.tok_start);
    float2 cs[4];
    bool rotate = local >= sq.text_len;
    if (rotate) {
      const int p = local - sq.text_len;
      const int hw = sq.H * sq.W;
      const int pos[3] = {p / hw, (p / sq.W) % sq.H, p % sq.W};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int d = chunk * 8 + 2 * u;          // first head dim of the pair
        int axis, j;
        if (d < d1) { axis = 0; j = d >> 1; }
        else if (d < d2) { axis = 1; j = (d - d1) >> 1; }
        else if (d < d3) { axis = 2; j = (d - d2) >> 1; }
        else { axis = -1; j = 0; }
        cs[u] = axis < 0 ? make_float2(1.f, 0.f)
                         : __ldg(&a.tables[a.g.tab_off[axis] + pos[axis] * (a.g.rope[axis] >> 1) + j]);
      }
    }
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      if (a.x[which] == nullptr) continue;
      const __nv_bfloat16* src = a.x[which] + tok * a.x_tok_stride[which] + chunk * 8;
      __nv_bfloat16* dst = a.y[which] + (tok * a.g.heads) * (long long)a.g.head_dim + chunk * 8;
      for (int h = hsub; h < a.g.heads; h += heads_per_pass) {
        uint4 v = __ldg(reinterpret_cast<const uint4*>(src + h * a.x_head_stride[which]));
        if (rotate) {
          v.x = rotate_pair(v.x, cs[0]);
          v.y = rotate_pair(v.y, cs[1]);
          v.z = rotate_pair(v.z, cs[2]);
          v.w = rotate_pair(v.w, cs[3]);
        }
        *reinterpret_cast<uint4*>(dst + (long long)h * a.g.head_dim) = v;
      }
    }
  }
}

}  // namespace sol
