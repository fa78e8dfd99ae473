// Prologue kernels: key-validity bits per 128-key tile, and the 3D rotary embedding of Q and K.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "device_types.cuh"
#include "exchange_kernels.cuh"

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
// Rectangular attention (fewer queries than keys): which 256-row query pairs hold at least one wanted
// query row.  One warp per (sequence, pair); grid = total pairs.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) pair_needed_kernel(const SeqDev* __restrict__ seqs, int n_seqs,
                                                         const uint8_t* __restrict__ query_mask,
                                                         uint8_t* __restrict__ pair_needed) {
  int s = 0;
  while (s + 1 < n_seqs && !((int)blockIdx.x >= seqs[s].pair_start && (int)blockIdx.x < seqs[s].pair_start + seqs[s].n_qpairs)) ++s;
  const SeqDev sq = seqs[s];
  const int pair = (int)blockIdx.x - sq.pair_start;
  bool any = false;
  for (int r = threadIdx.x; r < 256; r += 32) {
    const int row = pair * 256 + r;
    if (row < sq.n_tokens && query_mask[sq.tok_start + row] != 0) any = true;
  }
  any = __any_sync(0xffffffffu, any);
  if (threadIdx.x == 0) pair_needed[blockIdx.x] = any ? 1 : 0;
}

// ---------------------------------------------------------------------------------------------
// Producer of the attention operands: optional QK RMS-norm (over head_dim, learned gain) followed by
// the 3D rotary embedding of Q and K -- the paper's fusion group (2), "QK normalization with partial
// RoPE" (Section 3.5) -- written once as bf16.  A thread owns one 16-byte chunk (8 head dims = 4
// adjacent pairs) of a token, fetches the four (cos, sin) once and walks over the heads, so the angle
// lookups are amortised over all heads.  The chunks of one (token, head) row sit in adjacent lanes; the
// sum of squares is a shuffle reduction over them.  fp32 math throughout, one rounding to bf16 at the
// end.  Prefix tokens are normalised but not rotated.
// Layout in: [token][head][D] with element strides (tok, head); out: contiguous.
// Block: (D/8) x HEADS_PER_PASS threads handle one token per iteration; the host picks HEADS_PER_PASS as a divisor of
// the number of heads where it can, so that every thread has the same number of rows.
// ---------------------------------------------------------------------------------------------
struct RopeArgs {
  const __nv_bfloat16* x[2];
  __nv_bfloat16* y[2];
  long long x_tok_stride[2], x_head_stride[2];
  const float* gain[2];       // [head_dim] each, or nullptr: no normalisation for that tensor
  float eps;
  const SeqDev* seqs;
  int n_seqs;
  long long total_tokens;
  const float2* tables;
  RopeGeom g;
  int head_begin, head_end;   // heads [head_begin, head_end) are produced by this launch
  unsigned int* status;       // status word (written by the index checks of the debug build only)
};

template <bool kNorm>
__global__ void __launch_bounds__(256, 3) rope_qk_kernel(const RopeArgs a) {
  const int chunks = a.g.head_dim >> 3;          // 16-byte chunks per head row (8 or 16: divides the warp)
  const int heads_per_pass = blockDim.x / chunks;
  const int chunk = threadIdx.x % chunks;
  const int hsub = threadIdx.x / chunks;
  const int d1 = a.g.rope[0], d2 = d1 + a.g.rope[1], d3 = d2 + a.g.rope[2];
  const float inv_d = 1.0f / (float)a.g.head_dim;
  const unsigned warp_lanes = __activemask();    // the block's last warp may be partial; nothing diverges after this point
  // which table entry each of the thread's four pairs uses (fixed per thread: it depends on the chunk only)
  int axis[4], tab[4], step[4];                 // step: table entries per position of that axis
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int d = chunk * 8 + 2 * u;             // first head dim of the pair
    if (d < d1)      { axis[u] = 0; tab[u] = a.g.tab_off[0] + (d >> 1);        step[u] = a.g.rope[0] >> 1; }
    else if (d < d2) { axis[u] = 1; tab[u] = a.g.tab_off[1] + ((d - d1) >> 1); step[u] = a.g.rope[1] >> 1; }
    else if (d < d3) { axis[u] = 2; tab[u] = a.g.tab_off[2] + ((d - d2) >> 1); step[u] = a.g.rope[2] >> 1; }
    else             { axis[u] = -1; tab[u] = 0; step[u] = 0; }
  }

  for (long long tok = blockIdx.x; tok < a.total_tokens; tok += gridDim.x) {
    // which sequence, which grid position
    int s = 0;
    while (s + 1 < a.n_seqs && !(tok >= a.seqs[s].tok_start && tok < a.seqs[s].tok_start + a.seqs[s].n_tokens)) ++s;
    const SeqDev sq = a.seqs[s];
    const int local = (int)(tok - sq.tok_start);
    SOL_DEVICE_CHECK(a.status, local >= 0 && local < sq.n_tokens, kCheckTokenSequence);
    const bool rotate = local >= sq.text_len;
    // heads in groups of kBatch per thread and tensor: the loads of Q AND K of a group are all issued before any is
    // used, and the table lookups travel with them
    constexpr int kBatch = 4;
    for (int hb = a.head_begin; hb < a.head_end; hb += kBatch * heads_per_pass) {    // the same trip count for every thread
      const int h0 = hb + hsub;
      uint4 v[2][kBatch];
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        if (a.x[which] == nullptr) continue;
        const __nv_bfloat16* src = a.x[which] + tok * a.x_tok_stride[which] + chunk * 8;
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int h = h0 + b * heads_per_pass;
          if (kNorm)                v[which][b] = __ldg(reinterpret_cast<const uint4*>(src + min(h, a.head_end - 1) * a.x_head_stride[which]));
          else if (h < a.head_end)  v[which][b] = __ldg(reinterpret_cast<const uint4*>(src + h * a.x_head_stride[which]));
        }
      }
      float2 cs[4];
      if (rotate) {
        const int p = local - sq.text_len;
        const int hw = sq.H * sq.W;
        const int pt = p / hw, ph = (p / sq.W) % sq.H, pw = p % sq.W;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int pos = axis[u] == 0 ? pt : axis[u] == 1 ? ph : pw;
          cs[u] = axis[u] < 0 ? make_float2(1.f, 0.f) : __ldg(&a.tables[tab[u] + pos * step[u]]);
        }
      }
      // Normalising instantiation: the sums of squares of all rows of the group first, then their shuffle reductions
      // step by step across the rows (six independent chains instead of six dependent ones one after another), then
      // the reciprocal roots.  Rows past the head range were loaded from a clamped head and are not stored.
      float rinv[2][kBatch];
      if (kNorm) {
        float ss[2][kBatch];
#pragma unroll
        for (int which = 0; which < 2; ++which)
#pragma unroll
          for (int b = 0; b < kBatch; ++b) {
            const uint32_t w[4] = {v[which][b].x, v[which][b].y, v[which][b].z, v[which][b].w};
            float acc = 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const float lo = __uint_as_float(w[u] << 16), hi = __uint_as_float(w[u] & 0xffff0000u);
              acc = fmaf(lo, lo, acc);
              acc = fmaf(hi, hi, acc);
            }
            ss[which][b] = acc;
          }
        for (int off = chunks >> 1; off > 0; off >>= 1) {
#pragma unroll
          for (int which = 0; which < 2; ++which)
#pragma unroll
            for (int b = 0; b < kBatch; ++b) ss[which][b] += __shfl_xor_sync(warp_lanes, ss[which][b], off);
        }
#pragma unroll
        for (int which = 0; which < 2; ++which)
#pragma unroll
          for (int b = 0; b < kBatch; ++b) rinv[which][b] = rsqrtf(ss[which][b] * inv_d + a.eps);
      }
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        if (a.x[which] == nullptr) continue;
        const bool norm = kNorm && a.gain[which] != nullptr;
        __nv_bfloat16* dst = a.y[which] + (tok * a.g.heads) * (long long)a.g.head_dim + chunk * 8;
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int h = h0 + b * heads_per_pass;
          if (!kNorm && h >= a.head_end) break;
          const uint32_t w[4] = {v[which][b].x, v[which][b].y, v[which][b].z, v[which][b].w};
          float f[8];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            f[2 * u] = __uint_as_float(w[u] << 16);
            f[2 * u + 1] = __uint_as_float(w[u] & 0xffff0000u);
          }
          if (norm) {
            // the gains of this thread's eight head dims: 32 bytes that stay in L1
            const float4 g0 = __ldg(reinterpret_cast<const float4*>(a.gain[which] + chunk * 8));
            const float4 g1 = __ldg(reinterpret_cast<const float4*>(a.gain[which] + chunk * 8) + 1);
            const float r = rinv[which][b];
            f[0] *= r * g0.x; f[1] *= r * g0.y; f[2] *= r * g0.z; f[3] *= r * g0.w;
            f[4] *= r * g1.x; f[5] *= r * g1.y; f[6] *= r * g1.z; f[7] *= r * g1.w;
          }
          uint32_t o[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            float re = f[2 * u], ro = f[2 * u + 1];
            if (rotate) {
              re = f[2 * u] * cs[u].x - f[2 * u + 1] * cs[u].y;
              ro = f[2 * u] * cs[u].y + f[2 * u + 1] * cs[u].x;
            }
            const __nv_bfloat162 r2 = __floats2bfloat162_rn(re, ro);
            o[u] = *reinterpret_cast<const uint32_t*>(&r2);
          }
          if (h < a.head_end) *reinterpret_cast<uint4*>(dst + (long long)h * a.g.head_dim) = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The same producer fed by the block-INT8 QKV records of the exchange (Section 3.2, "Quantized communication"; the
// fusion of the receiver's dequantisation into the consumer is what Section 3.3, "Joint optimization with quantized
// communication" asks for): records [token][head][q int8 x D | k | v | 3 D/32 scale codes | pad] -> rotated Q~, K~
// and plain V, all bf16 [token][head][D].  value = q * s is rounded to bf16 first and rotated then, so Q~ and K~ are
// bit for bit what dequantize_records_kernel followed by rope_qk_kernel produce; the packed bf16 QKV tensor in
// between (a write and a read of the whole shard) is never made.  Thread mapping as in rope_qk_kernel: a thread owns
// 8 head dims of a token (8 record bytes in, 16 bytes out), fetches its four (cos, sin) once per token and walks
// over the heads.
// ---------------------------------------------------------------------------------------------
struct RopeRecordArgs {
  const uint8_t* records;     // [total_tokens][heads][rec_bytes]
  __nv_bfloat16* y[3];        // Q~, K~, V outputs, contiguous [token][head][D]
  int rec_bytes;
  const SeqDev* seqs;
  int n_seqs;
  long long total_tokens;
  const float2* tables;
  RopeGeom g;
  unsigned int* status;
};

// Thread = 16 head dims of one (token, head) record: one 16-byte load per tensor, two 16-byte stores per tensor.  A block
// is (head_dim / 16) x heads_per_pass x tokens_per_block threads; every thread takes its heads two at a time, the six
// loads of the pair in flight together.
__global__ void __launch_bounds__(256, 2) rope_records_kernel(const RopeRecordArgs a, int heads_per_pass) {
  const int D = a.g.head_dim;
  const int lanes = D >> 4;                       // threads per record
  const int part = threadIdx.x % lanes;           // which 16 head dims
  const int hsub = (threadIdx.x / lanes) % heads_per_pass;
  const int tsub = threadIdx.x / (lanes * heads_per_pass);
  const int toks_per_block = blockDim.x / (lanes * heads_per_pass);
  const int d1 = a.g.rope[0], d2 = d1 + a.g.rope[1], d3 = d2 + a.g.rope[2];
  int axis[8], tab[8], step[8];                   // per pair of this thread: which position, which table entries
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int d = part * 16 + 2 * u;
    if (d < d1)      { axis[u] = 0; tab[u] = a.g.tab_off[0] + (d >> 1);        step[u] = a.g.rope[0] >> 1; }
    else if (d < d2) { axis[u] = 1; tab[u] = a.g.tab_off[1] + ((d - d1) >> 1); step[u] = a.g.rope[1] >> 1; }
    else if (d < d3) { axis[u] = 2; tab[u] = a.g.tab_off[2] + ((d - d2) >> 1); step[u] = a.g.rope[2] >> 1; }
    else             { axis[u] = -1; tab[u] = 0; step[u] = 0; }
  }
  const int n_codes = D >> 5;
  const int code_idx = part >> 1;                 // this thread's group of 32 inside a tensor

  for (long long tok = (long long)blockIdx.x * toks_per_block + tsub; tok < a.total_tokens;
       tok += (long long)gridDim.x * toks_per_block) {
    int s = 0;
    while (s + 1 < a.n_seqs && !(tok >= a.seqs[s].tok_start && tok < a.seqs[s].tok_start + a.seqs[s].n_tokens)) ++s;
    const SeqDev sq = a.seqs[s];
    const int local = (int)(tok - sq.tok_start);
    SOL_DEVICE_CHECK(a.status, local >= 0 && local < sq.n_tokens, kCheckTokenSequence);
    const bool rotate = local >= sq.text_len;
    float2 cs[8];
    if (rotate) {
      const int p = local - sq.text_len;
      const int hw = sq.H * sq.W;
      const int pt = p / hw, ph = (p / sq.W) % sq.H, pw = p % sq.W;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int pos = axis[u] == 0 ? pt : axis[u] == 1 ? ph : pw;
        cs[u] = axis[u] < 0 ? make_float2(1.f, 0.f) : __ldg(&a.tables[tab[u] + pos * step[u]]);
      }
    }
    for (int h0 = hsub; h0 < a.g.heads; h0 += 2 * heads_per_pass) {
      uint4 v[2][3];
      float sc[2][3];
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        const int h = h0 + b * heads_per_pass;
        if (h >= a.g.heads) break;
        const uint8_t* rec = a.records + (tok * a.g.heads + h) * (long long)a.rec_bytes;
#pragma unroll
        for (int which = 0; which < 3; ++which) {
          v[b][which] = __ldg(reinterpret_cast<const uint4*>(rec + which * D + part * 16));
          sc[b][which] = ue5m3_value(__ldg(rec + 3 * D + which * n_codes + code_idx));
        }
      }
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        const int h = h0 + b * heads_per_pass;
        if (h >= a.g.heads) break;
        const long long row = (tok * a.g.heads + h) * (long long)D + part * 16;
#pragma unroll
        for (int which = 0; which < 3; ++which) {
          uint32_t o[8];
          dequant16(v[b][which], sc[b][which], o);            // the values the bf16 wire tensor would hold
          if (which < 2 && rotate) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float f0 = __uint_as_float(o[u] << 16), f1 = __uint_as_float(o[u] & 0xffff0000u);
              const __nv_bfloat162 r2 = __floats2bfloat162_rn(f0 * cs[u].x - f1 * cs[u].y, f0 * cs[u].y + f1 * cs[u].x);
              o[u] = *reinterpret_cast<const uint32_t*>(&r2);
            }
          }
          uint4* dst = reinterpret_cast<uint4*>(a.y[which] + row);
          dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
          dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
      }
    }
  }
}

}  // namespace sol
