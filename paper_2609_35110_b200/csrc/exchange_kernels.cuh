// Layout kernels of the sequence-parallel exchange around the attention (Section 3.3, "Optimized attention
// collectives"): the stride-aware QKV pack that writes the exchange buffer in one pass, and the inverse head
// merge on the return path.  Both move 16-byte chunks and change no byte.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sol {

constexpr int kMaxRanks = 8;

// Sender's side of the packed QKV exchange.  This rank holds n_local tokens of Q, K and V with all heads,
// read through their own strides (views into a packed QKV buffer are fine).  Destination g receives heads
// [g*hl, (g+1)*hl) of every local token as rows [dst_row0 + t][3][hl][row_bytes]:
//   * dst[g] = slice g of a local send buffer and dst_row0 = 0   -> the send buffer of ONE all-to-all;
//   * dst[g] = rank g's receive buffer mapped into this process and dst_row0 = this rank's first token
//     -> the pack and the transfer are the same pass (plain peer stores).
// In both cases rank g ends up with [total_tokens][3][hl][row_bytes]: Q, K, V of its head shard as strided
// views with a uniform token stride, which the attention plan takes as they are.
struct PackArgs {
  const uint8_t* src[3];
  long long tok_stride_bytes[3], head_stride_bytes[3];
  uint8_t* dst[kMaxRanks];
  long long dst_row0;
  long long n_local;
  int heads, hl, n_ranks;
  int chunks;                 // 16-byte chunks per head row
};

constexpr int kPackUnroll = 4;

__global__ void __launch_bounds__(256) exchange_pack_qkv_kernel(const PackArgs a) {
  // one item = one 16-byte chunk; items ordered (token, which, head, chunk): a warp reads a contiguous
  // stretch of one source row and writes contiguous stretches of hl * row_bytes per destination
  const long long per_tok = 3ll * a.heads * a.chunks;
  const long long items = a.n_local * per_tok;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long base = (long long)blockIdx.x * blockDim.x + threadIdx.x; base < items; base += stride * kPackUnroll) {
    uint4 v[kPackUnroll];
    uint8_t* out[kPackUnroll];
#pragma unroll
    for (int u = 0; u < kPackUnroll; ++u) {
      const long long i = base + u * stride;
      out[u] = nullptr;
      if (i < items) {
        const long long t = i / per_tok;
        int r = (int)(i - t * per_tok);
        const int which = r / (a.heads * a.chunks);
        r -= which * a.heads * a.chunks;
        const int h = r / a.chunks;
        const int c = r - h * a.chunks;
        const int g = h / a.hl;
        v[u] = __ldg(reinterpret_cast<const uint4*>(a.src[which] + t * a.tok_stride_bytes[which] +
                                                    h * a.head_stride_bytes[which] + c * 16));
        out[u] = a.dst[g] + ((((a.dst_row0 + t) * 3 + which) * a.hl + (h - g * a.hl)) * a.chunks + c) * 16;
      }
    }
#pragma unroll
    for (int u = 0; u < kPackUnroll; ++u)
      if (out[u] != nullptr) *reinterpret_cast<uint4*>(out[u]) = v[u];
  }
}

// Receiver's side of the output return: recv[g][t][hl][row_bytes] (what rank g computed for this rank's n
// tokens) -> out[t][g*hl + h][row_bytes], the row-major input of the output projection.  row_bytes is
// whatever one (token, head) record takes on the wire (2*head_dim for bf16, head_dim for raw E4M3).
__global__ void __launch_bounds__(256) exchange_merge_heads_kernel(const uint8_t* __restrict__ recv,
                                                                   uint8_t* __restrict__ out, long long n, int hl,
                                                                   int n_ranks, int chunks,
                                                                   long long out_tok_stride_bytes) {
  const long long per_tok = (long long)n_ranks * hl * chunks;
  const long long items = n * per_tok;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long base = (long long)blockIdx.x * blockDim.x + threadIdx.x; base < items; base += stride * kPackUnroll) {
    uint4 v[kPackUnroll];
    uint8_t* dst[kPackUnroll];
#pragma unroll
    for (int u = 0; u < kPackUnroll; ++u) {
      const long long i = base + u * stride;
      dst[u] = nullptr;
      if (i < items) {
        const long long t = i / per_tok;
        int r = (int)(i - t * per_tok);
        const int g = r / (hl * chunks);
        r -= g * hl * chunks;                                   // (local head, chunk) within the shard
        v[u] = __ldg(reinterpret_cast<const uint4*>(recv + (((long long)g * n + t) * hl * chunks + r) * 16));
        dst[u] = out + t * out_tok_stride_bytes + ((long long)g * hl * chunks + r) * 16;
      }
    }
#pragma unroll
    for (int u = 0; u < kPackUnroll; ++u)
      if (dst[u] != nullptr) *reinterpret_cast<uint4*>(dst[u]) = v[u];
  }
}

// ---------------------------------------------------------------------------------------------
// Block-INT8 wire formats (Section 3.3, "Quantized communication").  One (token, head) record:
//   QKV:    [q int8 x D | k int8 x D | v int8 x D | D/32 q scale codes | D/32 k codes | D/32 v codes | zeros]
//           padded to a multiple of 16 bytes (D = 128: 384 + 12 + 4 = 400 bytes);
//   output: [o int8 x D | D/32 scale codes | zeros] padded likewise (D = 128: 128 + 4 + 12 = 144 bytes).
// A scale code is an unsigned 8-bit float with 5 exponent bits (bias 15) and 3 mantissa bits, one per group of
// 32 values; only finite positive codes 0x01..0xf7 are written.  The scale of a group is the smallest such value
// s with 127 * s >= max|x| (127 * s is exact in fp32, so the choice is exact); q = clamp(rint(x * (1/s)), +-127)
// with reciprocal and product each rounded to fp32.  Every padding byte is written.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float ue5m3_value(int c) {
  const int e = c >> 3, m = c & 7;
  return e == 0 ? (float)m * 7.62939453125e-06f : (float)(8 + m) * __int_as_float((e - 18 + 127) << 23);
}

__device__ __forceinline__ int ue5m3_smallest_cover(float amax) {
  // candidate from the bits of amax / 127 (approximate), then one exact correction step either way
  const float y = amax * (1.0f / 127.0f);
  int c;
  if (!(y >= 6.103515625e-05f)) {
    c = (int)ceilf(y * 131072.0f);                              // subnormal ladder: multiples of 2^-17
  } else {
    const uint32_t b = __float_as_uint(y);
    c = ((int)(b >> 23) - 127 + 15) * 8 + (int)(((b & 0x7fffffu) + 0xfffffu) >> 20);
  }
  c = min(max(c, 1), 0xf7);
  if (c > 1 && 127.0f * ue5m3_value(c - 1) >= amax) --c;
  if (c < 0xf7 && 127.0f * ue5m3_value(c) < amax) ++c;
  return c;
}

struct QuantArgs {
  const uint8_t* src[3];                // bf16 rows, read through strides
  long long tok_stride_bytes[3], head_stride_bytes[3];
  uint8_t* dst[kMaxRanks];              // records: dst[g][dst_row0 + t][hl][rec_bytes]
  long long dst_row0;
  long long n_rows;
  int heads, hl, n_ranks;
  int head_dim, rec_bytes;
};

// NW = 3: the quantising QKV pack (sender's side of the exchange); NW = 1: output rows -> output records.
// One thread per 8 values; the 4 threads of a 32-value group sit in adjacent lanes.  A block of
// (threads per record) x (at most 16 records) threads handles that many records per iteration; their scale
// codes meet in shared memory and leave as one 16-byte tail each (both record kinds end in exactly 16 bytes
// of codes + zeros for head_dim 64 and 128).
template <int NW>
__global__ void __launch_bounds__(256) quantize_records_kernel(const QuantArgs a) {
  const int chunks = a.head_dim >> 3;
  const int per_rec = NW * chunks;                              // threads per record
  const int recs = blockDim.x / per_rec;                        // records per block iteration
  const int ng = a.head_dim >> 5;                               // groups (= scale codes) per tensor
  __shared__ __align__(16) uint8_t tails[16][16];
  const int r_in = threadIdx.x / per_rec;
  const int rem = threadIdx.x - r_in * per_rec;
  const int which = rem / chunks;
  const int c = rem - which * chunks;
  const long long n_recs = a.n_rows * a.heads;
  for (long long rec0 = (long long)blockIdx.x * recs; rec0 < n_recs; rec0 += (long long)gridDim.x * recs) {
    const long long rec = rec0 + r_in;
    const bool valid = r_in < recs && rec < n_recs;
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = 0.f;
    long long t = 0;
    int h = 0;
    if (valid) {
      t = rec / a.heads;
      h = (int)(rec - t * a.heads);
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.src[which] + t * a.tok_stride_bytes[which] +
                                                          h * a.head_stride_bytes[which] + c * 16));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const __nv_bfloat162 b2 = *reinterpret_cast<const __nv_bfloat162*>(&w[u]);
        f[2 * u] = __low2float(b2);
        f[2 * u + 1] = __high2float(b2);
      }
    }
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(f[e]));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    const int code = ue5m3_smallest_cover(amax);
    const float inv = __frcp_rn(ue5m3_value(code));
    uint32_t packed[2] = {0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      int q = __float2int_rn(__fmul_rn(f[e], inv));
      q = min(max(q, -127), 127);
      packed[e >> 2] |= (uint32_t)(q & 0xff) << (8 * (e & 3));
    }
    uint8_t* out = nullptr;
    if (valid) {
      const int g = h / a.hl;
      out = a.dst[g] + ((a.dst_row0 + t) * a.hl + (h - g * a.hl)) * a.rec_bytes;
      *reinterpret_cast<uint2*>(out + which * a.head_dim + c * 8) = make_uint2(packed[0], packed[1]);
    }
    // zero the tail first (codes overwrite their slots after the barrier)
    if (r_in < recs)
      for (int b = rem; b < 16; b += per_rec) tails[r_in][b] = 0;
    __syncthreads();
    if (r_in < recs && (c & 3) == 0) tails[r_in][which * ng + (c >> 2)] = (uint8_t)code;
    __syncthreads();
    if (valid && rem == 0) *reinterpret_cast<uint4*>(out + NW * a.head_dim) = *reinterpret_cast<const uint4*>(tails[r_in]);
    __syncthreads();
  }
}

// Receiver's side: records [rows][heads][rec_bytes] -> bf16 [rows][NW][heads][D] (NW = 3: the packed QKV tensor
// the attention reads through strides; NW = 1: output rows).  value = q * s, exact in fp32, one rounding to bf16.
template <int NW>
__global__ void __launch_bounds__(256) dequantize_records_kernel(const uint8_t* __restrict__ recs,
                                                                 __nv_bfloat16* __restrict__ out, long long n_rows,
                                                                 int heads, int head_dim, int rec_bytes) {
  const int chunks = head_dim >> 3;
  const long long per_row = (long long)heads * NW * chunks;
  const long long items = n_rows * per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / per_row;
    int r = (int)(i - t * per_row);
    const int h = r / (NW * chunks);
    r -= h * NW * chunks;
    const int which = r / chunks;
    const int c = r - which * chunks;
    const uint8_t* rec = recs + (t * heads + h) * rec_bytes;
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(rec + which * head_dim + c * 8));
    const float s = ue5m3_value(__ldg(rec + NW * head_dim + which * (head_dim >> 5) + (c >> 2)));
    const uint32_t w[2] = {v.x, v.y};
    uint32_t o[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int q0 = (int)(int8_t)((w[u >> 1] >> (16 * (u & 1))) & 0xff);
      const int q1 = (int)(int8_t)((w[u >> 1] >> (16 * (u & 1) + 8)) & 0xff);
      const __nv_bfloat162 b2 = __floats2bfloat162_rn((float)q0 * s, (float)q1 * s);
      o[u] = *reinterpret_cast<const uint32_t*>(&b2);
    }
    *reinterpret_cast<uint4*>(out + (((t * NW + which) * heads + h) * (long long)head_dim + c * 8)) =
        make_uint4(o[0], o[1], o[2], o[3]);
  }
}

}  // namespace sol
