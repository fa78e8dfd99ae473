// Layout kernels of the sequence-parallel exchange around the attention (Section 3.2, "Optimized attention
// collectives"): the stride-aware QKV pack that writes the exchange buffer in one pass, and the inverse head
// merge on the return path.  Both move 16-byte chunks and change no byte.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sol {

constexpr int kMaxRanks = 8;

// x = q * d + r.  Index spaces here almost always fit 32 bits, where the division is several times cheaper;
// `small` (uniform across the grid) says so.
__device__ __forceinline__ void divmod(long long x, int d, bool small, long long& q, int& r) {
  if (small) {
    const unsigned xq = (unsigned)x / (unsigned)d;
    q = xq;
    r = (int)((unsigned)x - xq * (unsigned)d);
  } else {
    q = x / d;
    r = (int)(x - q * d);
  }
}

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
  int h_begin, hg;            // of each rank's hl heads, heads [h_begin, h_begin + hg) are sent (a head group);
                              // destination rows then hold hg heads: [row][3][hg][row_bytes]
  int chunks;                 // 16-byte chunks per head row
};

constexpr int kPackVec = 4;      // 16-byte chunks per thread: the index arithmetic is paid once per 64 bytes

__global__ void __launch_bounds__(256) exchange_pack_qkv_kernel(const PackArgs a) {
  // one item = up to kPackVec consecutive chunks of one head row; items ordered (token, which, head, piece):
  // a warp reads a contiguous stretch of one source row and writes contiguous stretches of hl * row_bytes
  const int pieces = (a.chunks + kPackVec - 1) / kPackVec;
  const int sent = a.n_ranks * a.hg;                            // heads sent per token
  const int per_tok = 3 * sent * pieces;
  const long long items = a.n_local * per_tok;
  const bool small = items < (1ll << 32);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (long long)gridDim.x * blockDim.x) {
    long long t;
    int r;
    divmod(i, per_tok, small, t, r);
    const int which = r / (sent * pieces);
    r -= which * sent * pieces;
    const int hs = r / pieces;                                  // index among the heads sent
    const int c0 = (r - hs * pieces) * kPackVec;
    const int g = hs / a.hg;
    const int hj = hs - g * a.hg;                               // head within the group
    const int h = g * a.hl + a.h_begin + hj;                    // head of the source tensor
    const uint4* src = reinterpret_cast<const uint4*>(a.src[which] + t * a.tok_stride_bytes[which] +
                                                      h * a.head_stride_bytes[which]) + c0;
    uint4* dst = reinterpret_cast<uint4*>(a.dst[g]) + (((a.dst_row0 + t) * 3 + which) * a.hg + hj) * a.chunks + c0;
    uint4 v[kPackVec];
#pragma unroll
    for (int u = 0; u < kPackVec; ++u)
      if (c0 + u < a.chunks) v[u] = __ldg(src + u);
#pragma unroll
    for (int u = 0; u < kPackVec; ++u)
      if (c0 + u < a.chunks) dst[u] = v[u];
  }
}

// Receiver's side of the output return: recv[g][t][hl][row_bytes] (what rank g computed for this rank's n
// tokens) -> out[t][g*hl + h][row_bytes], the row-major input of the output projection.  row_bytes is
// whatever one (token, head) record takes on the wire (2*head_dim for bf16, head_dim for raw E4M3, 144 for
// block-INT8 records).  The hl records of one (rank, token) are contiguous on both sides: one run.  Rank g's run
// starts out_rank_chunks 16-byte chunks after rank g-1's in an output row (hl * chunks when recv holds all of a
// rank's heads; larger when recv holds one head group of each rank and out is the full row).
constexpr int kMergeUnroll = 4;  // independent 16-byte copies in flight per thread

__global__ void __launch_bounds__(256) exchange_merge_heads_kernel(const uint8_t* __restrict__ recv,
                                                                   uint8_t* __restrict__ out, long long n, int hl,
                                                                   int n_ranks, int chunks,
                                                                   long long out_tok_stride_bytes, int out_rank_chunks) {
  // one item = one 16-byte chunk, adjacent lanes take adjacent chunks (measured faster here than 64 bytes per lane)
  const int run = hl * chunks;                                  // chunks per (rank, token): contiguous on both sides
  const int per_tok = n_ranks * run;
  const long long items = n * per_tok;
  const bool small = items < (1ll << 32);
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long base = (long long)blockIdx.x * blockDim.x + threadIdx.x; base < items; base += stride * kMergeUnroll) {
    uint4 v[kMergeUnroll];
    uint4* dst[kMergeUnroll];
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u) {
      const long long i = base + u * stride;
      dst[u] = nullptr;
      if (i < items) {
        long long t;
        int r;
        divmod(i, per_tok, small, t, r);
        const int g = r / run;
        r -= g * run;
        v[u] = __ldg(reinterpret_cast<const uint4*>(recv) + ((long long)g * n + t) * run + r);
        dst[u] = reinterpret_cast<uint4*>(out + t * out_tok_stride_bytes) + (long long)g * out_rank_chunks + r;
      }
    }
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u)
      if (dst[u] != nullptr) *dst[u] = v[u];
  }
}

// ---------------------------------------------------------------------------------------------
// Block-INT8 wire formats (Section 3.2, "Quantized communication").  One (token, head) record:
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
  int h_begin, hg;                      // head group, as in PackArgs
  int head_dim, rec_bytes;
};

// NW = 3: the quantising QKV pack (sender's side of the exchange); NW = 1: output rows -> output records.
// rint(x) clamped to int8 in one instruction; |x| <= 127 (1 + 2^-22) here, so the result is within +-127
__device__ __forceinline__ uint32_t rint_sat_s8(float x) {
  int q;
  asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(q) : "f"(x));
  return (uint32_t)q;
}
// low bytes of four registers -> one word, a in the lowest byte
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

// One thread per group of 32 values (64 contiguous bytes in, 32 bytes + one scale code out): the scale search
// and the reciprocal are paid once per group and nothing is exchanged between lanes.  Items are ordered
// (record, tensor, group), so adjacent threads read adjacent 64-byte pieces.
template <int NW>
__global__ void __launch_bounds__(256) quantize_records_kernel(const QuantArgs a) {
  const int ng = a.head_dim >> 5;                               // groups (= scale codes) per tensor
  const int per_rec = NW * ng;                                  // threads per record
  const int sent = a.n_ranks * a.hg;                            // heads (records) written per token
  const long long n_items = a.n_rows * sent * per_rec;
  const bool small = n_items < (1ll << 32);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_items; i += (long long)gridDim.x * blockDim.x) {
    long long rec, t;
    int rem, hs;
    divmod(i, per_rec, small, rec, rem);
    divmod(rec, sent, small, t, hs);
    const int g = hs / a.hg;
    const int hj = hs - g * a.hg;
    const int h = g * a.hl + a.h_begin + hj;                    // head of the source tensor
    const int which = rem / ng;
    const int grp = rem - which * ng;
    const uint4* src = reinterpret_cast<const uint4*>(a.src[which] + t * a.tok_stride_bytes[which] +
                                                      h * a.head_stride_bytes[which] + grp * 64);
    uint4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = __ldg(src + j);
    float f[32];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        f[8 * j + 2 * u] = __uint_as_float(w[u] << 16);          // bf16 -> fp32 is a shift
        f[8 * j + 2 * u + 1] = __uint_as_float(w[u] & 0xffff0000u);
      }
    }
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e) amax = fmaxf(amax, fabsf(f[e]));
    const int code = ue5m3_smallest_cover(amax);
    const float inv = __frcp_rn(ue5m3_value(code));
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      o[j] = pack_low_bytes(rint_sat_s8(__fmul_rn(f[4 * j], inv)), rint_sat_s8(__fmul_rn(f[4 * j + 1], inv)),
                            rint_sat_s8(__fmul_rn(f[4 * j + 2], inv)), rint_sat_s8(__fmul_rn(f[4 * j + 3], inv)));
    uint8_t* out = a.dst[g] + ((a.dst_row0 + t) * a.hg + hj) * a.rec_bytes;
    uint4* dst = reinterpret_cast<uint4*>(out + which * a.head_dim + grp * 32);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    // tail of the record: the scale codes, then zeros up to the record size (written by the record's last thread)
    const int tail = NW * a.head_dim;
    out[tail + rem] = (uint8_t)code;
    if (rem == per_rec - 1) {
      int b = tail + per_rec;
      for (; (b & 3) != 0 && b < a.rec_bytes; ++b) out[b] = 0;
      for (; b < a.rec_bytes; b += 4) *reinterpret_cast<uint32_t*>(out + b) = 0u;   // record sizes are multiples of 16
    }
  }
}

// sixteen int8 values (one 16-byte load) times one scale -> eight packed bf16 pairs, each value q * s rounded to bf16.
// The int8 -> float step avoids the conversion unit: byte b xor 0x80 dropped into the mantissa of 2^23 + 2^22 gives
// m = 12582912 + (q + 128) exactly, and q * s = fma(m, s, -12583040 s): the addend is exact (21 significant bits) and so
// is the result, because q * s itself is representable (7 + 4 significant bits).
__device__ __forceinline__ void dequant16(const uint4 v, float s, uint32_t (&out)[8]) {
  const uint32_t w[4] = {v.x ^ 0x80808080u, v.y ^ 0x80808080u, v.z ^ 0x80808080u, v.w ^ 0x80808080u};
  const float ns = -12583040.0f * s;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float x0 = __fmaf_rn(__uint_as_float(__byte_perm(w[j], 0x4B400000u, 0x7650)), s, ns);
    const float x1 = __fmaf_rn(__uint_as_float(__byte_perm(w[j], 0x4B400000u, 0x7651)), s, ns);
    const float x2 = __fmaf_rn(__uint_as_float(__byte_perm(w[j], 0x4B400000u, 0x7652)), s, ns);
    const float x3 = __fmaf_rn(__uint_as_float(__byte_perm(w[j], 0x4B400000u, 0x7653)), s, ns);
    const __nv_bfloat162 lo = __floats2bfloat162_rn(x0, x1), hi = __floats2bfloat162_rn(x2, x3);
    out[2 * j] = *reinterpret_cast<const uint32_t*>(&lo);
    out[2 * j + 1] = *reinterpret_cast<const uint32_t*>(&hi);
  }
}

// Receiver's side: records [rows][heads][rec_bytes] -> bf16 [rows][NW][heads][D] (NW = 3: the packed QKV tensor
// the attention reads through strides; NW = 1: output rows).  value = q * s, exact in fp32, one rounding to bf16.
template <int NW>
__global__ void __launch_bounds__(256) dequantize_records_kernel(const uint8_t* __restrict__ recs,
                                                                 __nv_bfloat16* __restrict__ out, long long n_rows,
                                                                 int heads, int head_dim, int rec_bytes) {
  // one thread per group of 32 values: 32 bytes + one code in, 64 bytes out; items ordered (record, tensor, group)
  const int ng = head_dim >> 5;
  const int per_rec = NW * ng;
  const long long n_items = n_rows * heads * per_rec;
  const bool small = n_items < (1ll << 32);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_items; i += (long long)gridDim.x * blockDim.x) {
    long long rec, t;
    int rem, h;
    divmod(i, per_rec, small, rec, rem);
    divmod(rec, heads, small, t, h);
    const int which = rem / ng;
    const int grp = rem - which * ng;
    const uint8_t* r = recs + rec * rec_bytes;
    const uint4* src = reinterpret_cast<const uint4*>(r + which * head_dim + grp * 32);
    const uint4 v0 = __ldg(src), v1 = __ldg(src + 1);
    const float s = ue5m3_value(__ldg(r + NW * head_dim + rem));
    uint32_t o0[8], o1[8];
    dequant16(v0, s, o0);
    dequant16(v1, s, o1);
    uint4* dst = reinterpret_cast<uint4*>(out + (((t * NW + which) * heads + h) * (long long)head_dim + grp * 32));
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      dst[j] = make_uint4(o0[4 * j], o0[4 * j + 1], o0[4 * j + 2], o0[4 * j + 3]);
      dst[2 + j] = make_uint4(o1[4 * j], o1[4 * j + 1], o1[4 * j + 2], o1[4 * j + 3]);
    }
  }
}

}  // namespace sol
