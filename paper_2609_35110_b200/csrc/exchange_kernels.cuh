// Layout kernels of the sequence-parallel exchange around the attention (Section 3.3, "Optimized attention
// collectives"): the stride-aware QKV pack that writes the exchange buffer in one pass, and the inverse head
// merge on the return path.  Both move 16-byte chunks and change no byte.
#pragma once
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

}  // namespace sol
