// Host side of the C-ABI library: plan (pure host), workspace binding, forward.
#include "../../include/sol_attn3d.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "attn_fwd_sm100.cuh"
#include "device_types.cuh"
#include "prologue_kernels.cuh"
#include "sparse_kernels.cuh"

namespace {

using sol::SeqDev;

constexpr size_t kAlign = 256;
constexpr size_t kCountersOffset = 64;   // diagnostic counters inside the 256-byte status block of a workspace
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

struct Strides {
  long long tok, head;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct sol_attn3d_plan_s {
  int n_seqs = 0, heads = 0, head_dim = 0;
  int rope[3] = {0, 0, 0};
  double theta = 10000.0;
  Strides sq{}, sk{}, sv{}, so{};
  std::vector<int64_t> cu;            // caller order
  std::vector<SeqDev> sched;          // schedule order (longest first)
  long long total_tokens = 0;
  int total_work = 0;
  int total_quad_work = 0;            // work items when CTA pairs serve 512-row query blocks
  int pair_mode = 1;                  // CTA pairs (cta_group::2) where they apply: head_dim 128, not block-sparse
  int total_ktiles = 0;
  std::vector<float2> tables;
  int tab_off[3] = {0, 0, 0};

  // workspace layout (byte offsets)
  size_t off_status = 0, off_tables = 0, off_seqs = 0, off_keybits = 0, off_list = 0, off_count = 0, off_pairs = 0,
         off_qrot = 0, off_krot = 0, ws_bytes = 0;
  int total_pairs = 0;
  unsigned char* ws = nullptr;
  // block-sparse scratch (passed per call): byte offsets
  size_t sp_off_stats = 0, sp_off_count = 0, sp_off_qbar = 0, sp_off_kbar = 0, sp_off_list = 0, sp_bytes = 0;
  std::vector<size_t> sp_qbar_seq, sp_kbar_seq;   // per sequence (schedule order), in floats

  EncodeTiledFn encode = nullptr;
  CUtensorMap tm_q{}, tm_k{}, tm_v{};
  CUtensorMap tm_k64{};               // K~ with 64-token boxes: what one CTA of a pair loads of a key tile
  const void* v_cached = nullptr;
  bool v_cached_dense = false;        // the cached V map was encoded with dense strides (inputs were records)
  int keybits_state = 0;              // 0 unknown, 1 built for "no mask", 2 built from a mask
  int last_cuda = 0;
  unsigned long long wait_limit_ns = 2000000000ull;
  unsigned int v_lbo = 0, v_sbo = 1024;
  unsigned int fault_inject = 0;
  cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
  bool prof = false, prof_valid = false, prof_bits = false;
  // sol_attn3d_forward_host: copy streams and events, created on first use
  cudaStream_t s_h2d = nullptr, s_d2h = nullptr, s_alt = nullptr;
  cudaEvent_t ev_start = nullptr, ev_done = nullptr, ev_bits = nullptr, ev_in[8] = {}, ev_out[8] = {};
  bool host_pipe_ready = false;
  int sm_count = 148;                 // of the device the workspace was bound on
  int launches = 0;                   // kernels enqueued by the most recent forward-type call
};

namespace {

int fail_cuda(sol_attn3d_plan_t p, cudaError_t e) {
  p->last_cuda = (int)e;
  (void)cudaGetLastError();
  return SOL_ATTN3D_ERR_CUDA;
}

// Streams and events of sol_attn3d_forward_host (host-side objects only).
void release_host_pipe(sol_attn3d_plan_t p) {
  if (p->s_h2d != nullptr) (void)cudaStreamDestroy(p->s_h2d);
  if (p->s_d2h != nullptr) (void)cudaStreamDestroy(p->s_d2h);
  if (p->s_alt != nullptr) (void)cudaStreamDestroy(p->s_alt);
  if (p->ev_start != nullptr) (void)cudaEventDestroy(p->ev_start);
  if (p->ev_done != nullptr) (void)cudaEventDestroy(p->ev_done);
  if (p->ev_bits != nullptr) (void)cudaEventDestroy(p->ev_bits);
  for (int g = 0; g < 8; ++g) {
    if (p->ev_in[g] != nullptr) (void)cudaEventDestroy(p->ev_in[g]);
    if (p->ev_out[g] != nullptr) (void)cudaEventDestroy(p->ev_out[g]);
    p->ev_in[g] = p->ev_out[g] = nullptr;
  }
  p->s_h2d = p->s_d2h = p->s_alt = nullptr;
  p->ev_start = p->ev_done = p->ev_bits = nullptr;
  p->host_pipe_ready = false;
}

// The attention kernels use more dynamic shared memory than the default limit (per device, idempotent).
cudaError_t raise_shared_memory_limits() {
  cudaError_t e = cudaFuncSetAttribute(sol::attn_fwd_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       sol::AttnSmem<128, 1>::kDynBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(sol::attn_fwd_kernel<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sol::AttnSmem<64, 1>::kDynBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(sol::attn_fwd_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sol::AttnSmem<128, 2>::kDynBytes);
  return e;
}

bool stride_ok(long long s) { return s > 0 && (s * 2) % 16 == 0 && (s * 2) < (1ll << 40); }

int build_plan(sol_attn3d_plan_t* out, const sol_attn3d_desc* d) {
  if (out == nullptr || d == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (d->size != sizeof(sol_attn3d_desc)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (d->n_seqs < 1 || d->grids == nullptr || d->text_lens == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (d->heads < 1 || d->head_dim < 1) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (!(d->theta > 1.0) || !std::isfinite(d->theta)) return SOL_ATTN3D_ERR_INVALID_ARG;
  int rope_sum = 0;
  for (int a = 0; a < 3; ++a) {
    if (d->rope_dims[a] < 0 || (d->rope_dims[a] & 1)) return SOL_ATTN3D_ERR_INVALID_ARG;
    rope_sum += d->rope_dims[a];
  }
  if (d->head_dim != 64 && d->head_dim != 128) return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;
  if (rope_sum > d->head_dim) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (d->heads > 65535) return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;

  sol_attn3d_plan_s* p = new (std::nothrow) sol_attn3d_plan_s();
  if (p == nullptr) return SOL_ATTN3D_ERR_NO_MEMORY;
  int rc = SOL_ATTN3D_OK;
  try {
    p->n_seqs = d->n_seqs;
    p->heads = d->heads;
    p->head_dim = d->head_dim;
    p->theta = d->theta;
    for (int a = 0; a < 3; ++a) p->rope[a] = d->rope_dims[a];

    const long long dense_tok = (long long)d->heads * d->head_dim;
    auto take = [&](const int64_t s[2], Strides* dst) {
      dst->tok = s[0] == 0 ? dense_tok : s[0];
      dst->head = s[1] == 0 ? d->head_dim : s[1];
      return stride_ok(dst->tok) && stride_ok(dst->head);
    };
    if (!take(d->q_strides, &p->sq) || !take(d->k_strides, &p->sk) || !take(d->v_strides, &p->sv) ||
        !take(d->out_strides, &p->so)) {
      delete p;
      return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;
    }

    int max_pos[3] = {1, 1, 1};
    p->cu.assign(1, 0);
    std::vector<SeqDev> seqs((size_t)d->n_seqs);
    for (int s = 0; s < d->n_seqs; ++s) {
      const int T = d->grids[3 * s], H = d->grids[3 * s + 1], W = d->grids[3 * s + 2];
      const int L = d->text_lens[s];
      if (T < 0 || H < 1 || W < 1 || L < 0) { rc = SOL_ATTN3D_ERR_INVALID_ARG; break; }
      const long long nv = (long long)T * H * W;
      const long long n = nv + L;
      if (n < 1) { rc = SOL_ATTN3D_ERR_INVALID_ARG; break; }
      if (n > (1ll << 30)) { rc = SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE; break; }
      SeqDev& q = seqs[(size_t)s];
      q.tok_start = p->cu.back();
      q.n_tokens = (int)n;
      q.text_len = L;
      q.T = T; q.H = H; q.W = W;
      q.n_qpairs = (int)((n + 255) / 256);
      q.n_ktiles = (int)((n + 127) / 128);
      q.seq_id = s;
      p->cu.push_back(p->cu.back() + n);
      max_pos[0] = std::max(max_pos[0], T);
      max_pos[1] = std::max(max_pos[1], H);
      max_pos[2] = std::max(max_pos[2], W);
    }
    if (rc == SOL_ATTN3D_OK) {
      p->total_tokens = p->cu.back();
      if (p->total_tokens >= (1ll << 31) - 256) rc = SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;
    }
    if (rc != SOL_ATTN3D_OK) {
      delete p;
      return rc;
    }

    // schedule: longest sequence first; inside a sequence head-major with the query pair fastest,
    // so that CTAs running together stream the same head's K/V through L2
    std::stable_sort(seqs.begin(), seqs.end(), [](const SeqDev& a, const SeqDev& b) { return a.n_tokens > b.n_tokens; });
    long long work = 0;
    long long quad_work = 0;
    long long ktiles = 0;
    long long pairs = 0;
    for (SeqDev& q : seqs) {
      q.work_start = (int)work;
      q.quad_work_start = (int)quad_work;
      quad_work += (long long)((q.n_qpairs + 1) / 2) * d->heads;
      q.ktile_start = (int)ktiles;
      q.pair_start = (int)pairs;
      pairs += q.n_qpairs;
      work += (long long)q.n_qpairs * d->heads;
      ktiles += q.n_ktiles;
      if (work > 0x7fffffffll) break;
    }
    if (work > 0x7fffffffll) {
      delete p;
      return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;
    }
    {
      // block-sparse mode: per-CTA key-tile lists (n_ktiles slots each), pooled operands per sequence
      long long list_slots = 0;
      size_t qbar = 0, kbar = 0;
      for (SeqDev& q : seqs) {
        q.sparse_list_start = list_slots;
        list_slots += (long long)q.n_qpairs * d->heads * q.n_ktiles;
        p->sp_qbar_seq.push_back(qbar);
        p->sp_kbar_seq.push_back(kbar);
        qbar += (size_t)d->heads * q.n_qpairs * d->head_dim;
        kbar += (size_t)d->heads * q.n_ktiles * d->head_dim;
      }
      size_t o = 0;
      p->sp_off_stats = o; o = align_up(o + 256);
      p->sp_off_count = o; o = align_up(o + (size_t)work * sizeof(int));
      p->sp_off_qbar = o;  o = align_up(o + qbar * sizeof(float));
      p->sp_off_kbar = o;  o = align_up(o + kbar * sizeof(float));
      p->sp_off_list = o;  o = align_up(o + (size_t)list_slots * sizeof(int));
      p->sp_bytes = o;
    }
    p->sched = seqs;
    p->total_work = (int)work;
    p->total_quad_work = (int)quad_work;
    p->total_ktiles = (int)ktiles;
    p->total_pairs = (int)pairs;

    // cos/sin tables, built in fp64 and rounded once to fp32
    size_t n_entries = 0;
    for (int a = 0; a < 3; ++a) {
      p->tab_off[a] = (int)n_entries;
      n_entries += (size_t)max_pos[a] * (size_t)(p->rope[a] / 2);
    }
    p->tables.resize(std::max<size_t>(n_entries, 1));
    for (int a = 0; a < 3; ++a) {
      const int half = p->rope[a] / 2;
      for (int pos = 0; pos < max_pos[a]; ++pos)
        for (int j = 0; j < half; ++j) {
          const double omega = std::exp(-(2.0 * j / p->rope[a]) * std::log(p->theta));
          const double phi = pos * omega;
          p->tables[(size_t)p->tab_off[a] + (size_t)pos * half + j] = make_float2((float)std::cos(phi), (float)std::sin(phi));
        }
    }

    // workspace layout
    size_t off = 0;
    p->off_status = off;  off = align_up(off + 256);
    p->off_tables = off;  off = align_up(off + p->tables.size() * sizeof(float2));
    p->off_seqs = off;    off = align_up(off + p->sched.size() * sizeof(SeqDev));
    p->off_keybits = off; off = align_up(off + (size_t)p->total_ktiles * 16);
    p->off_list = off;    off = align_up(off + (size_t)p->total_ktiles * sizeof(int));
    p->off_count = off;   off = align_up(off + (size_t)p->n_seqs * sizeof(int));
    p->off_pairs = off;   off = align_up(off + (size_t)p->total_pairs);
    const size_t rot = (size_t)p->total_tokens * p->heads * p->head_dim * 2;
    p->off_qrot = off;    off = align_up(off + rot);
    p->off_krot = off;    off = align_up(off + rot);
    p->ws_bytes = off;

    if (const char* e = std::getenv("SOL_ATTN3D_WAIT_LIMIT_MS")) {
      const long v = std::atol(e);
      if (v > 0) p->wait_limit_ns = (unsigned long long)v * 1000000ull;
    }
    // Test hook for the failure-detection path: a wait inside the kernel is made to run out on purpose.
    if (const char* e = std::getenv("SOL_ATTN3D_FAULT_INJECT")) p->fault_inject = (unsigned)std::atol(e);
    // SOL_ATTN3D_PAIR=0 keeps every launch of this plan on single CTAs (for comparisons and tests).  By default two
    // CTAs on neighbouring SMs share every K / V tile (one tcgen05.mma.cta_group::2 over both CTAs' query rows):
    // half the L2 -> SM traffic and B-operand reads, which buys SM clock under the power cap at the large sizes.
    if (const char* e = std::getenv("SOL_ATTN3D_PAIR")) p->pair_mode = std::atol(e) != 0;
    p->v_lbo = p->head_dim == 128 ? 16384u : 16u;
    p->v_sbo = 1024u;
  } catch (const std::bad_alloc&) {
    delete p;
    return SOL_ATTN3D_ERR_NO_MEMORY;
  }
  *out = p;
  return SOL_ATTN3D_OK;
}

// [tokens][heads][D] bf16 tensor as a 3-D TMA map with 128 x 64-element boxes, 128-byte swizzle.
int encode_map(EncodeTiledFn fn, sol_attn3d_plan_t p, CUtensorMap* tm, const void* base, Strides st, unsigned box_tokens = 128) {
  const cuuint64_t dims[3] = {(cuuint64_t)p->head_dim, (cuuint64_t)p->heads, (cuuint64_t)p->total_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)st.head * 2, (cuuint64_t)st.tok * 2};
  const cuuint32_t box[3] = {64, 1, box_tokens};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    p->last_cuda = (int)r;
    return SOL_ATTN3D_ERR_CUDA;
  }
  return SOL_ATTN3D_OK;
}

bool aligned16(const void* x) { return (reinterpret_cast<uintptr_t>(x) & 15u) == 0; }

int launch_rope(sol_attn3d_plan_t p, const unsigned char* ws, const void* q, const void* k, void* qr, void* kr,
                const float* q_gain, const float* k_gain, float eps, cudaStream_t st, int head_begin = 0,
                int head_end = 0) {
  sol::RopeArgs a{};
  a.gain[0] = q_gain;
  a.gain[1] = k_gain;
  a.eps = eps;
  a.x[0] = static_cast<const __nv_bfloat16*>(q);
  a.x[1] = static_cast<const __nv_bfloat16*>(k);
  a.y[0] = static_cast<__nv_bfloat16*>(qr);
  a.y[1] = static_cast<__nv_bfloat16*>(kr);
  a.x_tok_stride[0] = p->sq.tok; a.x_head_stride[0] = p->sq.head;
  a.x_tok_stride[1] = p->sk.tok; a.x_head_stride[1] = p->sk.head;
  a.seqs = reinterpret_cast<const SeqDev*>(ws + p->off_seqs);
  a.n_seqs = p->n_seqs;
  a.total_tokens = p->total_tokens;
  a.tables = reinterpret_cast<const float2*>(ws + p->off_tables);
  for (int i = 0; i < 3; ++i) { a.g.rope[i] = p->rope[i]; a.g.tab_off[i] = p->tab_off[i]; }
  a.g.head_dim = p->head_dim;
  a.g.heads = p->heads;
  a.head_begin = head_begin;
  a.head_end = head_end > 0 ? head_end : p->heads;
  a.status = const_cast<unsigned int*>(reinterpret_cast<const unsigned int*>(ws + p->off_status));
  const int chunks = p->head_dim / 8;
  // heads per pass: the largest divisor of the head count that fits a 256-thread block, so that all threads carry the
  // same number of rows; a head count without a usable divisor (a large prime) takes what fits
  const int n_heads = a.head_end - a.head_begin, cap = 256 / chunks;
  const bool norm = q_gain != nullptr || k_gain != nullptr;
  int hpp = std::max(1, std::min(n_heads, cap));
  for (int d = std::min(n_heads, cap); d >= std::max(1, cap / 2); --d)
    if (n_heads % d == 0) { hpp = d; break; }
  const int threads = chunks * hpp;
  const long long blocks = std::min<long long>(p->total_tokens, 148ll * 16);
  if (norm) sol::rope_qk_kernel<true><<<(unsigned)blocks, threads, 0, st>>>(a);
  else                                        sol::rope_qk_kernel<false><<<(unsigned)blocks, threads, 0, st>>>(a);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(p, e);
  ++p->launches;
  return SOL_ATTN3D_OK;
}

}  // namespace

extern "C" {

int sol_attn3d_plan(sol_attn3d_plan_t* plan, int B, int heads, int head_dim, int T, int H, int W, int text_len,
                    const int rope_dims[3]) {
  if (plan == nullptr || rope_dims == nullptr || B < 1 || B > (1 << 20)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (T < 1) return SOL_ATTN3D_ERR_INVALID_ARG;
  std::vector<int32_t> grids, lens;
  try {
    grids.resize((size_t)B * 3);
    lens.resize((size_t)B);
  } catch (const std::bad_alloc&) {
    return SOL_ATTN3D_ERR_NO_MEMORY;
  }
  for (int b = 0; b < B; ++b) {
    grids[3 * b] = T; grids[3 * b + 1] = H; grids[3 * b + 2] = W;
    lens[b] = text_len;
  }
  sol_attn3d_desc d;
  std::memset(&d, 0, sizeof(d));
  d.size = sizeof(d);
  d.n_seqs = B;
  d.grids = grids.data();
  d.text_lens = lens.data();
  d.heads = heads;
  d.head_dim = head_dim;
  for (int a = 0; a < 3; ++a) d.rope_dims[a] = rope_dims[a];
  d.theta = 10000.0;
  return build_plan(plan, &d);
}

int sol_attn3d_plan_ex(sol_attn3d_plan_t* plan, const sol_attn3d_desc* desc) { return build_plan(plan, desc); }

int sol_attn3d_cu_seqlens(sol_attn3d_plan_t plan, const int64_t** cu, int* n_seqs) {
  if (plan == nullptr || cu == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  *cu = plan->cu.data();
  if (n_seqs) *n_seqs = plan->n_seqs;
  return SOL_ATTN3D_OK;
}

size_t sol_attn3d_workspace_bytes(sol_attn3d_plan_t plan) { return plan ? plan->ws_bytes : 0; }

int sol_attn3d_set_workspace(sol_attn3d_plan_t p, void* device_ptr, size_t bytes) {
  if (p == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (device_ptr == nullptr || bytes < p->ws_bytes || (reinterpret_cast<uintptr_t>(device_ptr) % kAlign) != 0)
    return SOL_ATTN3D_ERR_NO_WORKSPACE;
  int dev = 0, n_dev = 0;
  cudaError_t e = cudaGetDeviceCount(&n_dev);
  if (e != cudaSuccess || n_dev == 0) {
    (void)cudaGetLastError();
    return SOL_ATTN3D_ERR_NO_DEVICE;
  }
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return fail_cuda(p, e);
  int major = 0;
  if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess) return fail_cuda(p, e);
  if (major != 10) return SOL_ATTN3D_ERR_UNSUPPORTED_ARCH;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) p->sm_count = sms;

  if (p->encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return fail_cuda(p, e);
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return SOL_ATTN3D_ERR_CUDA;   // driver too old for TMA
    p->encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  if ((e = raise_shared_memory_limits()) != cudaSuccess) return fail_cuda(p, e);

  p->ws = static_cast<unsigned char*>(device_ptr);
  p->keybits_state = 0;
  p->v_cached = nullptr;
  if ((e = cudaMemset(p->ws + p->off_status, 0, 256)) != cudaSuccess) return fail_cuda(p, e);
  if ((e = cudaMemcpy(p->ws + p->off_tables, p->tables.data(), p->tables.size() * sizeof(float2),
                      cudaMemcpyHostToDevice)) != cudaSuccess)
    return fail_cuda(p, e);
  if ((e = cudaMemcpy(p->ws + p->off_seqs, p->sched.data(), p->sched.size() * sizeof(SeqDev),
                      cudaMemcpyHostToDevice)) != cudaSuccess)
    return fail_cuda(p, e);
  const Strides dense{(long long)p->heads * p->head_dim, (long long)p->head_dim};
  int rc = encode_map(p->encode, p, &p->tm_q, p->ws + p->off_qrot, dense);
  if (rc == SOL_ATTN3D_OK) rc = encode_map(p->encode, p, &p->tm_k, p->ws + p->off_krot, dense);
  if (rc == SOL_ATTN3D_OK) rc = encode_map(p->encode, p, &p->tm_k64, p->ws + p->off_krot, dense, 64);
  return rc;
}

int sol_attn3d_rope_qk(sol_attn3d_plan_t p, const void* q, const void* k, void* q_rot, void* k_rot,
                       sol_attn3d_stream_t stream) {
  if (p == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  if ((q == nullptr) != (q_rot == nullptr) || (k == nullptr) != (k_rot == nullptr)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (q == nullptr && k == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(q_rot) || !aligned16(k_rot)) return SOL_ATTN3D_ERR_INVALID_ARG;
  p->launches = 0;
  return launch_rope(p, p->ws, q, k, q_rot, k_rot, nullptr, nullptr, 0.f, static_cast<cudaStream_t>(stream));
}

namespace {
// Optional parts of a forward call.
struct FwdOpts {
  const float* q_gain = nullptr;      // QK RMS-norm gains (both or neither)
  const float* k_gain = nullptr;
  float eps = 0.f;
  unsigned char* sparse_ws = nullptr; // block-sparse scratch
  float tau = 0.f;
  const uint8_t* query_mask = nullptr;
  int out_fmt = sol::kOutBf16;
  int n_dst = 0;                      // > 0: rows are scattered to their token owners instead of `out`
  void* const* dst = nullptr;
  const int64_t* tok_begin = nullptr;
  int dst_heads = 0, head_offset = 0;
  int head_begin = 0, head_end = 0;   // serve heads [head_begin, head_end) only (0, 0 = all)
  const void* qkv_records = nullptr;  // Q, K, V arrive as block-INT8 records (q and k are then NULL, v is a bf16 scratch)
  bool skip_keybits = false;          // the key-validity bits of this mask were built by an earlier call
  bool keep_launch_count = false;     // one of several launch sets of the same API call: keep counting
  cudaEvent_t bits_done = nullptr;    // recorded on the stream once the key-validity bits are in place (built or kept)
  // Scratch other than the plan's bound workspace (sol_attn3d_forward_noalloc): the caller of forward_impl has put
  // the tables and the sequence table there; nothing about it is cached in the plan.
  unsigned char* ws = nullptr;
  unsigned int* status = nullptr;     // status word to use instead of the one inside the scratch
  EncodeTiledFn encode = nullptr;     // tensor-map encoder for such a call
  int sm_count = 0;                   // SMs of the current device for such a call (the plan may never have been bound)
};
int forward_impl(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out, const uint8_t* key_mask,
                 sol_attn3d_stream_t stream, const FwdOpts& o);
}

int sol_attn3d_forward(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out,
                       const uint8_t* key_mask, sol_attn3d_stream_t stream) {
  return forward_impl(p, q, k, v, out, key_mask, stream, FwdOpts{});
}

int sol_attn3d_forward_qknorm(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out,
                              const uint8_t* key_mask, const float* q_gain, const float* k_gain, float eps,
                              sol_attn3d_stream_t stream) {
  if (q_gain == nullptr || k_gain == nullptr || !(eps >= 0.f)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_gain) & 3u) != 0 || (reinterpret_cast<uintptr_t>(k_gain) & 3u) != 0)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  FwdOpts o;
  o.q_gain = q_gain;
  o.k_gain = k_gain;
  o.eps = eps;
  return forward_impl(p, q, k, v, out, key_mask, stream, o);
}

int sol_attn3d_forward_rect(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out,
                            const uint8_t* key_mask, const uint8_t* query_mask, sol_attn3d_stream_t stream) {
  if (query_mask == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  FwdOpts o;
  o.query_mask = query_mask;
  return forward_impl(p, q, k, v, out, key_mask, stream, o);
}

int sol_attn3d_forward_e4m3(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out_e4m3,
                            const uint8_t* key_mask, sol_attn3d_stream_t stream) {
  FwdOpts o;
  o.out_fmt = sol::kOutE4M3;
  return forward_impl(p, q, k, v, out_e4m3, key_mask, stream, o);
}

int sol_attn3d_forward_qkv_int8(sol_attn3d_plan_t p, const void* qkv_records, void* v_scratch, void* out,
                                const uint8_t* key_mask, int out_format, sol_attn3d_stream_t stream) {
  if (qkv_records == nullptr || v_scratch == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (out_format != SOL_ATTN3D_OUT_BF16 && out_format != SOL_ATTN3D_OUT_E4M3 && out_format != SOL_ATTN3D_OUT_INT8)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  if (out == qkv_records) return SOL_ATTN3D_ERR_INVALID_ARG;
  FwdOpts o;
  o.qkv_records = qkv_records;
  o.out_fmt = out_format == SOL_ATTN3D_OUT_E4M3 ? sol::kOutE4M3 : out_format == SOL_ATTN3D_OUT_INT8 ? sol::kOutInt8 : sol::kOutBf16;
  return forward_impl(p, nullptr, nullptr, v_scratch, out, key_mask, stream, o);
}

int sol_attn3d_forward_int8(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out_records,
                            const uint8_t* key_mask, sol_attn3d_stream_t stream) {
  FwdOpts o;
  o.out_fmt = sol::kOutInt8;
  return forward_impl(p, q, k, v, out_records, key_mask, stream, o);
}

int sol_attn3d_forward_scatter(sol_attn3d_plan_t p, const void* q, const void* k, const void* v,
                               const uint8_t* key_mask, int n_dst, void* const* dst, const int64_t* tok_begin,
                               int dst_heads, int head_offset, int out_format, sol_attn3d_stream_t stream) {
  if (n_dst < 1 || (out_format != SOL_ATTN3D_OUT_BF16 && out_format != SOL_ATTN3D_OUT_E4M3 && out_format != SOL_ATTN3D_OUT_INT8))
    return SOL_ATTN3D_ERR_INVALID_ARG;
  FwdOpts o;
  o.out_fmt = out_format == SOL_ATTN3D_OUT_E4M3 ? sol::kOutE4M3 : out_format == SOL_ATTN3D_OUT_INT8 ? sol::kOutInt8 : sol::kOutBf16;
  o.n_dst = n_dst;
  o.dst = dst;
  o.tok_begin = tok_begin;
  o.dst_heads = dst_heads;
  o.head_offset = head_offset;
  return forward_impl(p, q, k, v, nullptr, key_mask, stream, o);
}

int sol_attn3d_exchange_pack_qkv(const void* q, const void* k, const void* v, const int64_t q_strides[2],
                                 const int64_t k_strides[2], const int64_t v_strides[2], int64_t n_local, int heads,
                                 int head_dim, int n_ranks, int group_begin, int group_heads, void* const* dst,
                                 int64_t dst_row0, sol_attn3d_stream_t stream) {
  if (n_local < 0 || dst_row0 < 0 || heads < 1 || head_dim < 8 || (head_dim % 8) != 0 || n_ranks < 1 ||
      n_ranks > sol::kMaxRanks || (heads % n_ranks) != 0)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  if (group_heads == 0) group_heads = heads / n_ranks - group_begin;
  if (group_begin < 0 || group_heads < 1 || group_begin + group_heads > heads / n_ranks) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (n_local == 0) return SOL_ATTN3D_OK;            // a rank without tokens sends nothing (its pointers may be NULL)
  if (q == nullptr || k == nullptr || v == nullptr || dst == nullptr || q_strides == nullptr || k_strides == nullptr ||
      v_strides == nullptr)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  sol::PackArgs a{};
  const void* src[3] = {q, k, v};
  const int64_t* strides[3] = {q_strides, k_strides, v_strides};
  for (int w = 0; w < 3; ++w) {
    const long long tok = strides[w][0] == 0 ? (long long)heads * head_dim : strides[w][0];
    const long long head = strides[w][1] == 0 ? head_dim : strides[w][1];
    if (!aligned16(src[w]) || !stride_ok(tok) || !stride_ok(head)) return SOL_ATTN3D_ERR_INVALID_ARG;
    a.src[w] = static_cast<const uint8_t*>(src[w]);
    a.tok_stride_bytes[w] = tok * 2;
    a.head_stride_bytes[w] = head * 2;
  }
  for (int g = 0; g < n_ranks; ++g) {
    if (dst[g] == nullptr || !aligned16(dst[g])) return SOL_ATTN3D_ERR_INVALID_ARG;
    a.dst[g] = static_cast<uint8_t*>(dst[g]);
  }
  a.dst_row0 = dst_row0;
  a.n_local = n_local;
  a.heads = heads;
  a.hl = heads / n_ranks;
  a.n_ranks = n_ranks;
  a.h_begin = group_begin;
  a.hg = group_heads;
  a.chunks = head_dim * 2 / 16;
  const long long items = n_local * 3ll * n_ranks * group_heads * ((a.chunks + sol::kPackVec - 1) / sol::kPackVec);
  const long long want = (items + 255) / 256;
  const unsigned blocks = (unsigned)std::max<long long>(1, std::min<long long>(want, 148ll * 16));
  sol::exchange_pack_qkv_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? SOL_ATTN3D_OK : SOL_ATTN3D_ERR_CUDA;
}

int sol_attn3d_exchange_merge_heads(const void* recv, void* out, int64_t n_local, int heads, int record_bytes,
                                    int n_ranks, int64_t out_tok_stride_bytes, int64_t out_rank_stride_bytes,
                                    sol_attn3d_stream_t stream) {
  if (n_local < 0 || heads < 1 || record_bytes < 16 || (record_bytes % 16) != 0 || n_ranks < 1 ||
      n_ranks > sol::kMaxRanks || (heads % n_ranks) != 0)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  if (n_local == 0) return SOL_ATTN3D_OK;            // a rank without tokens receives nothing
  if (recv == nullptr || out == nullptr || recv == out || !aligned16(recv) || !aligned16(out))
    return SOL_ATTN3D_ERR_INVALID_ARG;
  const long long run_bytes = (long long)(heads / n_ranks) * record_bytes;
  const long long ors = out_rank_stride_bytes == 0 ? run_bytes : out_rank_stride_bytes;
  if (ors < run_bytes || (ors % 16) != 0) return SOL_ATTN3D_ERR_INVALID_ARG;
  const long long dense = ors * (n_ranks - 1) + run_bytes;
  const long long ots = out_tok_stride_bytes == 0 ? dense : out_tok_stride_bytes;
  if (ots < dense || (ots % 16) != 0) return SOL_ATTN3D_ERR_INVALID_ARG;
  const int chunks = record_bytes / 16;
  const long long items = n_local * (long long)heads * chunks;
  const long long want = (items + 256ll * sol::kMergeUnroll - 1) / (256ll * sol::kMergeUnroll);
  const unsigned blocks = (unsigned)std::max<long long>(1, std::min<long long>(want, 148ll * 16));
  sol::exchange_merge_heads_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint8_t*>(recv), static_cast<uint8_t*>(out), n_local, heads / n_ranks, n_ranks, chunks, ots,
      (int)(ors / 16));
  return cudaGetLastError() == cudaSuccess ? SOL_ATTN3D_OK : SOL_ATTN3D_ERR_CUDA;
}

size_t sol_attn3d_exchange_record_bytes(int kind, int head_dim) {
  if (head_dim != 64 && head_dim != 128) return 0;
  const size_t groups = (size_t)head_dim / 32;
  switch (kind) {
    case SOL_ATTN3D_WIRE_QKV_BF16: return 3u * head_dim * 2u;
    case SOL_ATTN3D_WIRE_QKV_INT8: return (3u * head_dim + 3u * groups + 15u) / 16u * 16u;
    case SOL_ATTN3D_WIRE_OUT_BF16: return (size_t)head_dim * 2u;
    case SOL_ATTN3D_WIRE_OUT_E4M3: return (size_t)head_dim;
    case SOL_ATTN3D_WIRE_OUT_INT8: return ((size_t)head_dim + groups + 15u) / 16u * 16u;
    default: return 0;
  }
}

extern "C++" {
namespace {
template <int NW>
int launch_quantize(const void* const src[3], const int64_t* const strides[3], int64_t n_rows, int heads, int head_dim,
                    int n_ranks, int group_begin, int group_heads, void* const* dst, int64_t dst_row0, size_t rec_bytes,
                    cudaStream_t st) {
  if (n_rows < 0 || dst_row0 < 0 || heads < 1 || (head_dim != 64 && head_dim != 128) || n_ranks < 1 ||
      n_ranks > sol::kMaxRanks || (heads % n_ranks) != 0)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  if (group_heads == 0) group_heads = heads / n_ranks - group_begin;
  if (group_begin < 0 || group_heads < 1 || group_begin + group_heads > heads / n_ranks) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (n_rows == 0) return SOL_ATTN3D_OK;
  if (dst == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  sol::QuantArgs a{};
  for (int w = 0; w < NW; ++w) {
    if (src[w] == nullptr || strides[w] == nullptr || !aligned16(src[w])) return SOL_ATTN3D_ERR_INVALID_ARG;
    const long long tok = strides[w][0] == 0 ? (long long)heads * head_dim : strides[w][0];
    const long long head = strides[w][1] == 0 ? head_dim : strides[w][1];
    if (!stride_ok(tok) || !stride_ok(head)) return SOL_ATTN3D_ERR_INVALID_ARG;
    a.src[w] = static_cast<const uint8_t*>(src[w]);
    a.tok_stride_bytes[w] = tok * 2;
    a.head_stride_bytes[w] = head * 2;
  }
  for (int g = 0; g < n_ranks; ++g) {
    if (dst[g] == nullptr || !aligned16(dst[g])) return SOL_ATTN3D_ERR_INVALID_ARG;
    a.dst[g] = static_cast<uint8_t*>(dst[g]);
  }
  a.dst_row0 = dst_row0;
  a.n_rows = n_rows;
  a.heads = heads;
  a.hl = heads / n_ranks;
  a.n_ranks = n_ranks;
  a.h_begin = group_begin;
  a.hg = group_heads;
  a.head_dim = head_dim;
  a.rec_bytes = (int)rec_bytes;
  const long long n_items = n_rows * n_ranks * group_heads * (long long)(NW * head_dim / 32);   // one thread per group of 32 values
  const unsigned blocks = (unsigned)std::max<long long>(1, std::min<long long>((n_items + 255) / 256, 148ll * 16));
  sol::quantize_records_kernel<NW><<<blocks, 256, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? SOL_ATTN3D_OK : SOL_ATTN3D_ERR_CUDA;
}
}  // namespace
}  // extern "C++"

int sol_attn3d_exchange_pack_qkv_int8(const void* q, const void* k, const void* v, const int64_t q_strides[2],
                                      const int64_t k_strides[2], const int64_t v_strides[2], int64_t n_local, int heads,
                                      int head_dim, int n_ranks, int group_begin, int group_heads, void* const* dst,
                                      int64_t dst_row0, sol_attn3d_stream_t stream) {
  const void* const src[3] = {q, k, v};
  const int64_t* const strides[3] = {q_strides, k_strides, v_strides};
  return launch_quantize<3>(src, strides, n_local, heads, head_dim, n_ranks, group_begin, group_heads, dst, dst_row0,
                            sol_attn3d_exchange_record_bytes(SOL_ATTN3D_WIRE_QKV_INT8, head_dim),
                            static_cast<cudaStream_t>(stream));
}

int sol_attn3d_exchange_quantize_out_int8(const void* out_rows, const int64_t out_strides[2], int64_t n_rows, int heads,
                                          int head_dim, void* records, sol_attn3d_stream_t stream) {
  const void* const src[3] = {out_rows, nullptr, nullptr};
  const int64_t* const strides[3] = {out_strides, nullptr, nullptr};
  void* const dst[1] = {records};
  return launch_quantize<1>(src, strides, n_rows, heads, head_dim, 1, 0, 0, dst, 0,
                            sol_attn3d_exchange_record_bytes(SOL_ATTN3D_WIRE_OUT_INT8, head_dim),
                            static_cast<cudaStream_t>(stream));
}

extern "C++" {
namespace {
template <int NW>
int launch_dequantize(const void* records, void* out, int64_t n_rows, int heads, int head_dim, size_t rec_bytes,
                      cudaStream_t st) {
  if (n_rows < 0 || heads < 1 || (head_dim != 64 && head_dim != 128)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (n_rows == 0) return SOL_ATTN3D_OK;
  if (records == nullptr || out == nullptr || records == out || !aligned16(records) || !aligned16(out))
    return SOL_ATTN3D_ERR_INVALID_ARG;
  const long long items = n_rows * (long long)heads * NW * (head_dim / 32);          // one thread per group of 32 values
  const unsigned blocks = (unsigned)std::max<long long>(1, std::min<long long>((items + 255) / 256, 148ll * 16));
  sol::dequantize_records_kernel<NW><<<blocks, 256, 0, st>>>(static_cast<const uint8_t*>(records),
                                                              static_cast<__nv_bfloat16*>(out), n_rows, heads, head_dim,
                                                              (int)rec_bytes);
  return cudaGetLastError() == cudaSuccess ? SOL_ATTN3D_OK : SOL_ATTN3D_ERR_CUDA;
}
}  // namespace
}  // extern "C++"

int sol_attn3d_exchange_unpack_qkv_int8(const void* records, void* qkv, int64_t n_rows, int heads, int head_dim,
                                        sol_attn3d_stream_t stream) {
  return launch_dequantize<3>(records, qkv, n_rows, heads, head_dim,
                              sol_attn3d_exchange_record_bytes(SOL_ATTN3D_WIRE_QKV_INT8, head_dim),
                              static_cast<cudaStream_t>(stream));
}

int sol_attn3d_exchange_dequantize_out_int8(const void* records, void* out_rows, int64_t n_rows, int heads, int head_dim,
                                            sol_attn3d_stream_t stream) {
  return launch_dequantize<1>(records, out_rows, n_rows, heads, head_dim,
                              sol_attn3d_exchange_record_bytes(SOL_ATTN3D_WIRE_OUT_INT8, head_dim),
                              static_cast<cudaStream_t>(stream));
}

size_t sol_attn3d_sparse_workspace_bytes(sol_attn3d_plan_t p) { return p ? p->sp_bytes : 0; }

int sol_attn3d_forward_sparse(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out,
                              const uint8_t* key_mask, float tau, void* sparse_ws, size_t sparse_ws_bytes,
                              sol_attn3d_stream_t stream) {
  if (p == nullptr || !(tau == tau)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (sparse_ws == nullptr || sparse_ws_bytes < p->sp_bytes || (reinterpret_cast<uintptr_t>(sparse_ws) % kAlign) != 0)
    return SOL_ATTN3D_ERR_NO_WORKSPACE;
  FwdOpts o;
  o.sparse_ws = static_cast<unsigned char*>(sparse_ws);
  o.tau = tau;
  return forward_impl(p, q, k, v, out, key_mask, stream, o);
}

int sol_attn3d_sparse_stats(sol_attn3d_plan_t p, const void* sparse_ws, long long* selected_tiles, long long* all_tiles) {
  if (p == nullptr || sparse_ws == nullptr || selected_tiles == nullptr || all_tiles == nullptr)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  unsigned long long h[2] = {0, 0};
  const cudaError_t e = cudaMemcpy(h, static_cast<const unsigned char*>(sparse_ws) + p->sp_off_stats, sizeof(h),
                                   cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(p, e);
  *selected_tiles = (long long)h[0];
  *all_tiles = (long long)h[1];
  return SOL_ATTN3D_OK;
}

int sol_attn3d_sparse_selection(sol_attn3d_plan_t p, const void* sparse_ws, int seq, int head, int query_block,
                                int* kv_blocks, int capacity, int* count) {
  if (p == nullptr || sparse_ws == nullptr || count == nullptr || seq < 0 || seq >= p->n_seqs || head < 0 ||
      head >= p->heads || query_block < 0 || (kv_blocks == nullptr && capacity > 0))
    return SOL_ATTN3D_ERR_INVALID_ARG;
  const SeqDev* sq = nullptr;
  for (const SeqDev& c : p->sched)
    if (c.seq_id == seq) sq = &c;
  if (sq == nullptr || query_block >= sq->n_qpairs) return SOL_ATTN3D_ERR_INVALID_ARG;
  const long long local = (long long)head * sq->n_qpairs + query_block;
  const unsigned char* base = static_cast<const unsigned char*>(sparse_ws);
  int n = 0;
  cudaError_t e = cudaMemcpy(&n, base + p->sp_off_count + (size_t)(sq->work_start + local) * sizeof(int), sizeof(int),
                             cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(p, e);
  *count = n;
  const int take = std::min(n, capacity);
  if (take > 0) {
    e = cudaMemcpy(kv_blocks, base + p->sp_off_list + (size_t)(sq->sparse_list_start + local * sq->n_ktiles) * sizeof(int),
                   (size_t)take * sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(p, e);
  }
  return SOL_ATTN3D_OK;
}

int sol_attn3d_qknorm_rope(sol_attn3d_plan_t p, const void* q, const void* k, const float* q_gain, const float* k_gain,
                           float eps, void* q_out, void* k_out, sol_attn3d_stream_t stream) {
  if (p == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  if ((q == nullptr) != (q_out == nullptr) || (k == nullptr) != (k_out == nullptr)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (q == nullptr && k == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if ((q != nullptr && q_gain == nullptr) || (k != nullptr && k_gain == nullptr) || !(eps >= 0.f))
    return SOL_ATTN3D_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(q_out) || !aligned16(k_out)) return SOL_ATTN3D_ERR_INVALID_ARG;
  p->launches = 0;
  return launch_rope(p, p->ws, q, k, q_out, k_out, q_gain, k_gain, eps, static_cast<cudaStream_t>(stream));
}

namespace {
int forward_impl(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out, const uint8_t* key_mask,
                 sol_attn3d_stream_t stream, const FwdOpts& o) {
  if (p == nullptr || v == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (o.qkv_records == nullptr && (q == nullptr || k == nullptr)) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o.qkv_records)) return SOL_ATTN3D_ERR_INVALID_ARG;
  sol::OutSink sink{};
  sink.fmt = o.out_fmt;
  long long o_tok_stride = p->so.tok, o_head_stride = p->so.head;
  // block-INT8 records: dense [token][head][record], strides in bytes (the plan's output strides describe bf16 rows)
  const long long rec_bytes = (long long)sol_attn3d_exchange_record_bytes(SOL_ATTN3D_WIRE_OUT_INT8, p->head_dim);
  if (o.out_fmt == sol::kOutInt8) { o_tok_stride = (long long)p->heads * rec_bytes; o_head_stride = rec_bytes; }
  if (o.n_dst > 0) {
    // scatter: destination g owns flat tokens [tok_begin[g], tok_begin[g+1]) as rows [n_g][dst_heads][head_dim]
    if (o.n_dst > sol::kMaxOutDst || o.dst == nullptr || o.tok_begin == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
    if (o.head_offset < 0 || o.dst_heads < o.head_offset + p->heads) return SOL_ATTN3D_ERR_INVALID_ARG;
    if (o.tok_begin[0] != 0 || o.tok_begin[o.n_dst] != p->total_tokens) return SOL_ATTN3D_ERR_INVALID_ARG;
    // bytes of one head's slot in a destination row
    const size_t slot = o.out_fmt == sol::kOutInt8 ? (size_t)rec_bytes : (size_t)p->head_dim * (o.out_fmt == sol::kOutE4M3 ? 1 : 2);
    for (int g = 0; g < o.n_dst; ++g) {
      if (o.tok_begin[g + 1] < o.tok_begin[g]) return SOL_ATTN3D_ERR_INVALID_ARG;
      const bool empty = o.tok_begin[g + 1] == o.tok_begin[g];
      if (!empty && (o.dst[g] == nullptr || !aligned16(o.dst[g]))) return SOL_ATTN3D_ERR_INVALID_ARG;
      if (o.dst[g] == q || o.dst[g] == k || o.dst[g] == v) return SOL_ATTN3D_ERR_INVALID_ARG;
      sink.base[g] = static_cast<unsigned char*>(o.dst[g]) + (size_t)o.head_offset * slot;
      sink.tok_begin[g] = o.tok_begin[g];
    }
    sink.tok_begin[o.n_dst] = o.tok_begin[o.n_dst];
    sink.n_dst = o.n_dst;
    o_tok_stride = (long long)o.dst_heads * (o.out_fmt == sol::kOutInt8 ? rec_bytes : p->head_dim);
    o_head_stride = o.out_fmt == sol::kOutInt8 ? rec_bytes : p->head_dim;
  } else {
    if (out == nullptr || !aligned16(out)) return SOL_ATTN3D_ERR_INVALID_ARG;
    if (out == q || out == k || out == v) return SOL_ATTN3D_ERR_INVALID_ARG;
    sink.base[0] = out;
    sink.tok_begin[0] = 0;
    sink.tok_begin[1] = p->total_tokens;
    sink.n_dst = 1;
  }
  const float* q_gain = o.q_gain;
  const float* k_gain = o.k_gain;
  const float eps = o.eps;
  unsigned char* sparse_ws = o.sparse_ws;
  const float tau = o.tau;
  const uint8_t* query_mask = o.query_mask;
  // the plan's bound workspace (tables uploaded, tensor maps of Q~ / K~ cached), or scratch handed in for this call
  const bool own = o.ws == nullptr;
  unsigned char* ws = own ? p->ws : o.ws;
  if (ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  const EncodeTiledFn encode = own ? p->encode : o.encode;
  if (encode == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (!o.keep_launch_count) p->launches = 0;

  const SeqDev* d_seqs = reinterpret_cast<const SeqDev*>(ws + p->off_seqs);
  uint32_t* d_bits = reinterpret_cast<uint32_t*>(ws + p->off_keybits);
  int* d_list = reinterpret_cast<int*>(ws + p->off_list);
  int* d_count = reinterpret_cast<int*>(ws + p->off_count);

  const int head_begin = o.head_begin, head_end = o.head_end > 0 ? o.head_end : p->heads;
  if (head_begin < 0 || head_end > p->heads || head_begin >= head_end) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->prof) {
    p->prof_valid = false;
    if ((e = cudaEventRecord(p->ev[0], st)) != cudaSuccess) return fail_cuda(p, e);
  }
  // (1) validity bits per key tile: rebuilt whenever a mask is given (its contents may have changed) and whenever
  //     the scratch is not the plan's own (nothing is known about what it holds)
  p->prof_bits = false;
  if (!o.skip_keybits && (!own || key_mask != nullptr || p->keybits_state != 1)) {
    p->prof_bits = true;
    sol::keybits_kernel<<<p->n_seqs, 256, 0, st>>>(d_seqs, key_mask, d_bits, d_list, d_count);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail_cuda(p, e);
    ++p->launches;
    if (own) p->keybits_state = key_mask ? 2 : 1;
  }
  if (o.bits_done != nullptr && (e = cudaEventRecord(o.bits_done, st)) != cudaSuccess) return fail_cuda(p, e);

  if (p->prof && (e = cudaEventRecord(p->ev[1], st)) != cudaSuccess) return fail_cuda(p, e);

  // (2) rotary prologue: Q~, K~ into the workspace (and V out of the records, when the inputs are records)
  int rc = SOL_ATTN3D_OK;
  const Strides dense_v{(long long)p->heads * p->head_dim, (long long)p->head_dim};
  if (o.qkv_records != nullptr) {
    sol::RopeRecordArgs ra{};
    ra.records = static_cast<const uint8_t*>(o.qkv_records);
    ra.y[0] = reinterpret_cast<__nv_bfloat16*>(ws + p->off_qrot);
    ra.y[1] = reinterpret_cast<__nv_bfloat16*>(ws + p->off_krot);
    ra.y[2] = static_cast<__nv_bfloat16*>(const_cast<void*>(v));
    ra.rec_bytes = (int)sol_attn3d_exchange_record_bytes(SOL_ATTN3D_WIRE_QKV_INT8, p->head_dim);
    ra.seqs = d_seqs;
    ra.n_seqs = p->n_seqs;
    ra.total_tokens = p->total_tokens;
    ra.tables = reinterpret_cast<const float2*>(ws + p->off_tables);
    for (int i = 0; i < 3; ++i) { ra.g.rope[i] = p->rope[i]; ra.g.tab_off[i] = p->tab_off[i]; }
    ra.g.head_dim = p->head_dim;
    ra.g.heads = p->heads;
    ra.status = reinterpret_cast<unsigned int*>(ws + p->off_status);
    // a record takes head_dim / 16 threads; heads per pass: the largest divisor of the head count that fits a block, so
    // that every thread has the same number of heads (two per batch); small shards put several tokens in a block
    const int lanes = p->head_dim / 16, cap = 256 / lanes;
    int hpp = 1;
    for (int d = std::min(p->heads, cap); d >= 1; --d)
      if (p->heads % d == 0) { hpp = d; break; }
    const int toks = std::max(1, 256 / (lanes * hpp));
    const long long want = (p->total_tokens + toks - 1) / toks;
    const long long blocks = std::max<long long>(1, std::min<long long>(want, 148ll * 16));
    sol::rope_records_kernel<<<(unsigned)blocks, lanes * hpp * toks, 0, st>>>(ra, hpp);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail_cuda(p, e);
    ++p->launches;
  } else {
    rc = launch_rope(p, ws, q, k, ws + p->off_qrot, ws + p->off_krot, q_gain, k_gain, eps, st, head_begin, head_end);
  }
  if (rc != SOL_ATTN3D_OK) return rc;
  if (p->prof && (e = cudaEventRecord(p->ev[2], st)) != cudaSuccess) return fail_cuda(p, e);

  // (2a) rectangular mode: which query pairs hold a wanted row
  const uint8_t* d_pair_needed = nullptr;
  if (query_mask != nullptr) {
    uint8_t* flags = ws + p->off_pairs;
    sol::pair_needed_kernel<<<p->total_pairs, 32, 0, st>>>(d_seqs, p->n_seqs, query_mask, flags);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail_cuda(p, e);
    ++p->launches;
    d_pair_needed = flags;
  }

  // (2b) block-sparse mode: pooled operands, block logits, selection -> per-CTA key-tile lists
  const int* d_cta_list = nullptr;
  const int* d_cta_count = nullptr;
  if (sparse_ws != nullptr) {
    if ((e = cudaMemsetAsync(sparse_ws + p->sp_off_stats, 0, 256, st)) != cudaSuccess) return fail_cuda(p, e);
    const __nv_bfloat16* q_rot = reinterpret_cast<const __nv_bfloat16*>(ws + p->off_qrot);
    const __nv_bfloat16* k_rot = reinterpret_cast<const __nv_bfloat16*>(ws + p->off_krot);
    float* qbar = reinterpret_cast<float*>(sparse_ws + p->sp_off_qbar);
    float* kbar = reinterpret_cast<float*>(sparse_ws + p->sp_off_kbar);
    int* lists = reinterpret_cast<int*>(sparse_ws + p->sp_off_list);
    int* counts = reinterpret_cast<int*>(sparse_ws + p->sp_off_count);
    unsigned long long* stats = reinterpret_cast<unsigned long long*>(sparse_ws + p->sp_off_stats);
    for (int s = 0; s < p->n_seqs; ++s) {
      const SeqDev& sq = p->sched[(size_t)s];
      sol::pool_blocks_kernel<<<sq.n_qpairs * p->heads, 256, 0, st>>>(q_rot, d_seqs, p->heads, p->head_dim, 256, s,
                                                                             sq.n_qpairs, 0, qbar + p->sp_qbar_seq[(size_t)s]);
      sol::pool_blocks_kernel<<<sq.n_ktiles * p->heads, 256, 0, st>>>(k_rot, d_seqs, p->heads, p->head_dim, 128, s,
                                                                             sq.n_ktiles, 1, kbar + p->sp_kbar_seq[(size_t)s]);
      const size_t smem = (size_t)sol::kSelectRows * ((size_t)p->head_dim + (size_t)sq.n_ktiles) * sizeof(float);
      if (smem > 48 * 1024) return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;      // > ~1400 key tiles (180k tokens) per sequence
      const int groups = (sq.n_qpairs + sol::kSelectRows - 1) / sol::kSelectRows;
      sol::select_blocks_kernel<<<groups * p->heads, 256, smem, st>>>(
          d_seqs, s, p->heads, p->head_dim, tau, qbar + p->sp_qbar_seq[(size_t)s], kbar + p->sp_kbar_seq[(size_t)s],
          reinterpret_cast<const uint4*>(d_bits), lists, counts, stats);
      if ((e = cudaGetLastError()) != cudaSuccess) return fail_cuda(p, e);
      p->launches += 3;
    }
    d_cta_list = lists;
    d_cta_count = counts;
  }

  // (3) attention.  Tensor maps: the plan's cached ones for its own workspace, per-call ones otherwise.
  // CTA pairs (two CTAs share every K / V tile) wherever they apply
  const bool pair = p->pair_mode != 0 && p->head_dim == 128 && sparse_ws == nullptr;
  CUtensorMap tm_q_call, tm_k_call, tm_v_call;
  const CUtensorMap *tm_q = &p->tm_q, *tm_k = pair ? &p->tm_k64 : &p->tm_k, *tm_v = &p->tm_v;
  if (own) {
    const bool v_dense = o.qkv_records != nullptr;
    if (p->v_cached != v || p->v_cached_dense != v_dense) {
      rc = encode_map(encode, p, &p->tm_v, v, v_dense ? dense_v : p->sv);
      if (rc != SOL_ATTN3D_OK) return rc;
      p->v_cached = v;
      p->v_cached_dense = v_dense;
    }
  } else {
    const Strides dense{(long long)p->heads * p->head_dim, (long long)p->head_dim};
    if ((rc = encode_map(encode, p, &tm_q_call, ws + p->off_qrot, dense)) != SOL_ATTN3D_OK) return rc;
    if ((rc = encode_map(encode, p, &tm_k_call, ws + p->off_krot, dense, pair ? 64 : 128)) != SOL_ATTN3D_OK) return rc;
    if ((rc = encode_map(encode, p, &tm_v_call, v, o.qkv_records != nullptr ? dense_v : p->sv)) != SOL_ATTN3D_OK) return rc;
    tm_q = &tm_q_call; tm_k = &tm_k_call; tm_v = &tm_v_call;
  }
  sol::AttnParams ap{};
  ap.seqs = d_seqs;
  ap.n_seqs = p->n_seqs;
  ap.heads = p->heads;
  ap.keybits = reinterpret_cast<const uint4*>(d_bits);
  ap.ktile_list = d_list;
  ap.ktile_count = d_count;
  ap.query_mask = query_mask;
  ap.pair_needed = d_pair_needed;
  ap.cta_list = d_cta_list;
  ap.cta_count = d_cta_count;
  ap.sink = sink;
  ap.o_tok_stride = o_tok_stride;
  ap.o_head_stride = o_head_stride;
  ap.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)p->head_dim));
  ap.status = o.status != nullptr ? o.status : reinterpret_cast<unsigned int*>(ws + p->off_status);
  ap.counters = reinterpret_cast<unsigned int*>(ws + p->off_status + kCountersOffset);
  ap.wait_limit_ns = p->wait_limit_ns;
  ap.v_lbo = p->v_lbo;
  ap.v_sbo = p->v_sbo;
  ap.fault_inject = own ? p->fault_inject : 0u;
  ap.head_begin = head_begin;
  ap.head_end = head_end;
  ap.wave_ctas = o.sm_count > 0 ? o.sm_count : p->sm_count;
  // one sequence: the CTAs of a head range are a contiguous range of work items; several sequences: launch
  // everything and let the CTAs of other heads leave at the door
  // work items: 256-row query blocks for single CTAs, 512-row blocks for pairs
  int units = pair ? p->total_quad_work : p->total_work;
  ap.cta_offset = 0;
  if (p->n_seqs == 1) {
    const int per_head = pair ? (p->sched[0].n_qpairs + 1) / 2 : p->sched[0].n_qpairs;
    ap.cta_offset = head_begin * per_head;
    units = (head_end - head_begin) * per_head;
  }
  if (pair) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)units * 2u, 1, 1);
    cfg.blockDim = dim3(sol::kAttnThreads, 1, 1);
    cfg.dynamicSmemBytes = sol::AttnSmem<128, 2>::kDynBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, sol::attn_fwd_kernel<128, 2>, *tm_q, *tm_k, *tm_v, ap);
    if (e != cudaSuccess) return fail_cuda(p, e);
  } else if (p->head_dim == 128) {
    sol::attn_fwd_kernel<128, 1><<<units, sol::kAttnThreads, sol::AttnSmem<128, 1>::kDynBytes, st>>>(*tm_q, *tm_k, *tm_v, ap);
  } else {
    sol::attn_fwd_kernel<64, 1><<<units, sol::kAttnThreads, sol::AttnSmem<64, 1>::kDynBytes, st>>>(*tm_q, *tm_k, *tm_v, ap);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return fail_cuda(p, e);
  ++p->launches;
  if (p->prof) {
    if ((e = cudaEventRecord(p->ev[3], st)) != cudaSuccess) return fail_cuda(p, e);
    p->prof_valid = true;
  }
  return SOL_ATTN3D_OK;
}
}  // namespace

int sol_attn3d_set_profiling(sol_attn3d_plan_t p, int enable) {
  if (p == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if ((enable != 0) == p->prof) return SOL_ATTN3D_OK;
  if (enable) {
    for (int i = 0; i < 4; ++i) {
      const cudaError_t e = cudaEventCreate(&p->ev[i]);
      if (e != cudaSuccess) {
        for (int j = 0; j < i; ++j) { cudaEventDestroy(p->ev[j]); p->ev[j] = nullptr; }
        return fail_cuda(p, e);
      }
    }
    p->prof = true;
  } else {
    for (int i = 0; i < 4; ++i) { cudaEventDestroy(p->ev[i]); p->ev[i] = nullptr; }
    p->prof = false;
  }
  p->prof_valid = false;
  return SOL_ATTN3D_OK;
}

int sol_attn3d_last_forward_ms(sol_attn3d_plan_t p, float ms[3]) {
  if (p == nullptr || ms == nullptr || !p->prof || !p->prof_valid) return SOL_ATTN3D_ERR_INVALID_ARG;
  cudaError_t e = cudaEventSynchronize(p->ev[3]);
  if (e != cudaSuccess) return fail_cuda(p, e);
  for (int i = 0; i < 3; ++i) {
    ms[i] = 0.f;
    if ((e = cudaEventElapsedTime(&ms[i], p->ev[i], p->ev[i + 1])) != cudaSuccess) return fail_cuda(p, e);
  }
  if (!p->prof_bits) ms[0] = 0.f;
  return SOL_ATTN3D_OK;
}

// ---------------------------------------------------------------------------------------------
// Variant of sol_attn3d_forward for callers that cannot allocate device memory at all.
//
// The scratch that the kernels need (rotated Q and K, rotary tables, sequence table, key-validity
// bits) lives in one array that is part of the library image.  Its size is fixed when the library is
// built; every GPU context that loads the library holds that much memory until the process exits.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = 32u << 20;   // 32 MiB
static __device__ __align__(256) unsigned char sol_attn3d_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
// Device address of the array per device.  The array's name is only a host-side handle in host code;
// the address a kernel can use comes from cudaGetSymbolAddress, asked once per device.
unsigned char* g_static_scratch_addr[kMaxDevices] = {};
int g_static_sm_count[kMaxDevices] = {};
EncodeTiledFn g_static_encode = nullptr;

int static_scratch_for_current_device(sol_attn3d_plan_t p, unsigned char** out, int* sm_count) {
  int dev = 0, n_dev = 0;
  cudaError_t e = cudaGetDeviceCount(&n_dev);
  if (e != cudaSuccess || n_dev == 0) {
    (void)cudaGetLastError();
    return SOL_ATTN3D_ERR_NO_DEVICE;
  }
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return fail_cuda(p, e);
  if (dev < 0 || dev >= kMaxDevices) return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;
  if (g_static_scratch_addr[dev] == nullptr) {
    int major = 0;
    if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess)
      return fail_cuda(p, e);
    if (major != 10) return SOL_ATTN3D_ERR_UNSUPPORTED_ARCH;
    int sms = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return fail_cuda(p, e);
    unsigned char* addr = nullptr;
    if ((e = cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), sol_attn3d_static_scratch)) != cudaSuccess)
      return fail_cuda(p, e);
    if (addr == nullptr || (reinterpret_cast<uintptr_t>(addr) % kAlign) != 0) return SOL_ATTN3D_ERR_NO_WORKSPACE;
    if ((e = raise_shared_memory_limits()) != cudaSuccess) return fail_cuda(p, e);
    if (g_static_encode == nullptr) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
      if (e != cudaSuccess) return fail_cuda(p, e);
      if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return SOL_ATTN3D_ERR_CUDA;   // driver too old for TMA
      g_static_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    g_static_sm_count[dev] = sms;
    g_static_scratch_addr[dev] = addr;
  }
  *sm_count = g_static_sm_count[dev];
  *out = g_static_scratch_addr[dev];
  return SOL_ATTN3D_OK;
}

}  // namespace

int sol_attn3d_forward_noalloc(sol_attn3d_plan_t p, const void* q, const void* k, const void* v, void* out,
                               const uint8_t* key_mask, unsigned int* device_status, sol_attn3d_stream_t stream) {
  if (p == nullptr || q == nullptr || k == nullptr || v == nullptr || out == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(device_status) & 3u) != 0) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws_bytes > kStaticScratchBytes) return SOL_ATTN3D_ERR_SCRATCH_LIMIT;
  unsigned char* ws = nullptr;
  int sm_count = 0;
  const int rc = static_scratch_for_current_device(p, &ws, &sm_count);
  if (rc != SOL_ATTN3D_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;

  // The array still holds whatever the previous call (of any plan) left there.  What this call reads
  // before writing is rewritten here: the status word starts at zero, tables and sequence table are
  // copied in again; Q~, K~ and the key bits are produced by this call's own kernels.
  unsigned int* status = device_status ? device_status : reinterpret_cast<unsigned int*>(ws + p->off_status);
  if ((e = cudaMemsetAsync(status, 0, sizeof(unsigned int), st)) != cudaSuccess) return fail_cuda(p, e);
  if ((e = cudaMemcpyAsync(ws + p->off_tables, p->tables.data(), p->tables.size() * sizeof(float2),
                           cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return fail_cuda(p, e);
  if ((e = cudaMemcpyAsync(ws + p->off_seqs, p->sched.data(), p->sched.size() * sizeof(SeqDev),
                           cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return fail_cuda(p, e);
  // from here on the same code as every other forward, pointed at the built-in array
  FwdOpts o;
  o.ws = ws;
  o.status = status;
  o.encode = g_static_encode;
  o.sm_count = sm_count;
  return forward_impl(p, q, k, v, out, key_mask, stream, o);
}

size_t sol_attn3d_host_staging_bytes(sol_attn3d_plan_t p) {
  if (p == nullptr) return 0;
  const size_t tensor = align_up((size_t)p->total_tokens * p->heads * p->head_dim * 2);
  return 4 * tensor + align_up((size_t)p->total_tokens);
}

int sol_attn3d_forward_host(sol_attn3d_plan_t p, const void* q_host, const void* k_host, const void* v_host,
                            void* out_host, const uint8_t* key_mask_host, void* staging, size_t staging_bytes,
                            int n_groups, sol_attn3d_stream_t stream) {
  if (p == nullptr || q_host == nullptr || k_host == nullptr || v_host == nullptr || out_host == nullptr)
    return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  if (staging == nullptr || staging_bytes < sol_attn3d_host_staging_bytes(p) ||
      (reinterpret_cast<uintptr_t>(staging) % kAlign) != 0)
    return SOL_ATTN3D_ERR_NO_WORKSPACE;
  const long long dense_tok = (long long)p->heads * p->head_dim;
  for (const Strides* s : {&p->sq, &p->sk, &p->sv, &p->so})
    if (s->tok != dense_tok || s->head != p->head_dim) return SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE;   // dense tensors only
  // head-group boundaries: equal groups when the caller names a count; by default a ramp (small first group:
  // its host-to-device copy is exposed; small last group: its device-to-host copy is) with larger groups between
  int bounds[9];
  if (n_groups <= 0 && p->heads >= 16) {
    static const int kRamp[9] = {0, 1, 4, 10, 19, 28, 34, 38, 40};      // group weights 1, 3, 6, 9, 9, 6, 4, 2 (of 40)
    n_groups = 8;
    for (int g = 0; g <= 8; ++g) bounds[g] = (int)(((long long)p->heads * kRamp[g] + 20) / 40);
    for (int g = 1; g <= 8; ++g) bounds[g] = std::max(bounds[g], bounds[g - 1] + 1);
    bounds[8] = p->heads;
  } else {
    if (n_groups <= 0) n_groups = 8;
    n_groups = std::min(std::min(n_groups, 8), p->heads);
    for (int g = 0; g <= n_groups; ++g) bounds[g] = (int)((long long)p->heads * g / n_groups);
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (!p->host_pipe_ready) {
    e = cudaStreamCreateWithFlags(&p->s_h2d, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->s_d2h, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->s_alt, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_start, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_bits, cudaEventDisableTiming);
    for (int g = 0; g < 8 && e == cudaSuccess; ++g) {
      e = cudaEventCreateWithFlags(&p->ev_in[g], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_out[g], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
      release_host_pipe(p);                          // whatever was created goes away again; the next call retries
      return fail_cuda(p, e);
    }
    p->host_pipe_ready = true;
  }
  const size_t tensor = align_up((size_t)p->total_tokens * p->heads * p->head_dim * 2);
  unsigned char* base = static_cast<unsigned char*>(staging);
  unsigned char* dq = base;
  unsigned char* dk = base + tensor;
  unsigned char* dv = base + 2 * tensor;
  unsigned char* dout = base + 3 * tensor;
  uint8_t* dmask = key_mask_host ? base + 4 * tensor : nullptr;
  const size_t pitch = (size_t)dense_tok * 2;

  // everything the caller queued before this call (an earlier forward reading the staging buffers included)
  // comes before the first copy
  if ((e = cudaEventRecord(p->ev_start, st)) != cudaSuccess) return fail_cuda(p, e);
  if ((e = cudaStreamWaitEvent(p->s_h2d, p->ev_start, 0)) != cudaSuccess) return fail_cuda(p, e);
  if ((e = cudaStreamWaitEvent(p->s_d2h, p->ev_start, 0)) != cudaSuccess) return fail_cuda(p, e);
  if (dmask != nullptr &&
      (e = cudaMemcpyAsync(dmask, key_mask_host, (size_t)p->total_tokens, cudaMemcpyHostToDevice, p->s_h2d)) != cudaSuccess)
    return fail_cuda(p, e);
  const bool was_prof = p->prof;
  p->prof = false;                                   // per-kernel events describe one launch set, not a pipeline
  int rc = SOL_ATTN3D_OK;
  for (int g = 0; g < n_groups && rc == SOL_ATTN3D_OK; ++g) {
    const int h0 = bounds[g], h1 = bounds[g + 1];
    const size_t off = (size_t)h0 * p->head_dim * 2, width = (size_t)(h1 - h0) * p->head_dim * 2;
    // K and V first: the rotary producer and the attention of this group need all three
    const void* srcs[3] = {k_host, v_host, q_host};
    unsigned char* dsts[3] = {dk, dv, dq};
    for (int w = 0; w < 3; ++w)
      if ((e = cudaMemcpy2DAsync(dsts[w] + off, pitch, static_cast<const unsigned char*>(srcs[w]) + off, pitch, width,
                                 (size_t)p->total_tokens, cudaMemcpyHostToDevice, p->s_h2d)) != cudaSuccess)
        return fail_cuda(p, e);
    if ((e = cudaEventRecord(p->ev_in[g], p->s_h2d)) != cudaSuccess) return fail_cuda(p, e);
    // Kernels of even groups run on the caller's stream, those of odd groups on an internal one: neighbouring groups may
    // then share the GPU, and the last, partly filled wave of one group's attention no longer leaves SMs idle until
    // the next group's kernels start.  (Different heads: disjoint parts of the workspace and of the output.)
    cudaStream_t sg = (g & 1) ? p->s_alt : st;
    if (g == 1) {
      // the internal stream joins after everything the caller queued before this call, and after group 0's launch set
      // has got far enough for the key-validity bits (built or kept by group 0) to be in place
      if ((e = cudaStreamWaitEvent(p->s_alt, p->ev_bits, 0)) != cudaSuccess) return fail_cuda(p, e);
    }
    if ((e = cudaStreamWaitEvent(sg, p->ev_in[g], 0)) != cudaSuccess) return fail_cuda(p, e);
    FwdOpts o;
    o.head_begin = h0;
    o.head_end = h1;
    o.skip_keybits = g > 0;
    o.keep_launch_count = g > 0;
    o.bits_done = g == 0 ? p->ev_bits : nullptr;
    rc = forward_impl(p, dq, dk, dv, dout, dmask, static_cast<sol_attn3d_stream_t>(sg), o);
    if (rc != SOL_ATTN3D_OK) break;
    if ((e = cudaEventRecord(p->ev_out[g], sg)) != cudaSuccess) return fail_cuda(p, e);
    if ((e = cudaStreamWaitEvent(p->s_d2h, p->ev_out[g], 0)) != cudaSuccess) return fail_cuda(p, e);
    if ((e = cudaMemcpy2DAsync(static_cast<unsigned char*>(out_host) + off, pitch, dout + off, pitch, width,
                               (size_t)p->total_tokens, cudaMemcpyDeviceToHost, p->s_d2h)) != cudaSuccess)
      return fail_cuda(p, e);
  }
  p->prof = was_prof;
  if (rc != SOL_ATTN3D_OK) return rc;
  // the caller's stream continues only when the last rows have reached the host
  if ((e = cudaEventRecord(p->ev_done, p->s_d2h)) != cudaSuccess) return fail_cuda(p, e);
  if ((e = cudaStreamWaitEvent(st, p->ev_done, 0)) != cudaSuccess) return fail_cuda(p, e);
  return SOL_ATTN3D_OK;
}

int sol_attn3d_status(sol_attn3d_plan_t p) {
  if (p == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  unsigned int w = 0;
  const cudaError_t e = cudaMemcpy(&w, p->ws + p->off_status, sizeof(w), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(p, e);
  if (w == 0) return SOL_ATTN3D_OK;
  return (w & 0xffu) == sol::kStatusAssert ? SOL_ATTN3D_ERR_DEVICE_ASSERT : SOL_ATTN3D_ERR_DEVICE_TIMEOUT;
}

int sol_attn3d_status_word(sol_attn3d_plan_t p, unsigned int* word) {
  if (p == nullptr || word == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  const cudaError_t e = cudaMemcpy(word, p->ws + p->off_status, sizeof(*word), cudaMemcpyDeviceToHost);
  return e == cudaSuccess ? SOL_ATTN3D_OK : fail_cuda(p, e);
}

int sol_attn3d_debug_build(void) { return SOL_ATTN3D_DEBUG; }

int sol_attn3d_last_launch_count(sol_attn3d_plan_t p) { return p == nullptr ? SOL_ATTN3D_ERR_INVALID_ARG : p->launches; }

int sol_attn3d_softmax_rescale_count(sol_attn3d_plan_t p, unsigned long long* count) {
  if (p == nullptr || count == nullptr) return SOL_ATTN3D_ERR_INVALID_ARG;
  if (p->ws == nullptr) return SOL_ATTN3D_ERR_NO_WORKSPACE;
  unsigned int w = 0;
  const cudaError_t e = cudaMemcpy(&w, p->ws + p->off_status + kCountersOffset, sizeof(w), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(p, e);
  *count = w;
  return SOL_ATTN3D_OK;
}

int sol_attn3d_last_cuda_error(sol_attn3d_plan_t p) { return p ? p->last_cuda : 0; }

const char* sol_attn3d_strerror(int code) {
  switch (code) {
    case SOL_ATTN3D_OK: return "ok";
    case SOL_ATTN3D_ERR_INVALID_ARG: return "invalid argument";
    case SOL_ATTN3D_ERR_UNSUPPORTED_SHAPE: return "unsupported shape or stride";
    case SOL_ATTN3D_ERR_NO_WORKSPACE: return "workspace missing, too small or misaligned";
    case SOL_ATTN3D_ERR_NO_DEVICE: return "no CUDA device";
    case SOL_ATTN3D_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    case SOL_ATTN3D_ERR_CUDA: return "CUDA call failed";
    case SOL_ATTN3D_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case SOL_ATTN3D_ERR_NO_MEMORY: return "out of host memory";
    case SOL_ATTN3D_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the built-in 32 MiB array holds";
    case SOL_ATTN3D_ERR_DEVICE_ASSERT: return "a device-side index check of the debug build failed";
    default: return "unknown error";
  }
}

int sol_attn3d_destroy(sol_attn3d_plan_t p) {
  if (p != nullptr && p->prof) (void)sol_attn3d_set_profiling(p, 0);
  if (p != nullptr) release_host_pipe(p);
  delete p;
  return SOL_ATTN3D_OK;
}


}  // extern "C"
