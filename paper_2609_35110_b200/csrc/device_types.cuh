// Plain structs shared between the host-side plan and the kernels.
#pragma once
#include <stdint.h>

namespace sol {

// One packed sequence as the kernels see it.  The array is in SCHEDULE order (longest first).
struct SeqDev {
  long long tok_start;  // first token of the sequence in the packed tensors
  int n_tokens;         // text_len + T*H*W
  int text_len;
  int T, H, W;
  int n_qpairs;         // ceil(n_tokens / 256): one CTA handles two 128-row query tiles
  int n_ktiles;         // ceil(n_tokens / 128)
  int work_start;       // first CTA index of this sequence (CTAs: head-major, query pair fastest)
  int ktile_start;      // offset of this sequence in keybits / ktile_list
  int seq_id;           // index in the caller's order
  int pair_start;       // index of this sequence's first query pair in per-pair arrays
  int quad_work_start;  // first work item of this sequence when CTA pairs serve 512-row query blocks (head-major)
  long long sparse_list_start;  // block-sparse mode: offset of this sequence's per-CTA key-tile lists
};

// Rotary tables: for axis a, entry [tab_off[a] + pos * (rope[a]/2) + j] = (cos, sin)(pos * theta^(-2j/rope[a])).
struct RopeGeom {
  int rope[3];
  int tab_off[3];
  int head_dim;
  int heads;
};

// Where the output rows go.  Destination g receives the rows of flat tokens [tok_begin[g], tok_begin[g+1]);
// base[g] addresses row tok_begin[g] (head 0 of this launch) in that destination, which may be this GPU's
// memory or a peer's mapped into this process.  Plain forward: one destination starting at token 0.
constexpr int kMaxOutDst = 8;
enum : int { kOutBf16 = 0, kOutE4M3 = 1, kOutInt8 = 2 };
struct OutSink {
  void* base[kMaxOutDst];
  long long tok_begin[kMaxOutDst + 1];
  int n_dst;
  int fmt;                  // kOutBf16: 2-byte elements; kOutE4M3: one raw E4M3 byte per element (unit scale);
                            // kOutInt8: one block-INT8 record per (token, head), strides counted in bytes
};

struct AttnParams {
  const SeqDev* seqs;
  int n_seqs;
  int heads;
  int head_begin, head_end; // this launch serves heads [head_begin, head_end) (all heads: 0, heads)
  int cta_offset;           // work item of CTA 0 of this launch (a head range of one sequence is a contiguous range)
  int wave_ctas;            // CTAs that run at the same time (one per SM): the key direction alternates per wave
  const uint4* keybits;     // [ktile] 128 validity bits (bit b of word w = key 32*w + b of the tile)
  const int* ktile_list;    // per sequence, tiles that hold at least one valid key, ascending
  const int* ktile_count;   // per sequence (schedule order)
  const uint8_t* query_mask;   // rectangular mode: uint8 [total_tokens], nonzero = this query row is wanted; else nullptr
  const uint8_t* pair_needed;  // rectangular mode: per (sequence, query pair), nonzero = at least one wanted row
  const int* cta_list;      // block-sparse mode: per CTA, the key tiles it attends (n_ktiles slots each); else nullptr
  const int* cta_count;     // block-sparse mode: per CTA, how many
  OutSink sink;
  long long o_tok_stride, o_head_stride;  // in elements
  float scale_log2;         // log2(e) / sqrt(head_dim)
  unsigned int* status;     // 0 = fine; written once on a wait time-out
  unsigned int* counters;   // [0]: (warp, key tile) events in which the softmax moved its reference maximum
  unsigned long long wait_limit_ns;
  unsigned int fault_inject;  // test hooks: 1 = work item 0 never publishes S of query tile 1 (exercises the bounded
                              // waits); 2 = work item 0 fails a device-side check on purpose (debug build)
  unsigned int v_lbo, v_sbo;  // byte offsets of the V (MN-major) shared-memory descriptor
};

// Status word: low byte = what happened (first event wins), upper bits = detail.
enum : unsigned int {
  kStatusTimeoutProducer = 1,
  kStatusTimeoutMma = 2,
  kStatusTimeoutSoftmax = 3,
  kStatusBadAlignment = 4,
  kStatusAssert = 5,          // debug build only: a device-side index check failed; bits [8,32) = which one
};

// Device-side index checks of the debug build (compile with -DSOL_ATTN3D_DEBUG=1).  A failing check records its
// site in the status word and execution goes on (the checks guard nothing by themselves): nothing traps, the kernel
// returns and the host reads the word.  In the release build the macro expands to nothing.
enum : unsigned int {
  kCheckWorkItem = 1,         // attention: (sequence, head, query block) decoded from the CTA index is in range
  kCheckKeyTile = 2,          // attention: a key tile number taken from a list is inside the sequence
  kCheckTileCount = 3,        // attention: the number of key tiles to walk does not exceed the sequence's
  kCheckOutputRow = 4,        // attention epilogue: the token of a stored row is inside the packed tensor
  kCheckTokenSequence = 5,    // rotary producer: the token lies inside the sequence found for it
  kCheckInjected = 6,         // test hook: the host asked for a failing check
};
#ifndef SOL_ATTN3D_DEBUG
#define SOL_ATTN3D_DEBUG 0
#endif
#if SOL_ATTN3D_DEBUG
#define SOL_DEVICE_CHECK(status_ptr, cond, site)                                                       \
  do {                                                                                                 \
    if (!(cond)) atomicCAS((status_ptr), 0u, sol::kStatusAssert | (static_cast<unsigned int>(site) << 8)); \
  } while (0)
#else
#define SOL_DEVICE_CHECK(status_ptr, cond, site) \
  do {                                           \
  } while (0)
#endif

}  // namespace sol
