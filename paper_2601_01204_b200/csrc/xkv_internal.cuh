// Internal declarations shared by the translation units of libxkv.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "xkv.h"

namespace xkv {

constexpr int kHeadDim = 64;          // d
constexpr int kGroup = 64;            // G: cache slots per key group (Sec. 4.1)
constexpr int kTile = 128;            // key slots per attention tile; segment alignment
constexpr int kWordsPerRow = 8;       // 32-bit words of one packed 4-bit row (64 codes)

// One of the two buffer sets of a cache (physical layout, see xkv.h).
struct BufSet {
  uint8_t* k;        // [H][cap][row_bytes]
  float2* kpar;      // [H][cap/64][64]   (scale, zero)
  uint8_t* v;        // [H][cap][row_bytes]
  float2* vpar;      // [H][cap]          (scale, zero)
  int32_t* origin;   // [cap]
  float* kbar;       // [cap][64] head means of the keys after the first frame (Eq. 4), by rest-local position
  int32_t* kslot;    // [cap] quantise-once mode: parameter-table slot of each token's key group
};

// Phases of the maintenance kernel (bit mask) and its arguments.
constexpr uint32_t kPhAppend = 1u, kPhPool = 2u, kPhKbar = 4u, kPhScore = 8u, kPhSel = 16u, kPhPack = 32u;
constexpr uint32_t kPhKbarNew = 64u;   // quantise-once mode: head means of the frame just quantised
struct MaintArgs {
  uint32_t phases;
  // the frame
  const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v;
  int n;                           // tokens that arrive (one frame, or a chunk of frames)
  int n_q;                         // tokens of the scoring query (the frame; of a chunk, its last frame)
  int64_t ts_q, hs_q, ts_kv, hs_kv;
  // the cache
  int H, cap, max_n, frame, first;
  BufSet cur, oth;                 // current buffer set (source) and the other one (destination)
  int dst_slot;                    // physical slot of the frame's first token in the destination
  int rest_base, r_old, kk, r_new, identity;
  int n_special, pool_g, n_pooled;
  int kbar_on_other, kbar_lo, kbar_hi;   // KBAR phase: buffer set and rest-local range
  __nv_bfloat16* kstage;
  float* qbar; float* qvec; float* scores;
  const float* w_in;               // the pooled query's row mean from the caller (no POOL phase), or null
  float* stats;                    // [4] sum S, sum S^2, k-th largest score, -   of this launch
  float* stats_next;               // the next selecting launch's (cleared by this one)
  int32_t* kept;
  unsigned int* hist;
  unsigned int* run_hi;            // [cap / 64] sure keeps of every 64-token run
  unsigned long long* cand;        // [cap] candidates (key << 32 | ~position)
  unsigned int* cand_count;        // counter of this launch
  unsigned int* cand_count_next;   // counter of the next selecting launch (cleared by this one)
  unsigned int* hist2;             // [256] histogram of the candidates' next 8 key bits
  unsigned int* hist2_next;        // the next selecting launch's (cleared by this one)
  // quantise-once mode: the key parameter table and its bookkeeping
  float2* ktab32;                  // [n_slots][H][64] (scale, zero)
  uint32_t* ktab16;                // [n_slots][H][8][12] fp16 constants for the attention's operand path
  int32_t* ref;                    // [n_slots] cached tokens per slot
  int32_t* ring;                   // [n_slots] free slots, a ring: taken at host-known places, given back by atomics
  unsigned int* push_pos;          // slots given back so far (+ n_slots: the ring starts full)
  uint32_t pop_base;               // slots taken before this launch
  int n_slots;
  int force_plain;
  unsigned int* bar; uint32_t bar_base;
  int* status;
};

// Optional per-launch timing (xkv_profile_enable): one event pair per kernel launch.
struct ProfEvent { int cat; cudaEvent_t a, b; };
struct Profiler {
  bool on = false;
  std::vector<ProfEvent> pending;
  std::vector<cudaEvent_t> pool;
  double ms[XKV_PROF_CATEGORIES] = {0};
  long long launches[XKV_PROF_CATEGORIES] = {0};
};

}  // namespace xkv

// Host-side state of one layer's cache.
struct xkv_cache {
  xkv_params p;
  // geometry
  int cap;            // physical slots per head (multiple of 128)
  int row_bytes;      // 32 (4-bit) or 128 (bf16)
  size_t ws_bytes;
  uint8_t* ws;
  xkv::BufSet buf[2];
  __nv_bfloat16* kstage;   // [H][max_n][64] staged keys of the frame in flight (4-bit mode)
  float* qbar;             // [Np_max][64]
  float* qvec;             // [64]
  float* scores;           // [cap]
  int32_t* kept;           // [cap]
  unsigned int* counters;  // device counters: [0] grid barrier (only grows), [2], [3] candidate counters,
                           // [64..319], [320..575] the two sub-histograms of the selection
  uint32_t bar_base;       // value of the barrier counter when the next maintenance kernel starts
  int sel_parity;          // which candidate counter the next selecting launch uses
  unsigned int* sel_hist;  // [4096] histogram of the top 12 bits of the score keys (self-clearing)
  unsigned int* run_hi;    // [cap / 64]
  unsigned long long* cand;  // [cap]
  // quantise-once mode
  float2* ktab32; uint32_t* ktab16; int32_t* ref; int32_t* ring;
  int n_slots;
  uint32_t pop_base;       // key groups that have taken a table slot so far
  int* status;             // device status word
  float* attn_part;        // split-KV partials of the attention kernel
  size_t attn_part_bytes;
  // stream state (host)
  int frames, T, T_first, rest_base, cur, stage;
  int n_pending, nq_pending, kk_pending, rold_pending, evict_pending, first_pending;
  int last_evicted, last_kept, last_prunable;
  long long launches;
  int force_plain;         // 1: kernels take the plain (conversion-based) arithmetic forms everywhere
  int budget_now;          // the token budget in force (xkv_set_budget), <= p.budget
  int stats_parity;        // which statistics block the last selecting launch wrote (-1: none)
  int tail_mode;           // 1: the stream-step calls attend with the step's K, V unquantised
  int attn_max_blocks;     // test hook: cap on the thread blocks of the tensor-core attention (0: none)
  // head means of the keys after the first frame (Eq. 4; BufSet::kbar), filled by the stream step
  // beside the attention and used by the next step's scoring when the cache has not changed since
  cudaEvent_t kbar_done;
  int kbar_T, kbar_cur, kbar_frames;   // state of the cache the array was computed from (-1: none)
  xkv::Profiler* prof;
};

namespace xkv {

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

#ifdef __CUDACC__
// Constants of the attention's fp16 dequantisation for one (scale, zero-point) of Eq. 8: a pair
// of codes is formed as fma(biased_code - zo, s, c), the code carrying a bias of 1024 or 64
// (its fp16 bit pattern is built by OR-ing the nibble into the mantissa of 1024 resp. 64).
//   zo = bias + z, c = 0     when fp16 holds bias + z exactly (|bias + z| <= 2048, z an integer):
//                            the difference is q - z exactly and the product is rounded once;
//   zo = bias,     c = -s z  otherwise (c formed in fp32): s q + c, valid for any zero-point.
__device__ __forceinline__ void dequant_consts(float s, float z, float& zo_1024, float& zo_64, float& c) {
  const bool exact = fabsf(1024.f + z) <= 2048.f && fabsf(64.f + z) <= 2048.f;
  zo_1024 = exact ? 1024.f + z : 1024.f;
  zo_64 = exact ? 64.f + z : 64.f;
  c = exact ? 0.f : -s * z;
}
#endif

// Brackets one kernel launch with events when profiling is on; counts the launch.
struct LaunchScope {
  xkv_cache* c; int cat; cudaStream_t st; cudaEvent_t a = nullptr, b = nullptr;
  LaunchScope(xkv_cache* c_, int cat_, cudaStream_t st_) : c(c_), cat(cat_), st(st_) {
    c->launches++;
    Profiler* p = c->prof;
    if (p && p->on) {
      auto get = [&]() { cudaEvent_t e = nullptr;
        if (!p->pool.empty()) { e = p->pool.back(); p->pool.pop_back(); } else cudaEventCreate(&e);
        return e; };
      a = get(); b = get();
      cudaEventRecord(a, st);
    }
  }
  ~LaunchScope() {
    if (a) { cudaEventRecord(b, st); c->prof->pending.push_back({cat, a, b}); }
  }
};

// ---- launchers implemented in the kernel translation units -------------------
// All return cudaError_t of the launch (cudaGetLastError) and count launches.

// The maintenance kernel with the phases in a.phases (cooperative when it has a grid barrier).
// Fills in the barrier and status fields of `a`; everything else is the caller's.
cudaError_t launch_maint(xkv_cache* c, MaintArgs& a, int prof_cat, cudaStream_t st);
// Quantise-once mode: fills the ring of free parameter-table slots (after the workspace was zeroed).
cudaError_t launch_once_init(xkv_cache* c, cudaStream_t st);
// kv_quant_pack of a 4-bit cache: key regroup + re-quantisation fused with the survivor gather.
cudaError_t launch_regroup(xkv_cache* c, const MaintArgs& a, cudaStream_t st);
cudaError_t launch_attn_simple(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                               float scale, cudaStream_t st);
// Returns cudaErrorNotSupported when the tensor-core kernel cannot take the call.
// prefix > 0: only the first `prefix` tokens of the cache (logical order) are visible to these queries
// (frame-causal attention inside a chunk of frames); 0: all of them.
cudaError_t launch_attn_tc(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                           float scale, cudaStream_t st, int prefix = 0);
// Same kernel with the newest frame's keys and values taken unquantised from k_t, v_t (the tensors
// given to kv_append, same strides as q).
cudaError_t launch_attn_tc_tail(xkv_cache* c, const void* q, const void* k_t, const void* v_t, void* out, int n,
                                int64_t ts, int64_t hs, float scale, cudaStream_t st);
// Same kernel, split-KV partials in the library's fixed device array; cudaErrorMemoryAllocation
// when the launch would need more than XKV_STATIC_SCRATCH_BYTES.
cudaError_t launch_attn_tc_static(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                                  float scale, cudaStream_t st);
size_t attn_tc_scratch_bytes(const xkv_params* p);
// One small block running the attention kernel's bounded wait on a barrier nobody completes.
cudaError_t launch_timeout_probe(xkv_cache* c, cudaStream_t st);

}  // namespace xkv
