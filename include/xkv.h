/*
 * xkv - compressed KV cache for streaming frame-causal attention on one GPU.
 *
 * C ABI of the library.  One `xkv_cache` holds the key/value cache of ONE
 * global-attention layer under joint pruning and quantisation (Sec. 3.2-3.3 of
 * the paper).  Per incoming frame the caller runs, in this order,
 *
 *     kv_append -> kv_score_evict -> kv_quant_pack -> attn_packed_causal
 *
 * or xkv_stream_step, which does the same for a stack of layers.
 *
 * Conventions
 *   - Pointers named q, k, v, out and dev_workspace are DEVICE pointers; every
 *     other pointer is a HOST pointer.  All device pointers must be 16-byte
 *     aligned.  Q/K/V/out are bf16 (16-bit, truncated-fp32 format).
 *   - A frame tensor is addressed as  base[head*head_stride + token*tok_stride + c],
 *     c = 0..head_dim-1 contiguous, strides in ELEMENTS and multiples of 8.
 *     [H][n][d] is (tok_stride=d, head_stride=n*d); [n][H*d] is (H*d, d).
 *   - The first n_special tokens of a frame are its camera and register tokens,
 *     the rest its patch tokens in raster order (Sec. 3.1).
 *   - Calls are stream-ordered and never synchronise, allocate device memory or
 *     read device data on the host (exceptions: xkv_debug_export,
 *     xkv_poll_status, xkv_profile_read, xkv_stream_step_host).  All cache lengths are functions
 *     of the frame sizes seen so far and the budget, so they are tracked on the
 *     host.
 *   - The caller owns the workspace; the library never frees it.  Memory use of
 *     a cache is constant for its lifetime.
 *   - Every function returns XKV_OK (0) or a negative xkv_status.  Nothing
 *     throws, aborts or traps.  A cache is not thread-safe; different caches may
 *     be driven from different threads/streams.
 */
#ifndef XKV_H_
#define XKV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define XKV_API __attribute__((visibility("default")))
#else
#define XKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xkv_cache xkv_cache;          /* opaque, host-side handle of one layer's cache */
typedef void* xkv_stream;                    /* a cudaStream_t, passed as a plain pointer     */

typedef enum {
  XKV_OK            =  0,
  XKV_E_INVALID     = -1,   /* bad argument (null, misaligned, out of range)          */
  XKV_E_STATE       = -2,   /* call out of order for this cache                        */
  XKV_E_NOMEM       = -3,   /* workspace too small / host allocation failed            */
  XKV_E_UNSUPPORTED = -4,   /* parameter combination not implemented                   */
  XKV_E_CUDA        = -5,   /* a CUDA runtime/driver call failed                       */
  XKV_E_TIMEOUT     = -6,   /* a bounded device-side wait ran out (see xkv_poll_status)*/
  XKV_E_LIMIT       = -7,   /* the call needs more than a fixed built-in limit allows   */
  XKV_E_RANGE       = -8    /* a value left the range of the 16-bit tensor-core operands */
                            /* (see attn_packed_causal and xkv_poll_status)             */
} xkv_status;

/* Method parameters.  Defaults of the paper: n_special = 5 (1 camera + 4
 * register tokens, Sec. 3.1), pool_g = 16, quant_group = 64, kv_bits = 4
 * (Sec. 4.1).  kv_bits = 16 keeps bf16 values (pruning only).  kv_bits = 8 applies the same
 * Eq. 7-9 with 256 levels (the paper evaluates INT4 only); it is built for XKV_KEYS_ONCE. */
typedef struct {
  int32_t n_heads;           /* H, 1..64                                                 */
  int32_t head_dim;          /* d, only 64                                               */
  int32_t n_special;         /* special tokens at the head of each frame, >= 0           */
  int32_t pool_g;            /* g of GroupAvg (Eq. 2), >= 1                              */
  int32_t quant_group;       /* G, cache positions per key group, only 64                */
  int32_t kv_bits;           /* b: 4, 16, or 8 (XKV_KEYS_ONCE only)                      */
  int32_t budget;            /* L_max, the token budget (Sec. 3.2), >= 1                 */
  int32_t max_frame_tokens;  /* largest n any frame will have, 1..65535                  */
  int32_t key_mode;          /* XKV_KEYS_REGROUP (0) or XKV_KEYS_ONCE (1), see below; 4-bit only */
  int32_t key_table_slots;   /* XKV_KEYS_ONCE: key groups the parameter table can hold;  */
                             /* 0 = as many as the cache has token slots (never runs out)*/
} xkv_params;

/* How the per-channel key groups of Eq. 9 (64 tokens each, Sec. 4.1) live with eviction.
 *   XKV_KEYS_REGROUP  a group is a run of 64 cache positions.  kv_quant_pack regroups the keys
 *                     after the first frame every step and re-quantises every group whose
 *                     members changed (Sec. 3.3: "the final KV cache" is quantised).
 *   XKV_KEYS_ONCE     a group is a run of 64 tokens of one frame, quantised when the frame
 *                     arrives and never again (the quantiser the paper names, Sec. 4.1, works
 *                     this way).  A survivor keeps its codes and refers to its group's scales
 *                     and zero-points in a parameter table; a group's entry is given back when
 *                     its last token is evicted.  No re-quantisation error accumulates and
 *                     kv_quant_pack only moves rows.  If the table is sized below the worst case
 *                     (key_table_slots) and runs out, the status word reads XKV_E_LIMIT. */
enum { XKV_KEYS_REGROUP = 0, XKV_KEYS_ONCE = 1 };

/* Host-side counters and geometry; filled without touching the device. */
typedef struct {
  int32_t frames;            /* frames appended so far                                   */
  int32_t T;                 /* tokens in the packed cache                               */
  int32_t T_first;           /* tokens of the first frame                                */
  int32_t rest_base;         /* physical slot where the rest segment starts (128-aligned)*/
  int32_t T_phys;            /* physical slots in use = rest_base + (T - T_first)        */
  int32_t capacity;          /* physical slots per head                                  */
  int32_t cur;               /* which of the two buffer sets is current (0/1)            */
  int32_t last_evicted;      /* tokens evicted by the last kv_score_evict                */
  int32_t last_kept;         /* middle tokens kept by the last kv_score_evict            */
  int32_t last_prunable;     /* size of the middle segment at the last kv_score_evict    */
  int32_t stage;             /* 0 idle, 1 appended, 2 scored, 3 packed                   */
  int32_t n_pending;         /* tokens of the frame in flight                            */
  int64_t launches;          /* kernels launched for this cache so far                   */
  uint64_t workspace_bytes;
  int32_t key_table_slots;   /* XKV_KEYS_ONCE: slots of the key parameter table, else 0  */
  int32_t budget;            /* the token budget in force (xkv_set_budget)               */
} xkv_info;

/* Sub-buffers that xkv_debug_export can copy out (physical layout, current
 * buffer set).  Slot p of head h: logical token j lives at p = j for
 * j < T_first and at p = rest_base + (j - T_first) otherwise.
 *   K_CODES / V_CODES : kv_bits = 4 : uint8 [H][capacity][d/2]; the 8 codes of channels
 *                       8w..8w+7 form the little-endian 32-bit word
 *                       c0 | c2<<4 | c4<<8 | c6<<12 | c1<<16 | c3<<20 | c5<<24 | c7<<28
 *                       kv_bits = 8 : uint8 [H][capacity][d]; the 4 codes of channels 4w..4w+3 form the
 *                       little-endian word c0 | c2<<8 | c1<<16 | c3<<24
 *                       kv_bits = 16: bf16 [H][capacity][d]
 *   K_PARAMS          : float2 (scale, zero) [H][capacity/64][d], group = 64 slots
 *   V_PARAMS          : float2 (scale, zero) [H][capacity]
 *   ORIGIN            : int32 [capacity], (frame << 16) | token, frame counted from 1
 *   SCORES            : float [last_prunable]  importance scores S of Eq. 6 (last evicting step)
 *   KEPT              : int32 [last_kept]      kept middle positions, ascending (last evicting step)
 *   QVEC              : float [d]              row mean of the pooled query (last evicting step)
 * XKV_KEYS_ONCE only (K_PARAMS is then unused):
 *   K_SLOT            : int32 [capacity]       parameter-table slot of each token's key group
 *   K_TABLE           : float2 (scale, zero) [key_table_slots][H][d]
 *   K_REF             : int32 [key_table_slots] cached tokens that refer to each slot (0 = free)
 */
typedef enum {
  XKV_BUF_K_CODES = 0, XKV_BUF_K_PARAMS = 1, XKV_BUF_V_CODES = 2, XKV_BUF_V_PARAMS = 3,
  XKV_BUF_ORIGIN = 4, XKV_BUF_SCORES = 5, XKV_BUF_KEPT = 6, XKV_BUF_QVEC = 7,
  XKV_BUF_K_SLOT = 8, XKV_BUF_K_TABLE = 9, XKV_BUF_K_REF = 10
} xkv_buffer;

/* ---- set-up ---------------------------------------------------------------- */

/* Bytes of device workspace one cache needs; 0 if the parameters are invalid. */
XKV_API size_t xkv_workspace_bytes(const xkv_params* params);

/* Create a cache on `dev_workspace` (device memory, 256-byte aligned, at least
 * xkv_workspace_bytes(params) bytes, on the current device).  Zero-fills the
 * workspace on `stream`.  *out receives the handle. */
XKV_API int xkv_create(const xkv_params* params, void* dev_workspace, size_t bytes,
               xkv_stream stream, xkv_cache** out);

/* Back to the empty state on the same workspace (stream-ordered zero-fill, which also clears the
 * device status word).  `stream` is made to wait for any kernel that a stream step of this cache
 * still has in flight on the library's own stream; the host does not wait. */
XKV_API int xkv_reset(xkv_cache* cache, xkv_stream stream);

/* Free the host handle.  The workspace stays with the caller. */
XKV_API int xkv_destroy(xkv_cache* cache);

/* ---- the per-frame calls --------------------------------------------------- */

/* Step 1 (Sec. 3.1, the text after Eq. 1: the new frame joins the cache).  Takes frame
 * t's keys and values, n tokens, into the cache: values are quantised per token
 * (Eq. 7-9) straight into their final slot; keys are staged until kv_quant_pack.
 * k and v may be reused once the stream has passed this call.  At t = 1 this
 * fixes T_first = n.  Errors: XKV_E_STATE unless the cache is idle;
 * XKV_E_INVALID for n < 1, n > max_frame_tokens, bad strides or pointers. */
XKV_API int kv_append(xkv_cache* cache, const void* k, const void* v, int32_t n,
              int64_t tok_stride, int64_t head_stride, xkv_stream stream);

/* Steps 2-3 (Sec. 3.2, Eq. 2-6).  If the cache length T after the append
 * exceeds the budget: pooled query (special tokens kept, patch tokens averaged
 * in groups of g, then averaged over heads), head-averaged dequantised keys of
 * the middle segment, scores S, and the k = max(0, L_max - T_first - n) highest
 * scores kept (ties: lower position wins), in ascending position.  Otherwise a
 * no-op.  q is frame t's query, same n as the append (after a chunk of frames was appended: the
 * query and size of the chunk's last frame, see attn_packed_frame_causal).  Errors: XKV_E_STATE
 * unless kv_append was the previous call; XKV_E_INVALID as above. */
XKV_API int kv_score_evict(xkv_cache* cache, const void* q, int32_t n,
                   int64_t tok_stride, int64_t head_stride, xkv_stream stream);

/* Step 4 (Sec. 3.3, Eq. 7-9).  Builds the final cache = first frame, surviving
 * middle tokens, current frame: survivors' value codes and parameters are
 * gathered; the keys after the first frame are regrouped into runs of 64 and
 * re-quantised per channel (a complete group whose tokens all survive in place
 * is carried over unchanged).  With XKV_KEYS_ONCE the keys were quantised by kv_append and
 * their code rows and group references are gathered like the values.
 * Afterwards T <= max(L_max, T_first + n).
 * Errors: XKV_E_STATE unless kv_score_evict was the previous call. */
XKV_API int kv_quant_pack(xkv_cache* cache, xkv_stream stream);

/* Step 5 (Eq. 1 with the dequantisation of Eq. 10).  out = softmax(q K~^T *
 * softmax_scale) V~ per head over all T cached tokens (all of them belong to
 * frames <= t, so the frame-causal mask hides nothing).  out has the strides of
 * q.  impl: 0 = default (tensor-core kernel), 1 = the simple CUDA-core kernel
 * kept as a cross-check (fp32 throughout).  Errors: XKV_E_STATE unless kv_quant_pack was the
 * previous call (the cache returns to idle); XKV_E_INVALID as above.
 *
 * Operand range of the tensor-core kernel.  A 4-bit cache is multiplied in fp16 with fp32
 * accumulation: q, the dequantised keys and values x~ = s*q_code + (-s*z) (Eq. 10, the constant
 * formed in fp32 per group and channel resp. per token) and the softmax weights are rounded to
 * fp16, i.e. to 11 significant bits, with fp16's floor of 6e-8 on the absolute resolution.  Any
 * integer zero-point and any scale are accepted.  What fp16 cannot hold is a magnitude above
 * 65504: if a query element, a dequantised key or value, or (tail variant) a raw key or value
 * of the newest frame exceeds it, the kernel records XKV_E_RANGE in the cache's status word
 * (xkv_poll_status) and the output of that call is unspecified; impl = 1 has no such limit.
 * A 16-bit cache is multiplied in bf16 and has no range limit.  Keys whose spread within a
 * 64-token group is far below the resolution of a 16-bit number at their magnitude (a large
 * common offset, a tiny range) lose that spread in any 16-bit operand: the result then
 * carries the error of rounding x~ to 11 bits, no more. */
XKV_API int attn_packed_causal(xkv_cache* cache, const void* q, void* out, int32_t n,
                       int64_t tok_stride, int64_t head_stride, float softmax_scale,
                       int32_t impl, xkv_stream stream);

/* Step 5 with Eq. 1 read literally: the frame attends to its own K_t, V_t as they
 * arrived (bf16) and to the packed cache (Eq. 10) for every older token; Sec. 3.3
 * quantises "the final KV cache ... including the current frame", Eq. 1 shows the
 * raw K_t, V_t inside the attention, and this call is the second reading.  k_t,
 * v_t are the device tensors that kv_append took for this frame (n tokens, the
 * strides of q).  The cache is left exactly as attn_packed_causal leaves it: later
 * frames see this frame quantised either way.  A 16-bit cache stores the frame
 * unchanged, so there both calls give the same result.  Always the tensor-core
 * kernel.  Errors and state as attn_packed_causal; XKV_E_INVALID also when n is
 * not the size of the frame appended last. */
XKV_API int attn_packed_causal_tail(xkv_cache* cache, const void* q, const void* k_t, const void* v_t,
                            void* out, int32_t n, int64_t tok_stride, int64_t head_stride,
                            float softmax_scale, xkv_stream stream);

/* attn_packed_causal for callers that must not allocate device memory.
 * (The paper has no counterpart: this is a deployment variant of Step 5 with the
 * same arithmetic and the same kernel.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a host
 * application that forbids allocation after start-up, a plug-in whose host owns
 * the allocator, a process that shares its GPU with a job whose memory pool must
 * not be disturbed - and that therefore cannot grow a buffer for the attention
 * kernel's scratch.  The tensor-core kernel cuts the keys of a head between
 * thread blocks and needs global memory for the partial results (64
 * accumulators plus running max and sum per query row and cut).
 * attn_packed_causal keeps them in the cache workspace; this variant keeps them
 * in a fixed array of XKV_STATIC_SCRATCH_BYTES that is part of the library image
 * and leaves that region of the workspace untouched.  Every GPU on which the
 * library is used holds the array from first use until the process exits.  The
 * call allocates nothing, neither on the device nor through any allocating
 * routine.
 *
 * Rules of use
 *   - Same arguments, state requirements and result as attn_packed_causal with
 *     impl = 0; q and out are still the caller's.
 *   - The need does not grow with the frame or the cache: each thread block
 *     leaves at most two partial slots of 67 584 bytes (two query tiles of 128 rows, 64
 *     accumulators plus running max and sum each), and the kernel runs one block per
 *     multiprocessor.  The array holds XKV_STATIC_SCRATCH_BYTES / 67 584 = 496 slots, enough
 *     for 248 blocks; a GPU with more multiprocessors than that would run 248 blocks (each
 *     item of work cut into fewer, longer pieces: slower, same result).  A B200 has 148.
 *     XKV_E_LIMIT is returned, before anything is enqueued and with the cache left in the
 *     packed state, only if not even one block's slots fit.
 *   - The first call on a device looks up the array's device address (once per
 *     device, with that device current).  Make that first call outside any
 *     stream capture.
 *   - All callers in the process share the one array per GPU, and it keeps
 *     whatever the last call left there.  Nothing in it has to start at zero:
 *     every partial that is read was written by the same call.  Two calls whose
 *     kernels can overlap on one GPU (different streams or threads) race on it:
 *     serialise them. */
#define XKV_STATIC_SCRATCH_BYTES (32u << 20)
XKV_API int attn_packed_causal_static(xkv_cache* cache, const void* q, void* out, int32_t n,
                              int64_t tok_stride, int64_t head_stride, float softmax_scale,
                              xkv_stream stream);

/* A chunk of frames at once (offline sequences arrive many frames at a time; Eq. 1 is frame-causal:
 * a query sees the keys of its own and of earlier frames).  The chunk is one arrival for the cache
 * maintenance of Sec. 3.2 - it plays the part of the current frame: kv_append takes all its tokens
 * (n = their total, frames one after the other along the token axis, at most max_frame_tokens),
 * kv_score_evict takes the query of the chunk's LAST frame (n = that frame's size) and keeps
 * k = max(0, L_max - T_first - total) middle tokens, kv_quant_pack packs - and then this call
 * attends frame-causally: the queries of the chunk's frame f see every cached token that is older
 * than the chunk and the chunk's frames 0..f (the cache keeps arrival order, so that is a prefix
 * of it; one launch of the tensor-core kernel per frame).  q, out: the chunk's tensors,
 * [H][total][d] with the given strides; frame_tokens: HOST array of n_frames sizes that add up to
 * the appended total.  A chunk of one frame is attn_packed_causal.  State and errors as attn_packed_causal. */
XKV_API int attn_packed_frame_causal(xkv_cache* cache, const void* q, void* out, const int32_t* frame_tokens,
                             int32_t n_frames, int64_t tok_stride, int64_t head_stride, float softmax_scale,
                             xkv_stream stream);

/* The four calls above for one chunk, softmax_scale = 1/sqrt(head_dim). */
XKV_API int xkv_prefill_chunk(xkv_cache* cache, const void* q, const void* k, const void* v, void* out,
                      const int32_t* frame_tokens, int32_t n_frames, int64_t tok_stride, int64_t head_stride,
                      xkv_stream stream);

/* Steps 2-3 with the pooled query supplied by the caller.  Eq. 5-6 average the rows of Q-bar K-bar^T,
 * which by linearity is w . K-bar[j] with w the mean of the pooled rows of Eq. 2-3: whoever
 * produces Q (the projection that writes it) can form w on the way (Sec. 3.2 notes that pooling is
 * what keeps the scoring cheap) and hand it over.  w: DEVICE, 64 floats, exactly the value
 * kv_score_evict would compute (fixed-order fp32: per head and pooled row the sequential sum over the
 * row's tokens divided by their number; heads added in order, times 1/H; rows added in order,
 * divided by their number).  n is the frame's token count.  State and errors as kv_score_evict. */
XKV_API int kv_score_evict_w(xkv_cache* cache, const float* w, int32_t n, xkv_stream stream);

/* The token budget L_max in force from the next frame on, 1 <= budget <= the budget the cache was
 * created with (which sized the workspace).  A lower budget makes the next evicting step keep
 * k = max(0, budget - T_first - n) middle tokens by the same rule; raising it again lets the cache
 * grow back.  The paper names per-layer adaptive budgets as future work (Conclusion); this call
 * and xkv_read_score_stats are the mechanism, the policy is the caller's.  Idle cache only. */
XKV_API int xkv_set_budget(xkv_cache* cache, int32_t budget);

/* Statistics of the last evicting step's scores S (Eq. 6), for such a policy.  Synchronises
 * `stream`.  sum and sum_sq are accumulated with floating-point atomics (last digits may differ
 * between runs); threshold is the smallest kept score, exact. */
typedef struct {
  int32_t count;        /* scored (middle) tokens; 0 if no step has evicted since the reset */
  int32_t kept;         /* how many of them were kept                                        */
  float   sum, sum_sq;  /* sum of S and of S^2                                               */
  float   threshold;    /* the k-th largest score                                            */
} xkv_score_stats;
XKV_API int xkv_read_score_stats(const xkv_cache* cache, xkv_score_stats* out, xkv_stream stream);

/* Chooses the attention that xkv_stream_step and xkv_stream_step_host run for this
 * cache: 0 (default) attn_packed_causal, 1 attn_packed_causal_tail with the K, V
 * of the step.  The per-call entry points are not affected. */
XKV_API int xkv_set_unquantised_tail(xkv_cache* cache, int32_t on);

/* One frame through a stack of layers: for each layer in order, the four calls
 * above with softmax_scale = 1/sqrt(head_dim).  q, k, v, out are HOST arrays of
 * n_layers DEVICE pointers.  Stops at the first error and returns it; the layer that failed
 * may then be left between two of its four calls, and the only way on is xkv_reset.
 * Within a layer kv_append runs on a stream of the library's own (created on
 * first use, one per device) beside kv_score_evict, which does not depend on it;
 * both are ordered after everything already in `stream` and before the layer's
 * kv_quant_pack, and a layer starts only after the previous layer's attention.
 * After kv_quant_pack the step also computes, on that stream and beside the
 * attention, the head means of the cached keys (Eq. 4) into the cache's workspace;
 * the next frame's scoring of the same cache starts from them (same bits as
 * kv_score_evict computes).  `stream` waits for these kernels at the end of the call.
 * The library's stream and its events are shared by every cache on the device:
 * call the stream-step functions of one device from one host thread at a time. */
XKV_API int xkv_stream_step(xkv_cache* const* layers, int32_t n_layers,
                    const void* const* q, const void* const* k, const void* const* v,
                    void* const* out, int32_t n, int64_t tok_stride, int64_t head_stride,
                    xkv_stream stream);

/* The same step for callers whose tensors live in HOST memory (pinned memory
 * gives asynchronous copies).  q, k, v, out are HOST arrays of n_layers HOST
 * pointers to bf16 [H][n][d] tensors; dev_staging is device scratch of at least
 * xkv_stream_step_host_bytes(layers[0] params, n) bytes.  The layers run on
 * `stream`; the inputs of the next layer are copied on two further streams (two copy
 * engines) while a layer runs and the outputs go back on a fourth (all created by the
 * library on first use, one set per device), so that copies overlap the kernels.  All
 * of them are synchronised before the call returns.  Not for use inside a stream capture. */
XKV_API size_t xkv_stream_step_host_bytes(const xkv_params* params, int32_t n);
XKV_API int xkv_stream_step_host(xkv_cache* const* layers, int32_t n_layers,
                         const void* const* q, const void* const* k, const void* const* v,
                         void* const* out, int32_t n, void* dev_staging, size_t staging_bytes,
                         xkv_stream stream);

/* ---- introspection ---------------------------------------------------------- */

XKV_API int xkv_get_info(const xkv_cache* cache, xkv_info* info);

/* Tests only: synchronises `stream`, then copies up to `bytes` bytes of one
 * sub-buffer of the current buffer set to host_dst.  Returns the number of bytes
 * copied (>= 0) or a negative xkv_status. */
XKV_API int64_t xkv_debug_export(const xkv_cache* cache, int32_t which, void* host_dst, size_t bytes,
                         xkv_stream stream);

/* Tests and benchmarks only: puts an idle cache that holds at least one frame back
 * into the packed state, so that attn_packed_causal can run again on the same
 * cache contents (with the same or other queries).  XKV_E_STATE otherwise. */
XKV_API int xkv_debug_rewind_attention(xkv_cache* cache);

/* Synchronises `stream` and returns the device status word of the cache: XKV_OK,
 * XKV_E_TIMEOUT if a bounded wait inside a kernel ran out (the kernel still ended in order: it
 * drained its copies and freed its tensor memory; results of that call are void), or
 * XKV_E_RANGE (see attn_packed_causal).  The word is sticky until xkv_reset. */
XKV_API int xkv_poll_status(const xkv_cache* cache, xkv_stream stream);

XKV_API const char* xkv_strerror(int status);

/* ---- test hooks (per cache; no environment variables, no process-wide switches) ---------- */

/* Tests only.  The maintenance kernels evaluate Eq. 7 and Eq. 10 in conversion-free forms when
 * the zero-points and scaled values of a group are small enough, and in the plain forms
 * otherwise; on = 1 makes every kernel of this cache take the plain forms everywhere. */
XKV_API int xkv_debug_force_plain(xkv_cache* cache, int32_t on);

/* Tests only.  Caps the number of thread blocks of the tensor-core attention of this cache
 * (0 = no cap: one block per multiprocessor).  With fewer blocks every item of work is cut into
 * fewer, longer pieces and a block may cover several items; the result does not change. */
XKV_API int xkv_debug_limit_attention_blocks(xkv_cache* cache, int32_t max_blocks);

/* Tests and benchmarks only.  Recomputes, on `stream`, the head means of the keys after the first
 * frame (Eq. 4) that the stream step keeps for the next frame's scoring, from the cache as it
 * stands (idle cache; same values, nothing else changes).  Lets a benchmark time that kernel by
 * itself: inside the stream step it runs beside the attention. */
XKV_API int xkv_debug_head_means(xkv_cache* cache, xkv_stream stream);

/* Tests only.  Launches one small thread block that waits, with the attention kernel's bounded
 * wait, on a barrier that nothing will ever complete.  The wait gives up after its iteration
 * limit (a fraction of a second), the kernel ends normally and the cache's status word reads
 * XKV_E_TIMEOUT at the next xkv_poll_status; xkv_reset clears it.  Nothing faults or hangs. */
XKV_API int xkv_debug_timeout_probe(xkv_cache* cache, xkv_stream stream);

/* Optional per-kernel timing for benchmarks.  While enabled, every kernel the
 * library launches for this cache is bracketed by a pair of CUDA events on the
 * launching stream (a small overhead; leave it off in production).
 * xkv_profile_read synchronises `stream`, adds the elapsed time of all launches
 * recorded since the last read to the per-category totals, copies the totals to
 * *out and clears them. */
enum { XKV_PROF_APPEND = 0,       /* kv_append                                                       */
       XKV_PROF_SCORE_EVICT = 1,  /* kv_score_evict: pooled query, scores, selection                 */
       XKV_PROF_PACK = 2,         /* kv_quant_pack: key regroup / survivor gather                    */
       XKV_PROF_KBAR = 3,         /* head means of the keys, by the stream step beside the attention */
       XKV_PROF_MAINT = 4,        /* the three calls above as one launch (stream step)               */
       XKV_PROF_ATTN = 5, XKV_PROF_COMBINE = 6,
       XKV_PROF_CATEGORIES = 7 };
typedef struct {
  double  ms[XKV_PROF_CATEGORIES];        /* summed device time per category, milliseconds */
  int64_t launches[XKV_PROF_CATEGORIES];  /* launches per category                         */
} xkv_profile;
XKV_API int xkv_profile_enable(xkv_cache* cache, int enable);
XKV_API int xkv_profile_read(xkv_cache* cache, xkv_profile* out, xkv_stream stream);

/* ---- synthetic inputs (not part of the method) -------------------------------- */

/* Fills dst (device, bf16 [n_heads][n_tokens][head_dim]) with the seeded
 * Irwin-Hall(12) variates of the input recipe: element e of the tensor is built
 * from three 64-bit hash words of (key + 3e + i); entries of outlier_channels
 * (HOST int32 [n_heads][n_outliers], may be null) are multiplied by `gain`. */
XKV_API int xkv_synth_fill(void* dst, uint64_t key, int32_t n_heads, int32_t n_tokens, int32_t head_dim,
                   const int32_t* outlier_channels, int32_t n_outliers, float gain,
                   xkv_stream stream);

#ifdef __cplusplus
}
#endif
#endif  /* XKV_H_ */
