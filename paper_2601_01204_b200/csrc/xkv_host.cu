// Host side of libxkv: workspace layout, the per-cache call-order state machine,
// the C ABI, and the synthetic-input generator kernel.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>

#include "xkv_internal.cuh"

using namespace xkv;

namespace {

constexpr size_t kAlign = 256;

struct Layout {
  int cap, row_bytes;
  size_t off_k[2], off_kpar[2], off_v[2], off_vpar[2], off_origin[2], off_kbar[2];
  size_t off_kstage, off_qbar, off_qvec, off_scores, off_kept, off_counters, off_status, off_attn, off_hist;
  size_t off_run_hi, off_cand;
  size_t off_kslot[2], off_ktab32, off_ktab16, off_ref, off_ring;
  int n_slots;
  size_t attn_bytes;
  size_t total;
};

bool params_ok(const xkv_params* p) {
  if (!p) return false;
  if (p->n_heads < 1 || p->n_heads > 64) return false;
  if (p->head_dim != kHeadDim || p->quant_group != kGroup) return false;
  if (p->kv_bits != 4 && p->kv_bits != 8 && p->kv_bits != 16) return false;
  if (p->n_special < 0 || p->pool_g < 1 || p->budget < 1) return false;
  if (p->max_frame_tokens < 1 || p->max_frame_tokens > 65535) return false;
  if (p->budget > (1 << 24)) return false;
  if (p->key_mode != XKV_KEYS_REGROUP && p->key_mode != XKV_KEYS_ONCE) return false;
  if (p->key_mode == XKV_KEYS_ONCE && p->kv_bits == 16) return false;
  if (p->kv_bits == 8 && p->key_mode != XKV_KEYS_ONCE) return false;      // 8-bit codes: quantise-once mode only
  if (p->key_table_slots < 0 || (p->key_mode != XKV_KEYS_ONCE && p->key_table_slots != 0)) return false;
  return true;
}

Layout make_layout(const xkv_params* p) {
  Layout L;
  memset(&L, 0, sizeof(L));
  const int max_n = p->max_frame_tokens;
  // first segment padded to a tile; rest holds at most max(budget, max_n) tokens after a step
  const int cap_first = round_up(max_n, kTile);
  const int cap_rest = round_up(p->budget > max_n ? p->budget : max_n, kTile) + kTile;
  L.cap = cap_first + cap_rest;
  L.row_bytes = (p->kv_bits == 4) ? 32 : (p->kv_bits == 8) ? 64 : 128;
  const size_t H = (size_t)p->n_heads;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + kAlign - 1) / kAlign * kAlign; return o; };
  L.off_status = take(256);
  L.off_counters = take(576 * sizeof(unsigned int));
  L.off_hist = take(4 * 4096 * sizeof(unsigned int));
  for (int b = 0; b < 2; ++b) {
    L.off_k[b] = take(H * L.cap * L.row_bytes);
    L.off_kpar[b] = take(H * (L.cap / 64) * 64 * sizeof(float2));
    L.off_v[b] = take(H * L.cap * L.row_bytes);
    L.off_vpar[b] = take(H * L.cap * sizeof(float2));
    L.off_origin[b] = take((size_t)L.cap * sizeof(int32_t));
    L.off_kbar[b] = take((size_t)L.cap * 64 * sizeof(float));
  }
  L.off_kstage = take(H * max_n * 64 * sizeof(__nv_bfloat16));
  const int np_max = max_n;  // upper bound of N_pooled
  L.off_qbar = take((size_t)np_max * 64 * sizeof(float));
  L.off_qvec = take(64 * sizeof(float));
  L.off_scores = take((size_t)L.cap * sizeof(float));
  L.off_kept = take((size_t)L.cap * sizeof(int32_t));
  L.off_run_hi = take((size_t)(L.cap / 64) * sizeof(unsigned int));
  L.off_cand = take((size_t)L.cap * sizeof(unsigned long long));
  if (p->key_mode == XKV_KEYS_ONCE) {
    // every live group holds at least one cached token, so one slot per token slot never runs out;
    // at least the groups of two frames (the first and the one arriving) are needed in any case
    const int least = 2 * ((max_n + 63) / 64) + 1;
    L.n_slots = p->key_table_slots > 0 ? (p->key_table_slots > least ? p->key_table_slots : least) : L.cap;
    for (int b = 0; b < 2; ++b) L.off_kslot[b] = take((size_t)L.cap * sizeof(int32_t));
    L.off_ktab32 = take((size_t)L.n_slots * H * 64 * sizeof(float2));
    L.off_ktab16 = take((size_t)L.n_slots * H * 8 * 12 * sizeof(uint32_t));
    L.off_ref = take((size_t)L.n_slots * sizeof(int32_t));
    L.off_ring = take((size_t)L.n_slots * sizeof(int32_t));
  }
  L.attn_bytes = attn_tc_scratch_bytes(p);
  L.off_attn = take(L.attn_bytes);
  L.total = off;
  return L;
}

bool strides_ok(int64_t ts, int64_t hs) { return ts >= kHeadDim && (ts % 8) == 0 && hs >= 0 && (hs % 8) == 0; }
bool aligned16(const void* p) { return p && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int zero_workspace(xkv_cache* c, cudaStream_t st) {
  if (cudaMemsetAsync(c->ws, 0, c->ws_bytes, st) != cudaSuccess) return XKV_E_CUDA;
  if (c->p.key_mode == XKV_KEYS_ONCE && launch_once_init(c, st) != cudaSuccess) return XKV_E_CUDA;
  return XKV_OK;
}

void reset_host_state(xkv_cache* c) {
  c->frames = c->T = c->T_first = c->rest_base = c->cur = c->stage = 0;
  c->n_pending = c->kk_pending = c->rold_pending = c->evict_pending = c->first_pending = 0;
  c->last_evicted = c->last_kept = c->last_prunable = 0;
  c->kbar_T = c->kbar_cur = c->kbar_frames = -1;
  c->bar_base = 0;
  c->sel_parity = 0;
  c->stats_parity = -1;
  c->budget_now = c->p.budget;
  c->pop_base = 0;
}

}  // namespace

extern "C" {

size_t xkv_workspace_bytes(const xkv_params* params) {
  if (!params_ok(params)) return 0;
  return make_layout(params).total;
}

int xkv_create(const xkv_params* params, void* dev_workspace, size_t bytes, xkv_stream stream, xkv_cache** out) {
  if (!out) return XKV_E_INVALID;
  *out = nullptr;
  if (!params) return XKV_E_INVALID;
  if (!params_ok(params)) {
    if (params->head_dim != kHeadDim && params->head_dim > 0) return XKV_E_UNSUPPORTED;
    if (params->quant_group != kGroup && params->quant_group > 0) return XKV_E_UNSUPPORTED;
    if (params->kv_bits == 2 || params->kv_bits == 8) return XKV_E_UNSUPPORTED;   // 8 needs XKV_KEYS_ONCE
    return XKV_E_INVALID;
  }
  if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) % kAlign) != 0) return XKV_E_INVALID;
  const Layout L = make_layout(params);
  if (bytes < L.total) return XKV_E_NOMEM;
  xkv_cache* c = new (std::nothrow) xkv_cache;
  if (!c) return XKV_E_NOMEM;
  memset(c, 0, sizeof(*c));
  c->p = *params;
  c->cap = L.cap;
  c->row_bytes = L.row_bytes;
  c->ws = reinterpret_cast<uint8_t*>(dev_workspace);
  c->ws_bytes = L.total;
  for (int b = 0; b < 2; ++b) {
    c->buf[b].k = c->ws + L.off_k[b];
    c->buf[b].kpar = reinterpret_cast<float2*>(c->ws + L.off_kpar[b]);
    c->buf[b].v = c->ws + L.off_v[b];
    c->buf[b].vpar = reinterpret_cast<float2*>(c->ws + L.off_vpar[b]);
    c->buf[b].origin = reinterpret_cast<int32_t*>(c->ws + L.off_origin[b]);
    c->buf[b].kbar = reinterpret_cast<float*>(c->ws + L.off_kbar[b]);
    c->buf[b].kslot = params->key_mode == XKV_KEYS_ONCE ? reinterpret_cast<int32_t*>(c->ws + L.off_kslot[b]) : nullptr;
  }
  if (params->key_mode == XKV_KEYS_ONCE) {
    c->n_slots = L.n_slots;
    c->ktab32 = reinterpret_cast<float2*>(c->ws + L.off_ktab32);
    c->ktab16 = reinterpret_cast<uint32_t*>(c->ws + L.off_ktab16);
    c->ref = reinterpret_cast<int32_t*>(c->ws + L.off_ref);
    c->ring = reinterpret_cast<int32_t*>(c->ws + L.off_ring);
  }
  c->kstage = reinterpret_cast<__nv_bfloat16*>(c->ws + L.off_kstage);
  c->qbar = reinterpret_cast<float*>(c->ws + L.off_qbar);
  c->qvec = reinterpret_cast<float*>(c->ws + L.off_qvec);
  c->scores = reinterpret_cast<float*>(c->ws + L.off_scores);
  c->kept = reinterpret_cast<int32_t*>(c->ws + L.off_kept);
  c->counters = reinterpret_cast<unsigned int*>(c->ws + L.off_counters);
  c->sel_hist = reinterpret_cast<unsigned int*>(c->ws + L.off_hist);
  c->run_hi = reinterpret_cast<unsigned int*>(c->ws + L.off_run_hi);
  c->cand = reinterpret_cast<unsigned long long*>(c->ws + L.off_cand);
  c->status = reinterpret_cast<int*>(c->ws + L.off_status);
  c->attn_part = reinterpret_cast<float*>(c->ws + L.off_attn);
  c->attn_part_bytes = L.attn_bytes;
  reset_host_state(c);
  c->prof = new (std::nothrow) Profiler;
  if (!c->prof) { delete c; return XKV_E_NOMEM; }
  if (cudaEventCreateWithFlags(&c->kbar_done, cudaEventDisableTiming) != cudaSuccess) {
    delete c->prof; delete c; return XKV_E_CUDA;
  }
  const int rc = zero_workspace(c, reinterpret_cast<cudaStream_t>(stream));
  if (rc != XKV_OK) { cudaEventDestroy(c->kbar_done); delete c->prof; delete c; return rc; }
  *out = c;
  return XKV_OK;
}

int xkv_reset(xkv_cache* c, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  // a head-mean kernel of the last stream step may still run on the library's stream
  if (c->kbar_done && cudaStreamWaitEvent(reinterpret_cast<cudaStream_t>(stream), c->kbar_done, 0) != cudaSuccess)
    return XKV_E_CUDA;
  reset_host_state(c);
  return zero_workspace(c, reinterpret_cast<cudaStream_t>(stream));
}

int xkv_destroy(xkv_cache* c) {
  if (!c) return XKV_E_INVALID;
  if (c->prof) {
    for (auto& e : c->prof->pending) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
    for (auto& e : c->prof->pool) cudaEventDestroy(e);
    delete c->prof;
  }
  if (c->kbar_done) { cudaEventSynchronize(c->kbar_done); cudaEventDestroy(c->kbar_done); }
  delete c;
  return XKV_OK;
}

}  // extern "C"

namespace {

// What the cache will look like once the frame of n tokens is in: a pure function of the sizes
// seen so far and the budget (Sec. 3.2), so no device data is needed.
struct FramePlan { int first, r_old, kk, evict, dst_slot; };

int plan_frame(const xkv_cache* c, int n, FramePlan* p) {
  p->first = (c->frames == 0) ? 1 : 0;
  p->r_old = p->kk = p->evict = p->dst_slot = 0;
  if (!p->first) {
    p->r_old = c->T - c->T_first;
    p->evict = (c->T + n > c->budget_now) ? 1 : 0;             // pruning is triggered when T > L_max
    p->kk = p->evict ? (c->budget_now - c->T_first - n) : p->r_old;   // k = max(0, L_max - T_first - T_current)
    if (p->kk < 0) p->kk = 0;
    p->dst_slot = c->rest_base + p->kk;
    if (p->dst_slot + n > c->cap) return XKV_E_NOMEM;
  }
  return XKV_OK;
}

// Everything of MaintArgs that describes the cache and the pending frame.
void maint_args(const xkv_cache* c, MaintArgs* a) {
  memset(a, 0, sizeof(*a));
  a->H = c->p.n_heads; a->cap = c->cap; a->max_n = c->p.max_frame_tokens;
  a->frame = c->frames + 1;
  a->first = c->first_pending;
  a->cur = c->buf[c->cur]; a->oth = c->buf[c->cur ^ 1];
  a->n = c->n_pending;
  a->n_q = c->nq_pending > 0 ? c->nq_pending : c->n_pending;
  a->rest_base = c->rest_base; a->r_old = c->rold_pending; a->kk = c->kk_pending;
  a->r_new = c->kk_pending + c->n_pending;
  a->dst_slot = c->first_pending ? 0 : c->rest_base + c->kk_pending;
  a->identity = !(c->evict_pending && c->kk_pending > 0 && c->kk_pending < c->rold_pending);
  a->n_special = c->p.n_special < a->n_q ? c->p.n_special : a->n_q;
  a->pool_g = c->p.pool_g;
  a->n_pooled = a->n_special + (a->n_q - a->n_special + c->p.pool_g - 1) / c->p.pool_g;
  a->kstage = c->kstage; a->qbar = c->qbar; a->qvec = c->qvec; a->scores = c->scores; a->kept = c->kept;
  a->hist = c->sel_hist; a->run_hi = c->run_hi; a->cand = c->cand;
  a->force_plain = c->force_plain;
  a->ktab32 = c->ktab32; a->ktab16 = c->ktab16; a->ref = c->ref; a->ring = c->ring;
  a->n_slots = c->n_slots; a->pop_base = c->pop_base;
}

bool keys_once(const xkv_cache* c) { return c->p.key_mode == XKV_KEYS_ONCE; }

void set_pending(xkv_cache* c, int n, const FramePlan& p) {
  c->n_pending = n;
  c->nq_pending = 0;
  c->kk_pending = p.kk;
  c->rold_pending = p.r_old;
  c->evict_pending = p.evict;
  c->first_pending = p.first;
}

bool selecting(const xkv_cache* c) {
  return c->evict_pending && c->kk_pending > 0 && c->kk_pending < c->rold_pending;
}

bool kbar_fresh(const xkv_cache* c) {
  return c->kbar_T == c->T && c->kbar_cur == c->cur && c->kbar_frames == c->frames;
}

void note_scored(xkv_cache* c) {
  c->last_evicted = 0;
  if (c->evict_pending) {
    c->last_prunable = c->rold_pending;
    c->last_kept = c->kk_pending;
    c->last_evicted = c->rold_pending - c->kk_pending;
  }
}

void note_packed(xkv_cache* c) {
  const int n = c->n_pending;
  if (c->first_pending) {
    c->T_first = n;
    c->rest_base = round_up(n, kTile);
    c->T = n;
  } else {
    c->T = c->T_first + c->kk_pending + n;
    c->cur ^= 1;
  }
  c->frames += 1;
}

}  // namespace

extern "C" {

int kv_append(xkv_cache* c, const void* k, const void* v, int32_t n, int64_t ts, int64_t hs, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 0) return XKV_E_STATE;
  if (n < 1 || n > c->p.max_frame_tokens || !aligned16(k) || !aligned16(v) || !strides_ok(ts, hs))
    return XKV_E_INVALID;
  FramePlan plan;
  const int rc = plan_frame(c, n, &plan);
  if (rc != XKV_OK) return rc;
  set_pending(c, n, plan);
  MaintArgs a;
  maint_args(c, &a);
  a.phases = kPhAppend;
  if (keys_once(c) && !plan.first) a.phases |= kPhKbarNew;
  a.k = reinterpret_cast<const __nv_bfloat16*>(k);
  a.v = reinterpret_cast<const __nv_bfloat16*>(v);
  a.ts_kv = ts; a.hs_kv = hs;
  if (launch_maint(c, a, XKV_PROF_APPEND, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
  if (keys_once(c)) c->pop_base += (uint32_t)((n + 63) / 64);
  c->stage = 1;
  return XKV_OK;
}

int kv_score_evict(xkv_cache* c, const void* q, int32_t n, int64_t ts, int64_t hs, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 1) return XKV_E_STATE;
  // n is the frame's size; after a chunk of frames was appended, the size of its last frame
  if (n < 1 || n > c->n_pending || !aligned16(q) || !strides_ok(ts, hs)) return XKV_E_INVALID;
  c->nq_pending = n;
  note_scored(c);
  if (selecting(c)) {
    MaintArgs a;
    maint_args(c, &a);
    a.phases = kPhPool | kPhScore | kPhSel;
    if (!keys_once(c) && !kbar_fresh(c)) {          // head means of the keys (Eq. 4) of the cache as it stands
      a.phases |= kPhKbar;
      a.kbar_on_other = 0; a.kbar_lo = 0; a.kbar_hi = c->rold_pending;
    }
    a.q = reinterpret_cast<const __nv_bfloat16*>(q);
    a.ts_q = ts; a.hs_q = hs;
    if (launch_maint(c, a, XKV_PROF_SCORE_EVICT, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
    if (!keys_once(c)) { c->kbar_T = c->T; c->kbar_cur = c->cur; c->kbar_frames = c->frames; }
  }
  c->stage = 2;
  return XKV_OK;
}

int kv_score_evict_w(xkv_cache* c, const float* w, int32_t n, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 1) return XKV_E_STATE;
  if (n < 1 || n > c->n_pending || !aligned16(w)) return XKV_E_INVALID;
  note_scored(c);
  if (selecting(c)) {
    MaintArgs a;
    maint_args(c, &a);
    a.phases = kPhScore | kPhSel;
    if (!keys_once(c) && !kbar_fresh(c)) {
      a.phases |= kPhKbar;
      a.kbar_on_other = 0; a.kbar_lo = 0; a.kbar_hi = c->rold_pending;
    }
    a.w_in = w;
    if (launch_maint(c, a, XKV_PROF_SCORE_EVICT, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
    if (!keys_once(c)) { c->kbar_T = c->T; c->kbar_cur = c->cur; c->kbar_frames = c->frames; }
  }
  c->stage = 2;
  return XKV_OK;
}

int xkv_set_budget(xkv_cache* c, int32_t budget) {
  if (!c || budget < 1 || budget > c->p.budget) return XKV_E_INVALID;
  if (c->stage != 0) return XKV_E_STATE;
  c->budget_now = budget;
  return XKV_OK;
}

int xkv_read_score_stats(const xkv_cache* c, xkv_score_stats* out, xkv_stream stream) {
  if (!c || !out) return XKV_E_INVALID;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
  memset(out, 0, sizeof(*out));
  if (c->stats_parity < 0) return XKV_OK;
  float v[4];
  if (cudaMemcpy(v, c->counters + 16 + 4 * c->stats_parity, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return XKV_E_CUDA;
  out->count = c->last_prunable; out->kept = c->last_kept;
  out->sum = v[0]; out->sum_sq = v[1]; out->threshold = v[2];
  return XKV_OK;
}

int kv_quant_pack(xkv_cache* c, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 2) return XKV_E_STATE;
  MaintArgs a;
  maint_args(c, &a);
  if (c->p.kv_bits == 4 && !keys_once(c)) {
    if (launch_regroup(c, a, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
  } else if (c->kk_pending > 0 || (keys_once(c) && c->rold_pending > 0)) {   // survivors to move, or table slots to release
    a.phases = kPhPack;
    if (launch_maint(c, a, XKV_PROF_PACK, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
  }
  note_packed(c);
  c->stage = 3;
  return XKV_OK;
}

int attn_packed_causal(xkv_cache* c, const void* q, void* out, int32_t n, int64_t ts, int64_t hs,
                       float softmax_scale, int32_t impl, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 3) return XKV_E_STATE;
  if (n < 1 || n > c->p.max_frame_tokens || !aligned16(q) || !aligned16(out) || !strides_ok(ts, hs) ||
      !(softmax_scale > 0.f) || (impl != 0 && impl != 1))
    return XKV_E_INVALID;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (impl == 1) {
    e = launch_attn_simple(c, q, out, n, ts, hs, softmax_scale, st);
  } else {
    e = launch_attn_tc(c, q, out, n, ts, hs, softmax_scale, st);
    if (e == cudaErrorNotSupported) return XKV_E_UNSUPPORTED;
  }
  if (e != cudaSuccess) return XKV_E_CUDA;
  c->stage = 0;
  return XKV_OK;
}

int attn_packed_causal_tail(xkv_cache* c, const void* q, const void* k_t, const void* v_t, void* out, int32_t n,
                            int64_t ts, int64_t hs, float softmax_scale, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 3) return XKV_E_STATE;
  if (n < 1 || n != c->n_pending || !aligned16(q) || !aligned16(k_t) || !aligned16(v_t) || !aligned16(out) ||
      !strides_ok(ts, hs) || !(softmax_scale > 0.f))
    return XKV_E_INVALID;
  const cudaError_t e =
      launch_attn_tc_tail(c, q, k_t, v_t, out, n, ts, hs, softmax_scale, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorNotSupported) return XKV_E_UNSUPPORTED;
  if (e != cudaSuccess) return XKV_E_CUDA;
  c->stage = 0;
  return XKV_OK;
}

int attn_packed_frame_causal(xkv_cache* c, const void* q, void* out, const int32_t* frame_tokens, int32_t n_frames,
                             int64_t ts, int64_t hs, float softmax_scale, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 3) return XKV_E_STATE;
  if (!frame_tokens || n_frames < 1 || !aligned16(q) || !aligned16(out) || !strides_ok(ts, hs) || !(softmax_scale > 0.f))
    return XKV_E_INVALID;
  long long total = 0;
  for (int f = 0; f < n_frames; ++f) {
    if (frame_tokens[f] < 1) return XKV_E_INVALID;
    total += frame_tokens[f];
  }
  if (total != c->n_pending) return XKV_E_INVALID;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int before = c->T - c->n_pending;              // cached tokens older than the chunk
  int r0 = 0;
  for (int f = 0; f < n_frames; ++f) {
    const int nf = frame_tokens[f];
    const __nv_bfloat16* qf = reinterpret_cast<const __nv_bfloat16*>(q) + (int64_t)r0 * ts;
    __nv_bfloat16* of = reinterpret_cast<__nv_bfloat16*>(out) + (int64_t)r0 * ts;
    // (strides are multiples of 8 elements, so every frame's first row is 16-byte aligned)
    const cudaError_t e = launch_attn_tc(c, qf, of, nf, ts, hs, softmax_scale, st, before + r0 + nf);
    if (e == cudaErrorNotSupported) return XKV_E_UNSUPPORTED;
    if (e != cudaSuccess) return XKV_E_CUDA;
    r0 += nf;
  }
  c->stage = 0;
  return XKV_OK;
}

int xkv_prefill_chunk(xkv_cache* c, const void* q, const void* k, const void* v, void* out,
                      const int32_t* frame_tokens, int32_t n_frames, int64_t ts, int64_t hs, xkv_stream stream) {
  if (!c || !frame_tokens || n_frames < 1) return XKV_E_INVALID;
  long long total = 0;
  for (int f = 0; f < n_frames; ++f) { if (frame_tokens[f] < 1) return XKV_E_INVALID; total += frame_tokens[f]; }
  if (total > c->p.max_frame_tokens) return XKV_E_INVALID;
  const int n = (int)total, n_last = frame_tokens[n_frames - 1];
  int rc = kv_append(c, k, v, n, ts, hs, stream);
  if (rc != XKV_OK) return rc;
  const __nv_bfloat16* q_last = reinterpret_cast<const __nv_bfloat16*>(q) + (int64_t)(n - n_last) * ts;
  rc = kv_score_evict(c, q_last, n_last, ts, hs, stream);
  if (rc != XKV_OK) return rc;
  rc = kv_quant_pack(c, stream);
  if (rc != XKV_OK) return rc;
  return attn_packed_frame_causal(c, q, out, frame_tokens, n_frames, ts, hs, 1.0f / sqrtf((float)c->p.head_dim), stream);
}

int xkv_set_unquantised_tail(xkv_cache* c, int32_t on) {
  if (!c || (on != 0 && on != 1)) return XKV_E_INVALID;
  c->tail_mode = on;
  return XKV_OK;
}

int attn_packed_causal_static(xkv_cache* c, const void* q, void* out, int32_t n, int64_t ts, int64_t hs,
                              float softmax_scale, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 3) return XKV_E_STATE;
  if (n < 1 || n > c->p.max_frame_tokens || !aligned16(q) || !aligned16(out) || !strides_ok(ts, hs) ||
      !(softmax_scale > 0.f))
    return XKV_E_INVALID;
  const cudaError_t e = launch_attn_tc_static(c, q, out, n, ts, hs, softmax_scale, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorMemoryAllocation) return XKV_E_LIMIT;
  if (e == cudaErrorNotSupported) return XKV_E_UNSUPPORTED;
  if (e != cudaSuccess) return XKV_E_CUDA;
  c->stage = 0;
  return XKV_OK;
}

namespace {

// Streams and events of the stream-step calls, one set per device, created on first use.
struct HostStepPipe {
  bool ready = false;
  cudaStream_t up = nullptr, down = nullptr;      // host -> device, device -> host
  cudaStream_t up2 = nullptr;                     // a second host -> device stream (two copy engines: 49 GB/s against
                                                  // 31 GB/s for 2.8 MB copies on one stream)
  cudaEvent_t up2_done[2] = {nullptr, nullptr};
  cudaStream_t side = nullptr;                    // kv_append of a layer, beside its scoring
  cudaEvent_t fork = nullptr, join = nullptr;
  cudaEvent_t start = nullptr;                    // the caller's stream at entry
  cudaEvent_t up_done[2] = {nullptr, nullptr};    // inputs of the layer in slot s are on the device
  cudaEvent_t comp_done[2] = {nullptr, nullptr};  // the layer in slot s has run: inputs free, output ready
  cudaEvent_t down_done[2] = {nullptr, nullptr};  // output of slot s is in host memory: output buffer free
};
std::mutex g_pipe_mutex;
HostStepPipe g_pipe[64];

HostStepPipe* host_step_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostStepPipe& p = g_pipe[dev];
  if (!p.ready) {
    bool ok = cudaStreamCreateWithFlags(&p.up, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.down, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.up2, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.side, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.join, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaEventCreateWithFlags(&p.up_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&p.up2_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&p.comp_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&p.down_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    p.ready = true;
  }
  return &p;
}

// One layer, one frame: the three maintenance calls as one launch, then -- on the library's side
// stream, beside the attention -- the head means of the keys of the cache just built (Eq. 4), from
// which the next frame's scoring starts.
int run_layer(HostStepPipe* pipe, xkv_cache* c, const void* q, const void* k, const void* v, void* out, int32_t n,
              int64_t ts, int64_t hs, cudaStream_t st) {
  xkv_stream stream = reinterpret_cast<xkv_stream>(st);
  if (c->stage != 0) return XKV_E_STATE;
  if (n < 1 || n > c->p.max_frame_tokens || !aligned16(k) || !aligned16(v) || !aligned16(q) || !strides_ok(ts, hs))
    return XKV_E_INVALID;
  FramePlan plan;
  int rc = plan_frame(c, n, &plan);
  if (rc != XKV_OK) return rc;
  set_pending(c, n, plan);
  note_scored(c);
  MaintArgs a;
  maint_args(c, &a);
  const bool once = keys_once(c);
  a.phases = kPhAppend;
  if ((c->p.kv_bits == 16 && c->kk_pending > 0) || (once && (c->kk_pending > 0 || c->rold_pending > 0))) a.phases |= kPhPack;
  if (selecting(c)) {
    a.phases |= kPhPool | kPhScore | kPhSel;
    if (once) {
      // the head means travel with the tokens; those of the frame before were computed beside its attention
      if (c->kbar_frames == c->frames && cudaStreamWaitEvent(st, c->kbar_done, 0) != cudaSuccess) return XKV_E_CUDA;
    } else if (kbar_fresh(c)) {
      if (cudaStreamWaitEvent(st, c->kbar_done, 0) != cudaSuccess) return XKV_E_CUDA;
    } else {
      a.phases |= kPhKbar;
      a.kbar_on_other = 0; a.kbar_lo = 0; a.kbar_hi = c->rold_pending;
    }
  }
  a.q = reinterpret_cast<const __nv_bfloat16*>(q);
  a.k = reinterpret_cast<const __nv_bfloat16*>(k);
  a.v = reinterpret_cast<const __nv_bfloat16*>(v);
  a.ts_q = a.ts_kv = ts; a.hs_q = a.hs_kv = hs;
  if (launch_maint(c, a, XKV_PROF_MAINT, st) != cudaSuccess) return XKV_E_CUDA;
  if (once) c->pop_base += (uint32_t)((n + 63) / 64);
  if (c->p.kv_bits == 4 && !once && launch_regroup(c, a, st) != cudaSuccess) return XKV_E_CUDA;
  note_packed(c);
  c->stage = 3;
  // Head means of the keys (Eq. 4), needed by the next frame's scoring only: on the side stream,
  // beside the attention.  The side stream forks here (after the packing) but its kernel is
  // launched after the attention has been enqueued, so that the attention's blocks get the
  // multiprocessors first and the head means fill in as they retire.
  const bool want_kbar = once ? !plan.first : (c->T > c->T_first);
  if (want_kbar && !(cudaEventRecord(pipe->fork, st) == cudaSuccess &&
                     cudaStreamWaitEvent(pipe->side, pipe->fork, 0) == cudaSuccess))
    return XKV_E_CUDA;
  const float scale = 1.0f / sqrtf((float)c->p.head_dim);
  rc = c->tail_mode ? attn_packed_causal_tail(c, q, k, v, out, n, ts, hs, scale, stream)
                    : attn_packed_causal(c, q, out, n, ts, hs, scale, 0, stream);
  if (want_kbar && rc == XKV_OK) {
    MaintArgs b;
    if (once) {               // of the frame just quantised (the rest travelled with their tokens)
      b = a;
      b.phases = kPhKbarNew;
    } else {                  // of the whole cache after the first frame: re-quantisation changed the keys
      maint_args(c, &b);
      b.phases = kPhKbar;
      b.kbar_on_other = 0; b.kbar_lo = 0; b.kbar_hi = c->T - c->T_first;
    }
    const bool launched = launch_maint(c, b, XKV_PROF_KBAR, pipe->side) == cudaSuccess;
    const bool ok = cudaEventRecord(c->kbar_done, pipe->side) == cudaSuccess;
    // (the caller's stream waits for it at the end of the stream-step call, and at the next
    // frame's scoring)
    if (!launched || !ok) return XKV_E_CUDA;
    c->kbar_T = c->T; c->kbar_cur = c->cur; c->kbar_frames = c->frames;
  }
  return rc;
}

// Everything a stream-step call started on the side stream is ordered before what the caller
// enqueues next: the caller's stream waits for the head-mean kernels of all layers.
bool join_side_work(xkv_cache* const* layers, int n_layers, cudaStream_t st) {
  bool ok = true;
  for (int l = 0; l < n_layers; ++l)
    if (layers[l] && layers[l]->kbar_frames == layers[l]->frames && layers[l]->kbar_frames > 0)
      ok = cudaStreamWaitEvent(st, layers[l]->kbar_done, 0) == cudaSuccess && ok;
  return ok;
}

}  // namespace

int xkv_stream_step(xkv_cache* const* layers, int32_t n_layers, const void* const* q, const void* const* k,
                    const void* const* v, void* const* out, int32_t n, int64_t ts, int64_t hs,
                    xkv_stream stream) {
  if (!layers || !q || !k || !v || !out || n_layers < 1) return XKV_E_INVALID;
  HostStepPipe* pipe = host_step_pipe();
  if (!pipe) return XKV_E_CUDA;
  for (int l = 0; l < n_layers; ++l) {
    xkv_cache* c = layers[l];
    if (!c) return XKV_E_INVALID;
    const int rc = run_layer(pipe, c, q[l], k[l], v[l], out[l], n, ts, hs, reinterpret_cast<cudaStream_t>(stream));
    if (rc != XKV_OK) { join_side_work(layers, l + 1, reinterpret_cast<cudaStream_t>(stream)); return rc; }
  }
  return join_side_work(layers, n_layers, reinterpret_cast<cudaStream_t>(stream)) ? XKV_OK : XKV_E_CUDA;
}

size_t xkv_stream_step_host_bytes(const xkv_params* params, int32_t n) {
  if (!params_ok(params) || n < 1) return 0;
  // two slots (double buffering) of Q, K, V, out
  const size_t t = (size_t)params->n_heads * n * kHeadDim * sizeof(__nv_bfloat16);
  return 2 * 4 * ((t + kAlign - 1) / kAlign * kAlign);
}

// The layers run on the caller's stream; the inputs of layer l + 1 are copied to the other half of
// the staging buffer on a copy stream while layer l runs, and outputs go back on a third stream.
int xkv_stream_step_host(xkv_cache* const* layers, int32_t n_layers, const void* const* q,
                         const void* const* k, const void* const* v, void* const* out, int32_t n,
                         void* dev_staging, size_t staging_bytes, xkv_stream stream) {
  if (!layers || !q || !k || !v || !out || n_layers < 1 || !layers[0] || !dev_staging) return XKV_E_INVALID;
  const xkv_params* p = &layers[0]->p;
  if (n < 1 || n > p->max_frame_tokens) return XKV_E_INVALID;
  if (staging_bytes < xkv_stream_step_host_bytes(p, n)) return XKV_E_NOMEM;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l] || !q[l] || !k[l] || !v[l] || !out[l]) return XKV_E_INVALID;
  HostStepPipe* pipe = host_step_pipe();
  if (!pipe) return XKV_E_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t t = (size_t)p->n_heads * n * kHeadDim * sizeof(__nv_bfloat16);
  const size_t slot = (t + kAlign - 1) / kAlign * kAlign;
  uint8_t* base = reinterpret_cast<uint8_t*>(dev_staging);
  const int64_t ts = kHeadDim, hs = (int64_t)n * kHeadDim;
  int rc = XKV_OK;
  bool cuda_ok = true;
  auto ck = [&](cudaError_t e) { if (e != cudaSuccess) cuda_ok = false; };
  // the copy streams start where the caller's stream stands (the staging buffer may be in use there)
  ck(cudaEventRecord(pipe->start, st));
  ck(cudaStreamWaitEvent(pipe->up, pipe->start, 0));
  ck(cudaStreamWaitEvent(pipe->up2, pipe->start, 0));
  ck(cudaStreamWaitEvent(pipe->down, pipe->start, 0));
  int l = 0;
  for (; l < n_layers && cuda_ok && rc == XKV_OK; ++l) {
    xkv_cache* c = layers[l];
    const int sl = l & 1;
    uint8_t* s = base + (size_t)sl * 4 * slot;
    void* dq = s;
    void* dk = s + slot;
    void* dv = s + 2 * slot;
    void* dout = s + 3 * slot;
    // inputs: once the layer that used this half two layers ago has run
    if (l >= 2) {
      ck(cudaStreamWaitEvent(pipe->up, pipe->comp_done[sl], 0));
      ck(cudaStreamWaitEvent(pipe->up2, pipe->comp_done[sl], 0));
    }
    ck(cudaMemcpyAsync(dk, k[l], t, cudaMemcpyHostToDevice, pipe->up));
    ck(cudaMemcpyAsync(dq, q[l], t, cudaMemcpyHostToDevice, pipe->up2));
    ck(cudaMemcpyAsync(dv, v[l], t, cudaMemcpyHostToDevice, pipe->up));
    ck(cudaEventRecord(pipe->up_done[sl], pipe->up));
    ck(cudaEventRecord(pipe->up2_done[sl], pipe->up2));
    // the layer: inputs present, and the output of two layers ago copied out of this half
    ck(cudaStreamWaitEvent(st, pipe->up_done[sl], 0));
    ck(cudaStreamWaitEvent(st, pipe->up2_done[sl], 0));
    if (l >= 2) ck(cudaStreamWaitEvent(st, pipe->down_done[sl], 0));
    if (!cuda_ok) break;
    rc = run_layer(pipe, c, dq, dk, dv, dout, n, ts, hs, st);
    ck(cudaEventRecord(pipe->comp_done[sl], st));
    if (rc != XKV_OK) break;
    // output
    ck(cudaStreamWaitEvent(pipe->down, pipe->comp_done[sl], 0));
    ck(cudaMemcpyAsync(out[l], dout, t, cudaMemcpyDeviceToHost, pipe->down));
    ck(cudaEventRecord(pipe->down_done[sl], pipe->down));
  }
  // everything started above ends before the call returns, also after an error
  if (!join_side_work(layers, n_layers, st)) cuda_ok = false;
  ck(cudaStreamSynchronize(pipe->up));
  ck(cudaStreamSynchronize(pipe->up2));
  ck(cudaStreamSynchronize(st));
  ck(cudaStreamSynchronize(pipe->down));
  if (rc != XKV_OK) return rc;
  return cuda_ok ? XKV_OK : XKV_E_CUDA;
}

int xkv_get_info(const xkv_cache* c, xkv_info* info) {
  if (!c || !info) return XKV_E_INVALID;
  info->frames = c->frames;
  info->T = c->T;
  info->T_first = c->T_first;
  info->rest_base = c->rest_base;
  info->T_phys = c->rest_base + (c->T - c->T_first);
  info->capacity = c->cap;
  info->cur = c->cur;
  info->last_evicted = c->last_evicted;
  info->last_kept = c->last_kept;
  info->last_prunable = c->last_prunable;
  info->stage = c->stage;
  info->n_pending = c->n_pending;
  info->launches = c->launches;
  info->workspace_bytes = c->ws_bytes;
  info->key_table_slots = c->n_slots;
  info->budget = c->budget_now;
  return XKV_OK;
}

int64_t xkv_debug_export(const xkv_cache* c, int32_t which, void* host_dst, size_t bytes, xkv_stream stream) {
  if (!c || !host_dst) return XKV_E_INVALID;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return XKV_E_CUDA;
  const BufSet& b = c->buf[c->cur];
  const size_t H = (size_t)c->p.n_heads;
  const void* src = nullptr;
  size_t avail = 0;
  switch (which) {
    case XKV_BUF_K_CODES: src = b.k; avail = H * c->cap * c->row_bytes; break;
    case XKV_BUF_K_PARAMS: src = b.kpar; avail = H * (c->cap / 64) * 64 * sizeof(float2); break;
    case XKV_BUF_V_CODES: src = b.v; avail = H * c->cap * c->row_bytes; break;
    case XKV_BUF_V_PARAMS: src = b.vpar; avail = H * c->cap * sizeof(float2); break;
    case XKV_BUF_ORIGIN: src = b.origin; avail = (size_t)c->cap * sizeof(int32_t); break;
    case XKV_BUF_SCORES: src = c->scores; avail = (size_t)c->last_prunable * sizeof(float); break;
    case XKV_BUF_KEPT: src = c->kept; avail = (size_t)c->last_kept * sizeof(int32_t); break;
    case XKV_BUF_QVEC: src = c->qvec; avail = 64 * sizeof(float); break;
    case XKV_BUF_K_SLOT: src = b.kslot; avail = b.kslot ? (size_t)c->cap * sizeof(int32_t) : 0; break;
    case XKV_BUF_K_TABLE: src = c->ktab32; avail = (size_t)c->n_slots * H * 64 * sizeof(float2); break;
    case XKV_BUF_K_REF: src = c->ref; avail = (size_t)c->n_slots * sizeof(int32_t); break;
    default: return XKV_E_INVALID;
  }
  const size_t nbytes = bytes < avail ? bytes : avail;
  if (nbytes && cudaMemcpy(host_dst, src, nbytes, cudaMemcpyDeviceToHost) != cudaSuccess) return XKV_E_CUDA;
  return (int64_t)nbytes;
}

int xkv_debug_rewind_attention(xkv_cache* c) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 0 || c->frames < 1) return XKV_E_STATE;
  c->stage = 3;
  return XKV_OK;
}

int xkv_poll_status(const xkv_cache* c, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
  int word = 0;
  if (cudaMemcpy(&word, c->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return XKV_E_CUDA;
  if (word == 0) return XKV_OK;
  return (word == (int)XKV_E_RANGE || word == (int)XKV_E_LIMIT) ? word : XKV_E_TIMEOUT;
}

int xkv_debug_force_plain(xkv_cache* c, int32_t on) {
  if (!c || (on != 0 && on != 1)) return XKV_E_INVALID;
  c->force_plain = on;
  return XKV_OK;
}

int xkv_debug_limit_attention_blocks(xkv_cache* c, int32_t max_blocks) {
  if (!c || max_blocks < 0) return XKV_E_INVALID;
  c->attn_max_blocks = max_blocks;
  return XKV_OK;
}

int xkv_debug_head_means(xkv_cache* c, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  if (c->stage != 0) return XKV_E_STATE;
  if (c->T <= c->T_first || keys_once(c)) return XKV_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (c->kbar_done && cudaStreamWaitEvent(st, c->kbar_done, 0) != cudaSuccess) return XKV_E_CUDA;
  MaintArgs a;
  maint_args(c, &a);
  a.phases = kPhKbar;
  a.kbar_on_other = 0; a.kbar_lo = 0; a.kbar_hi = c->T - c->T_first;
  if (launch_maint(c, a, XKV_PROF_KBAR, st) != cudaSuccess) return XKV_E_CUDA;
  if (cudaEventRecord(c->kbar_done, st) != cudaSuccess) return XKV_E_CUDA;
  c->kbar_T = c->T; c->kbar_cur = c->cur; c->kbar_frames = c->frames;
  return XKV_OK;
}

int xkv_debug_timeout_probe(xkv_cache* c, xkv_stream stream) {
  if (!c) return XKV_E_INVALID;
  return launch_timeout_probe(c, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? XKV_OK : XKV_E_CUDA;
}

int xkv_profile_enable(xkv_cache* c, int enable) {
  if (!c || !c->prof) return XKV_E_INVALID;
  c->prof->on = enable != 0;
  return XKV_OK;
}

int xkv_profile_read(xkv_cache* c, xkv_profile* out, xkv_stream stream) {
  if (!c || !c->prof || !out) return XKV_E_INVALID;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return XKV_E_CUDA;
  Profiler* p = c->prof;
  for (auto& e : p->pending) {
    float ms = 0.f;
    if (cudaEventSynchronize(e.b) != cudaSuccess || cudaEventElapsedTime(&ms, e.a, e.b) != cudaSuccess)
      return XKV_E_CUDA;
    p->ms[e.cat] += ms;
    p->launches[e.cat] += 1;
    p->pool.push_back(e.a);
    p->pool.push_back(e.b);
  }
  p->pending.clear();
  for (int i = 0; i < XKV_PROF_CATEGORIES; ++i) {
    out->ms[i] = p->ms[i];
    out->launches[i] = p->launches[i];
    p->ms[i] = 0;
    p->launches[i] = 0;
  }
  return XKV_OK;
}

const char* xkv_strerror(int status) {
  switch (status) {
    case XKV_OK: return "ok";
    case XKV_E_INVALID: return "invalid argument";
    case XKV_E_STATE: return "call out of order for this cache";
    case XKV_E_NOMEM: return "workspace too small or host allocation failed";
    case XKV_E_UNSUPPORTED: return "parameter combination not supported";
    case XKV_E_CUDA: return "CUDA call failed";
    case XKV_E_TIMEOUT: return "bounded device-side wait ran out";
    case XKV_E_LIMIT: return "request exceeds a fixed built-in limit (static scratch size)";
    case XKV_E_RANGE: return "a value exceeds the range of the 16-bit tensor-core operands";
    default: return "unknown status";
  }
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Synthetic inputs: integer hash -> sum of twelve 16-bit fields -> bf16.
// ---------------------------------------------------------------------------
namespace {

struct OutlierTable { int32_t ch[64 * 4]; };

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27; x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}

__global__ void synth_kernel(__nv_bfloat16* dst, uint64_t key, long long count, int n_tokens, int head_dim,
                             OutlierTable tab, int n_out, float gain) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= count) return;
  int u = 0;
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const uint64_t w = mix64(key + 3ull * (uint64_t)e + (uint64_t)i);
    u += (int)(w & 0xFFFF) + (int)((w >> 16) & 0xFFFF) + (int)((w >> 32) & 0xFFFF) + (int)(w >> 48);
  }
  float x = __fmul_rn((float)(u - 6 * 65535), 1.52587890625e-05f);
  const int c = (int)(e % head_dim);
  const int h = (int)(e / ((long long)n_tokens * head_dim));
  for (int j = 0; j < n_out; ++j)
    if (tab.ch[h * 4 + j] == c) x = __fmul_rn(x, gain);
  dst[e] = __float2bfloat16_rn(x);
}

}  // namespace

extern "C" int xkv_synth_fill(void* dst, uint64_t key, int32_t n_heads, int32_t n_tokens, int32_t head_dim,
                              const int32_t* outlier_channels, int32_t n_outliers, float gain,
                              xkv_stream stream) {
  if (!dst || n_heads < 1 || n_heads > 64 || n_tokens < 1 || head_dim < 1 || n_outliers < 0 || n_outliers > 4)
    return XKV_E_INVALID;
  if (n_outliers > 0 && !outlier_channels) return XKV_E_INVALID;
  OutlierTable tab;
  for (int i = 0; i < 64 * 4; ++i) tab.ch[i] = -1;
  for (int h = 0; h < n_heads; ++h)
    for (int j = 0; j < n_outliers; ++j) tab.ch[h * 4 + j] = outlier_channels[h * n_outliers + j];
  const long long count = (long long)n_heads * n_tokens * head_dim;
  synth_kernel<<<(int)((count + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<__nv_bfloat16*>(dst), key, count, n_tokens, head_dim, tab, n_outliers, gain);
  return cudaGetLastError() == cudaSuccess ? XKV_OK : XKV_E_CUDA;
}
