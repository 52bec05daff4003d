// Cache-maintenance kernels: append (+ per-token value quantisation), pooled
// query, importance scores, top-k selection, key regroup/re-quantisation and the
// survivor gather.  All bandwidth- or latency-bound; fp32 arithmetic whose every
// operation and order is fixed, because it decides integers (kept indices, 4-bit
// codes) that must be reproducible bit for bit.
#include "xkv_internal.cuh"

namespace xkv {

// ---------------------------------------------------------------------------
// Eq. 7-8, fixed-order fp32:  s = (max-min)/15 (1 if the range is 0),
// inv = 1/s, z = rint(-min*inv) + 0, q = clamp(rint(x*inv) + z, 0, 15).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void quant_params(float mn, float mx, float& s, float& inv, float& z) {
  const float r = __fsub_rn(mx, mn);
  s = (r == 0.f) ? 1.f : __fdiv_rn(r, 15.f);
  inv = __fdiv_rn(1.f, s);
  z = __fadd_rn(rintf(__fmul_rn(-mn, inv)), 0.f);
}

__device__ __forceinline__ uint32_t quant_code(float x, float inv, float z) {
  float q = __fadd_rn(rintf(__fmul_rn(x, inv)), z);
  q = fminf(fmaxf(q, 0.f), 15.f);
  return (uint32_t)q;
}

// Bit position of channel j (0..7) inside the packed word:
// word = c0 | c2<<4 | c4<<8 | c6<<12 | c1<<16 | c3<<20 | c5<<24 | c7<<28.
__device__ __forceinline__ int nib_shift(int j) { return ((j >> 1) << 2) + ((j & 1) << 4); }

__device__ __forceinline__ uint32_t pack8(const uint32_t (&c)[8]) {
  uint32_t w = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) w |= c[j] << nib_shift(j);
  return w;
}

__device__ __forceinline__ void bf16x8_to_float(const uint4& u, float (&x)[8]) {
  const uint32_t r[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(r[i] << 16);
    x[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
  }
}

// Eq. 10 for the 8 channels of one packed word: x~ = s * (q - z).
__device__ __forceinline__ void dequant8(uint32_t word, const float2* __restrict__ par, float (&x)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float2 sz = par[j];
    const float q = (float)((word >> nib_shift(j)) & 0xFu);
    x[j] = __fmul_rn(sz.x, __fsub_rn(q, sz.y));
  }
}

// ---------------------------------------------------------------------------
// kv_append.  Thread = (head, token, 8-channel word).  Values: per-token
// min/max over the 64 channels by xor-shuffle inside the 8-lane group, then
// codes -> one 32-bit word per lane.  Keys: copied to the staging buffer (4-bit)
// or to their final slot (16-bit).
// ---------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(256)
append_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, int n,
              int64_t ts, int64_t hs, int H, int cap, int max_n, int dst_slot, int frame,
              BufSet d0, BufSet d1, bool two, __nv_bfloat16* __restrict__ kstage) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int w = (int)(g & 7);
  const long long th = g >> 3;
  const bool valid = th < (long long)H * n;
  const int h = valid ? (int)(th / n) : 0;
  const int tok = valid ? (int)(th % n) : 0;
  const int64_t src = (int64_t)h * hs + (int64_t)tok * ts + 8 * w;
  const uint4 kv = *reinterpret_cast<const uint4*>(k + src);
  const uint4 vv = *reinterpret_cast<const uint4*>(v + src);
  const size_t slot = (size_t)h * cap + dst_slot + tok;

  if (BITS == 16) {
    if (valid) {
      *reinterpret_cast<uint4*>(d0.k + slot * 128 + 16 * w) = kv;
      *reinterpret_cast<uint4*>(d0.v + slot * 128 + 16 * w) = vv;
      if (two) {
        *reinterpret_cast<uint4*>(d1.k + slot * 128 + 16 * w) = kv;
        *reinterpret_cast<uint4*>(d1.v + slot * 128 + 16 * w) = vv;
      }
    }
  } else {
    float x[8];
    bf16x8_to_float(vv, x);
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) { mn = fminf(mn, x[j]); mx = fmaxf(mx, x[j]); }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    float s, inv, z;
    quant_params(mn, mx, s, inv, z);
    uint32_t c[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) c[j] = quant_code(x[j], inv, z);
    const uint32_t word = pack8(c);
    if (valid) {
      *reinterpret_cast<uint32_t*>(d0.v + slot * 32 + 4 * w) = word;
      if (w == 0) d0.vpar[slot] = make_float2(s, z);
      if (two) {
        *reinterpret_cast<uint32_t*>(d1.v + slot * 32 + 4 * w) = word;
        if (w == 0) d1.vpar[slot] = make_float2(s, z);
      }
      *reinterpret_cast<uint4*>(kstage + ((size_t)h * max_n + tok) * 64 + 8 * w) = kv;
    }
  }
  if (valid && h == 0 && w == 0) {
    const int32_t o = (frame << 16) | tok;
    d0.origin[dst_slot + tok] = o;
    if (two) d1.origin[dst_slot + tok] = o;
  }
}

cudaError_t launch_append(xkv_cache* c, const void* k, const void* v, int n, int64_t ts, int64_t hs,
                          int dst_slot, bool first, cudaStream_t st) {
  const long long threads = (long long)c->p.n_heads * n * 8;
  const int blocks = (int)((threads + 255) / 256);
  const BufSet d0 = c->buf[c->cur ^ 1];
  const BufSet d1 = c->buf[c->cur];
  auto kk = reinterpret_cast<const __nv_bfloat16*>(k);
  auto vv = reinterpret_cast<const __nv_bfloat16*>(v);
  LaunchScope ls(c, XKV_PROF_APPEND, st);
  if (c->p.kv_bits == 16)
    append_kernel<16><<<blocks, 256, 0, st>>>(kk, vv, n, ts, hs, c->p.n_heads, c->cap,
                                              c->p.max_frame_tokens, dst_slot, c->frames + 1, d0, d1,
                                              first, c->kstage);
  else
    append_kernel<4><<<blocks, 256, 0, st>>>(kk, vv, n, ts, hs, c->p.n_heads, c->cap,
                                             c->p.max_frame_tokens, dst_slot, c->frames + 1, d0, d1,
                                             first, c->kstage);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Pooled query, Eq. 2-3, then the row mean that Eq. 5-6 reduce to.
// One CTA per pooled row i; thread (c, hs) builds pooled[h][i][c] for heads
// h = hs, hs+16, ... (sequential sum over the group's tokens, divided by the
// group size); threads with hs == 0 add the heads in order and scale by 1/H.
// The last CTA to finish adds the rows in order and divides by N_pooled.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
pool_q_kernel(const __nv_bfloat16* __restrict__ q, int n, int64_t ts, int64_t hs, int H, int n_special,
              int g, int n_pooled, float* __restrict__ qbar, float* __restrict__ qvec,
              unsigned int* __restrict__ counter) {
  extern __shared__ float s_pooled[];  // [H][64]
  __shared__ bool s_last;
  const int i = blockIdx.x;
  const int c = threadIdx.x;   // 0..63
  const int hslot = threadIdx.y;
  int a, b;
  if (i < n_special) { a = i; b = i + 1; }
  else { a = n_special + (i - n_special) * g; b = min(a + g, n); }
  for (int h = hslot; h < H; h += blockDim.y) {
    const __nv_bfloat16* base = q + (int64_t)h * hs + c;
    float acc = __bfloat162float(base[(int64_t)a * ts]);
    for (int t = a + 1; t < b; ++t) acc = __fadd_rn(acc, __bfloat162float(base[(int64_t)t * ts]));
    if (i >= n_special) acc = __fdiv_rn(acc, (float)(b - a));
    s_pooled[h * 64 + c] = acc;
  }
  __syncthreads();
  if (hslot == 0) {
    float acc = s_pooled[c];
    for (int h = 1; h < H; ++h) acc = __fadd_rn(acc, s_pooled[h * 64 + c]);
    const float inv_h = __fdiv_rn(1.f, (float)H);
    __stcg(&qbar[i * 64 + c], __fmul_rn(acc, inv_h));
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0 && threadIdx.y == 0) {
    const unsigned int done = atomicAdd(counter, 1u);
    s_last = (done == (unsigned int)n_pooled - 1u);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    if (hslot == 0) {
      float acc = __ldcg(&qbar[c]);
      for (int r = 1; r < n_pooled; ++r) acc = __fadd_rn(acc, __ldcg(&qbar[r * 64 + c]));
      qvec[c] = __fdiv_rn(acc, (float)n_pooled);
    }
    if (threadIdx.x == 0 && threadIdx.y == 0) *counter = 0u;  // re-arm for the next launch
  }
}

cudaError_t launch_pool_q(xkv_cache* c, const void* q, int n, int64_t ts, int64_t hs, cudaStream_t st) {
  const int H = c->p.n_heads;
  const int nsp = min(c->p.n_special, n);
  const int np = nsp + (n - nsp + c->p.pool_g - 1) / c->p.pool_g;
  const dim3 block(64, H < 16 ? H : 16);
  LaunchScope ls(c, XKV_PROF_POOL, st);
  pool_q_kernel<<<np, block, (size_t)H * 64 * sizeof(float), st>>>(
      reinterpret_cast<const __nv_bfloat16*>(q), n, ts, hs, H, nsp, c->p.pool_g, np, c->qbar, c->qvec,
      c->counters);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Scores, Eq. 4-6.  One CTA per 64-slot key group of the middle segment (the
// rest segment starts on a 128-slot boundary, so a CTA's tokens share their
// quantisation parameters).  Thread = (token, 8-channel word): dequantise the
// word of every head in order (Eq. 10), accumulate the head sum sequentially,
// scale by 1/H (Eq. 4), multiply by the query vector, and add the 64 products
// with a balanced tree: three levels inside the lane, three by xor-shuffle.
// ---------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(512)
score_kernel(BufSet cur, int H, int cap, int rest_base, int r_old, const float* __restrict__ qvec,
             float* __restrict__ scores) {
  extern __shared__ float2 s_par[];  // [H][64]
  __shared__ float s_w[64];
  const int tid = threadIdx.x;
  const int w = tid & 7;
  const int tok = tid >> 3;
  const int i = blockIdx.x * 64 + tok;          // rest-local index
  const int slot = rest_base + i;
  const int grp = (rest_base >> 6) + blockIdx.x;
  if (BITS == 4) {
    for (int e = tid; e < H * 64; e += 512)
      s_par[e] = cur.kpar[((size_t)(e >> 6) * (cap >> 6) + grp) * 64 + (e & 63)];
  }
  if (tid < 64) s_w[tid] = qvec[tid];
  __syncthreads();
  const bool valid = i < r_old;
  float acc[8];
  for (int h = 0; h < H; ++h) {
    float x[8];
    if (BITS == 4) {
      const uint32_t word =
          valid ? *reinterpret_cast<const uint32_t*>(cur.k + ((size_t)h * cap + slot) * 32 + 4 * w) : 0u;
      dequant8(word, s_par + h * 64 + 8 * w, x);
    } else {
      uint4 u = make_uint4(0, 0, 0, 0);
      if (valid) u = *reinterpret_cast<const uint4*>(cur.k + ((size_t)h * cap + slot) * 128 + 16 * w);
      bf16x8_to_float(u, x);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = (h == 0) ? x[j] : __fadd_rn(acc[j], x[j]);
  }
  const float inv_h = __fdiv_rn(1.f, (float)H);
  float p[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) p[j] = __fmul_rn(__fmul_rn(acc[j], inv_h), s_w[8 * w + j]);
  float t0 = __fadd_rn(p[0], p[1]), t1 = __fadd_rn(p[2], p[3]);
  float t2 = __fadd_rn(p[4], p[5]), t3 = __fadd_rn(p[6], p[7]);
  t0 = __fadd_rn(t0, t1);
  t2 = __fadd_rn(t2, t3);
  float s = __fadd_rn(t0, t2);
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
  if (valid && w == 0) scores[i] = s;
}

cudaError_t launch_score(xkv_cache* c, int r_old, cudaStream_t st) {
  const int blocks = (r_old + 63) / 64;
  const size_t smem = (size_t)c->p.n_heads * 64 * sizeof(float2);
  LaunchScope ls(c, XKV_PROF_SCORE, st);
  if (c->p.kv_bits == 16)
    score_kernel<16><<<blocks, 512, smem, st>>>(c->buf[c->cur], c->p.n_heads, c->cap, c->rest_base, r_old,
                                                c->qvec, c->scores);
  else
    score_kernel<4><<<blocks, 512, smem, st>>>(c->buf[c->cur], c->p.n_heads, c->cap, c->rest_base, r_old,
                                               c->qvec, c->scores);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Top-k of the scores (Sec. 3.2) by radix select on the order key
// (fp32 bit pattern mapped to an unsigned whose order is the float total order),
// then a stable compaction: keep every key above the threshold and the first
// (k - #above) keys equal to it.  One CTA; the input is at most a few hundred KB
// and L2-resident.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 1024;

__device__ __forceinline__ unsigned int block_excl_scan(unsigned int v, unsigned int* s_warp,
                                                        unsigned int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) s_warp[warp] = x;
  __syncthreads();
  if (warp == 0) {
    unsigned int t = s_warp[lane];
    unsigned int y = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int z = __shfl_up_sync(0xffffffffu, y, o);
      if (lane >= o) y += z;
    }
    s_warp[lane] = y - t;          // exclusive warp offsets
    if (lane == 31) s_warp[32] = y;  // grand total
  }
  __syncthreads();
  const unsigned int res = s_warp[warp] + x - v;
  total = s_warp[32];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int tp, int k, int32_t* __restrict__ kept) {
  __shared__ unsigned int s_hist[256];
  __shared__ unsigned int s_scan[256];
  __shared__ unsigned int s_warp[33];
  __shared__ unsigned int s_prefix, s_need;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  if (tid == 0) { s_prefix = 0u; s_need = (unsigned int)k; }
  unsigned int mask = 0u;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) s_hist[tid] = 0u;
    __syncthreads();
    const unsigned int prefix = s_prefix;
    for (int base = 0; base < tp; base += kSelThreads) {
      const int j = base + tid;
      const bool in = j < tp;
      const uint32_t key = in ? order_key(scores[j]) : 0u;
      const bool cand = in && ((key & mask) == prefix);
      const unsigned int digit = cand ? ((key >> shift) & 255u) : 256u;
      // warp-aggregated histogram update: one atomic per distinct digit per warp
      const unsigned int peers = __match_any_sync(0xffffffffu, digit);
      if (cand && lane == (__ffs(peers) - 1)) atomicAdd(&s_hist[digit], (unsigned int)__popc(peers));
    }
    __syncthreads();
    // s_scan[b] = number of candidates with digit > b (suffix sum), 256 threads, 8 doubling steps
    if (tid < 256) s_scan[tid] = (tid < 255) ? s_hist[tid + 1] : 0u;
    __syncthreads();
    for (int o = 1; o < 256; o <<= 1) {
      unsigned int add = 0u;
      if (tid < 256 && tid + o < 256) add = s_scan[tid + o];
      __syncthreads();
      if (tid < 256) s_scan[tid] += add;
      __syncthreads();
    }
    if (tid < 256) {
      const unsigned int above = s_scan[tid];
      const unsigned int need = s_need;
      if (above < need && need <= above + s_hist[tid]) {
        s_prefix = prefix | ((unsigned int)tid << shift);
        s_need = need - above;
      }
    }
    mask |= 0xFFu << shift;
    __syncthreads();
  }
  const uint32_t tau = s_prefix;
  const unsigned int need_eq = s_need;
  // stable compaction; each thread owns a run of consecutive positions
  const int ipt = (tp + kSelThreads - 1) / kSelThreads;
  const int j0 = min(tid * ipt, tp), j1 = min(j0 + ipt, tp);
  unsigned int cnt_eq = 0u, cnt_gt = 0u;
  for (int j = j0; j < j1; ++j) {
    const uint32_t key = order_key(scores[j]);
    cnt_eq += (key == tau);
    cnt_gt += (key > tau);
  }
  unsigned int total;
  const unsigned int eq_before = block_excl_scan(cnt_eq, s_warp, total);
  unsigned int take_eq = 0u;
  if (eq_before < need_eq) take_eq = min(cnt_eq, need_eq - eq_before);
  unsigned int out = block_excl_scan(cnt_gt + take_eq, s_warp, total);
  for (int j = j0; j < j1; ++j) {
    const uint32_t key = order_key(scores[j]);
    bool keep = key > tau;
    if (key == tau && take_eq > 0u) { keep = true; --take_eq; }
    if (keep) kept[out++] = j;
  }
}

cudaError_t launch_select(xkv_cache* c, int r_old, int k, cudaStream_t st) {
  LaunchScope ls(c, XKV_PROF_SELECT, st);
  select_kernel<<<1, kSelThreads, 0, st>>>(c->scores, r_old, k, c->kept);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// kv_quant_pack, keys (4-bit).  One CTA per (new 64-slot group, head); thread =
// (token, 8-channel word).  Survivors are dequantised with the parameters of
// the group they came from (Eq. 10), new keys come from the bf16 staging buffer;
// per-channel min/max over the group's tokens; new parameters and codes
// (Eq. 7-8).  A complete group whose 64 tokens all survive in place is copied.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(512)
regroup_k_kernel(BufSet src, BufSet dst, BufSet dst2, bool two, int cap, int max_n, int base_slot, int kk,
                 int r_new, const int32_t* __restrict__ kept, const __nv_bfloat16* __restrict__ kstage) {
  __shared__ float s_mn[16][64];
  __shared__ float s_mx[16][64];
  __shared__ float2 s_iz[64];
  const int tid = threadIdx.x;
  const int w = tid & 7;
  const int tok = tid >> 3;
  const int warp = tid >> 5;
  const int gamma = blockIdx.x;
  const int h = blockIdx.y;
  const int i = gamma * 64 + tok;
  const bool valid = i < r_new;
  const size_t dslot = (size_t)h * cap + base_slot + i;
  const size_t dgrp = ((size_t)h * (cap >> 6) + (base_slot >> 6) + gamma) * 64;
  const int last = gamma * 64 + 63;
  const bool carried = (last < kk) && (kept == nullptr || kept[last] == last);
  if (carried) {
    const uint32_t word = *reinterpret_cast<const uint32_t*>(src.k + dslot * 32 + 4 * w);
    *reinterpret_cast<uint32_t*>(dst.k + dslot * 32 + 4 * w) = word;
    if (two) *reinterpret_cast<uint32_t*>(dst2.k + dslot * 32 + 4 * w) = word;
    if (tid < 64) {
      const float2 sz = src.kpar[dgrp + tid];
      dst.kpar[dgrp + tid] = sz;
      if (two) dst2.kpar[dgrp + tid] = sz;
    }
    return;
  }
  float x[8];
  if (valid && i < kk) {
    const int old = kept ? kept[i] : i;
    const size_t sslot = (size_t)h * cap + base_slot + old;
    const uint32_t word = *reinterpret_cast<const uint32_t*>(src.k + sslot * 32 + 4 * w);
    const float2* par = src.kpar + ((size_t)h * (cap >> 6) + ((base_slot + old) >> 6)) * 64 + 8 * w;
    dequant8(word, par, x);
  } else if (valid) {
    const uint4 u = *reinterpret_cast<const uint4*>(kstage + ((size_t)h * max_n + (i - kk)) * 64 + 8 * w);
    bf16x8_to_float(u, x);
  }
  float mn[8], mx[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    mn[j] = valid ? x[j] : INFINITY;
    mx[j] = valid ? x[j] : -INFINITY;
  }
  // tokens of a warp: lanes with equal (lane & 7) hold the same channels
#pragma unroll
  for (int o = 8; o < 32; o <<= 1) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      mn[j] = fminf(mn[j], __shfl_xor_sync(0xffffffffu, mn[j], o));
      mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], o));
    }
  }
  if ((tid & 31) < 8) {
#pragma unroll
    for (int j = 0; j < 8; ++j) { s_mn[warp][8 * w + j] = mn[j]; s_mx[warp][8 * w + j] = mx[j]; }
  }
  __syncthreads();
  // one thread per channel finishes the reduction and derives the group's parameters
  if (tid < 64) {
    float a = s_mn[0][tid], b = s_mx[0][tid];
#pragma unroll
    for (int r = 1; r < 16; ++r) { a = fminf(a, s_mn[r][tid]); b = fmaxf(b, s_mx[r][tid]); }
    float sc, inv, z;
    quant_params(a, b, sc, inv, z);
    s_iz[tid] = make_float2(inv, z);
    dst.kpar[dgrp + tid] = make_float2(sc, z);
    if (two) dst2.kpar[dgrp + tid] = make_float2(sc, z);
  }
  __syncthreads();
  uint32_t c[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float2 iz = s_iz[8 * w + j];
    c[j] = valid ? quant_code(x[j], iz.x, iz.y) : 0u;
  }
  if (valid) {
    const uint32_t word = pack8(c);
    *reinterpret_cast<uint32_t*>(dst.k + dslot * 32 + 4 * w) = word;
    if (two) *reinterpret_cast<uint32_t*>(dst2.k + dslot * 32 + 4 * w) = word;
  }
}

// ---------------------------------------------------------------------------
// Survivor gather: rows of value codes (and of bf16 keys/values in 16-bit mode),
// value parameters and origins move from the current buffer set to the other,
// preserving order.  Thread = (head, survivor, 16-byte chunk).
// ---------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(256)
gather_kernel(BufSet src, BufSet dst, int H, int cap, int base_slot, int kk, const int32_t* __restrict__ kept) {
  constexpr int kChunks = (BITS == 4) ? 2 : 8;
  constexpr int kRow = (BITS == 4) ? 32 : 128;
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int ch = (int)(g % kChunks);
  const long long r = g / kChunks;
  if (r >= (long long)H * kk) return;
  const int i = (int)(r % kk);
  const int h = (int)(r / kk);
  const int old = kept ? kept[i] : i;
  const size_t s = (size_t)h * cap + base_slot + old;
  const size_t d = (size_t)h * cap + base_slot + i;
  *reinterpret_cast<uint4*>(dst.v + d * kRow + 16 * ch) = *reinterpret_cast<const uint4*>(src.v + s * kRow + 16 * ch);
  if (BITS == 16)
    *reinterpret_cast<uint4*>(dst.k + d * kRow + 16 * ch) = *reinterpret_cast<const uint4*>(src.k + s * kRow + 16 * ch);
  if (BITS == 4 && ch == 0) dst.vpar[d] = src.vpar[s];
  if (h == 0 && ch == 0) dst.origin[base_slot + i] = src.origin[base_slot + old];
}

cudaError_t launch_pack(xkv_cache* c, int n, int kk, bool identity, bool first, cudaStream_t st) {
  const BufSet src = c->buf[c->cur];
  const BufSet dst = c->buf[c->cur ^ 1];
  const int32_t* kept = identity ? nullptr : c->kept;
  const int H = c->p.n_heads;
  if (c->p.kv_bits == 4) {
    const int base = first ? 0 : c->rest_base;
    const int r_new = kk + n;
    const dim3 grid((r_new + 63) / 64, H);
    cudaError_t e;
    {
      LaunchScope ls(c, XKV_PROF_REGROUP, st);
      regroup_k_kernel<<<grid, 512, 0, st>>>(src, dst, src, first, c->cap, c->p.max_frame_tokens, base, kk,
                                             r_new, kept, c->kstage);
      e = cudaGetLastError();
    }
    if (e != cudaSuccess) return e;
  }
  if (kk > 0) {
    LaunchScope ls(c, XKV_PROF_GATHER, st);
    if (c->p.kv_bits == 4) {
      const long long threads = (long long)H * kk * 2;
      gather_kernel<4><<<(int)((threads + 255) / 256), 256, 0, st>>>(src, dst, H, c->cap, c->rest_base, kk, kept);
    } else {
      const long long threads = (long long)H * kk * 8;
      gather_kernel<16><<<(int)((threads + 255) / 256), 256, 0, st>>>(src, dst, H, c->cap, c->rest_base, kk, kept);
    }
  }
  return cudaGetLastError();
}

}  // namespace xkv
