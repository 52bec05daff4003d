// Cache-maintenance kernels: append (+ per-token value quantisation), pooled
// query, importance scores, top-k selection, key regroup/re-quantisation and the
// survivor gather.  All bandwidth- or latency-bound; fp32 arithmetic whose every
// operation and order is fixed, because it decides integers (kept indices, 4-bit
// codes) that must be reproducible bit for bit.
#include <stdlib.h>

#include <mutex>

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
// Conversion-free forms of Eq. 10 and Eq. 7.  They produce the same fp32 results
// as dequant8 / quant_code whenever their preconditions hold (callers check them
// and take the plain forms otherwise), but use no int<->float conversion or
// round instruction, which issue at a quarter of the fp32 rate.
//
// A 4-bit code q sitting at bit 4i of a word, OR-ed into the mantissa of
// 2^(23-4i), is the float 2^(23-4i) + q.  Subtracting 2^(23-4i) + z (exact for
// integer |z| < 2^22) gives q - z exactly, like float(q) - z.
// ---------------------------------------------------------------------------
constexpr float kZLimit = 4194304.f;     // 2^22
constexpr float kRoundMagic = 12582912.f;  // 1.5 * 2^23: y + magic has rint(y) in its mantissa for |y| < 2^22

__device__ __forceinline__ uint32_t magic_bits(int j) { return 0x4B000000u - (uint32_t)(j >> 1) * 0x02000000u; }
__device__ __forceinline__ float magic_val(int j) { return __uint_as_float(magic_bits(j)); }

// par[j] = (s, magic_val(j) + z) for the 8 channels of the word.
__device__ __forceinline__ void dequant8_magic(uint32_t word, const float2 (&par)[8], float (&x)[8]) {
  const uint32_t hi = word >> 16;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t src = (j & 1) ? hi : word;
    const uint32_t bits = (src & (0xFu << (4 * (j >> 1)))) | magic_bits(j);
    x[j] = __fmul_rn(par[j].x, __fsub_rn(__uint_as_float(bits), par[j].y));
  }
}

// clamp(rint(x * inv) + z, 0, 15) for |x * inv| < 2^21 and integer |z| < 2^22; zadj = int(z) - bits(magic).
__device__ __forceinline__ uint32_t quant_code_magic(float x, float inv, int zadj) {
  const float t = __fadd_rn(__fmul_rn(x, inv), kRoundMagic);
  const int q = (int)__float_as_uint(t) + zadj;
  int r;
  asm("min.relu.s32 %0, %1, 15;" : "=r"(r) : "r"(q));   // max(min(q, 15), 0)
  return (uint32_t)r;
}

// The plain forms as real calls on scalars, so that the rarely taken fallback costs a branch and
// not predicated copies of its instructions in the hot path, and arrays stay in registers.
__device__ __noinline__ float dequant_one_call(uint32_t q, float s, float z) {
  return __fmul_rn(s, __fsub_rn((float)q, z));
}
__device__ __noinline__ uint32_t quant_code_call(float x, float inv, float z) { return quant_code(x, inv, z); }

__device__ __forceinline__ void dequant8_plain(uint32_t word, const float2* par, float (&x)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) x[j] = dequant_one_call((word >> nib_shift(j)) & 0xFu, par[j].x, par[j].y);
}

// ---------------------------------------------------------------------------
// Pooled query, Eq. 2-3, then the row mean that Eq. 5-6 reduce to.
// One CTA per pooled row i; thread (c, hs) builds pooled[h][i][c] for heads
// h = hs, hs+16, ... (sequential sum over the group's tokens, divided by the
// group size); threads with hs == 0 add the heads in order and scale by 1/H.
// The last CTA to finish adds the rows in order and divides by N_pooled.
// Loads are issued in batches ahead of the (ordered) additions.
// ---------------------------------------------------------------------------
constexpr int kPoolRows = 128;   // pooled rows staged in shared memory at a time by the last CTA

__global__ void __launch_bounds__(1024)
pool_q_kernel(const __nv_bfloat16* __restrict__ q, int n, int64_t ts, int64_t hs, int H, int n_special,
              int g, int n_pooled, float* __restrict__ qbar, float* __restrict__ qvec,
              unsigned int* __restrict__ counter) {
  extern __shared__ float s_pooled[];  // [H][64]
  __shared__ float s_rows[kPoolRows * 64];
  __shared__ float s_acc[64];
  __shared__ bool s_last;
  const int i = blockIdx.x;
  const int c = threadIdx.x;   // 0..63
  const int hslot = threadIdx.y;
  int a, b;
  if (i < n_special) { a = i; b = i + 1; }
  else { a = n_special + (i - n_special) * g; b = min(a + g, n); }
  for (int h = hslot; h < H; h += blockDim.y) {
    const __nv_bfloat16* base = q + (int64_t)h * hs + c;
    float acc = 0.f;
    for (int t0 = a; t0 < b; t0 += 16) {
      float x[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) x[u] = (t0 + u < b) ? __bfloat162float(base[(int64_t)(t0 + u) * ts]) : 0.f;
#pragma unroll
      for (int u = 0; u < 16; ++u)
        if (t0 + u < b) acc = (t0 + u == a) ? x[u] : __fadd_rn(acc, x[u]);
    }
    if (i >= n_special) acc = __fdiv_rn(acc, (float)(b - a));
    s_pooled[h * 64 + c] = acc;
  }
  __syncthreads();
  if (hslot == 0) {
    // (reads in batches ahead of the ordered additions)
    float acc = 0.f;
    for (int h0 = 0; h0 < H; h0 += 16) {
      float v[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) v[u] = (h0 + u < H) ? s_pooled[(h0 + u) * 64 + c] : 0.f;
#pragma unroll
      for (int u = 0; u < 16; ++u)
        if (h0 + u < H) acc = (h0 + u == 0) ? v[u] : __fadd_rn(acc, v[u]);
    }
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
    // all threads fetch the rows (one round trip), then one thread per channel adds them in order
    const int tid = threadIdx.y * 64 + threadIdx.x, nthr = blockDim.y * 64;
    for (int r0 = 0; r0 < n_pooled; r0 += kPoolRows) {
      const int rows = min(kPoolRows, n_pooled - r0);
      __syncthreads();
      for (int e = tid; e < rows * 64; e += nthr) s_rows[e] = __ldcg(&qbar[r0 * 64 + e]);
      __syncthreads();
      if (hslot == 0) {
        float acc = (r0 == 0) ? 0.f : s_acc[c];
        for (int q0 = 0; q0 < rows; q0 += 16) {
          float v[16];
#pragma unroll
          for (int u = 0; u < 16; ++u) v[u] = (q0 + u < rows) ? s_rows[(q0 + u) * 64 + c] : 0.f;
#pragma unroll
          for (int u = 0; u < 16; ++u)
            if (q0 + u < rows) acc = (r0 == 0 && q0 + u == 0) ? v[u] : __fadd_rn(acc, v[u]);
        }
        s_acc[c] = acc;
      }
    }
    if (hslot == 0) qvec[c] = __fdiv_rn(s_acc[c], (float)n_pooled);
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
// The words of sixteen heads (4-bit; four 16-byte pieces for 16-bit storage) are fetched ahead of
// their (ordered) use.
// ---------------------------------------------------------------------------
// Unsigned key whose order is the total order of fp32 bit patterns (so that -0 < +0).
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelBins = 4096;          // histogram of the top 12 key bits, filled by the score kernel

// MODE 0: the whole computation.  MODE 1: only Eq. 4, the head means K-bar[i][c] (fp32, exactly the
// value MODE 0 holds at that point) stored to `kbar` -- run beside the attention of the step that
// built the cache.  MODE 2: only Eq. 5-6 from a stored K-bar -- the next step's scoring.  1 + 2
// perform the operations of 0 in the same order, so the scores are the same bits.
template <int BITS, int MODE>
__global__ void __launch_bounds__(512)
score_kernel(BufSet cur, int H, int cap, int rest_base, int r_old, const float* __restrict__ qvec,
             float* __restrict__ scores, unsigned int* __restrict__ hist, int force_plain,
             float* __restrict__ kbar) {
  // Parameters of the CTA's key group.  Fast path: float4 [H][4][8] = (s, magic + z) of channels
  // 8w + 2v and 8w + 2v + 1 at [h][v][w], so that the eight lanes of a quarter-warp read
  // consecutive 16-byte chunks.  Plain path: float2 (s, z) [H][64].
  extern __shared__ __align__(16) float2 s_par[];
  __shared__ float s_w[64];
  const int tid = threadIdx.x;
  const int w = tid & 7;
  const int tok = tid >> 3;
  const int i = blockIdx.x * 64 + tok;          // rest-local index
  const int slot = rest_base + i;
  const int grp = (rest_base >> 6) + blockIdx.x;
  bool plain = false;
  if (BITS == 4 && MODE != 2) {
    int big = force_plain;
    float2 mine[4];                              // H <= 64: at most 8 elements per thread, 4 at a time
    for (int e0 = 0; e0 < H * 64; e0 += 2048) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * 512 + tid;
        mine[u] = make_float2(0.f, 0.f);
        if (e < H * 64) mine[u] = cur.kpar[((size_t)(e >> 6) * (cap >> 6) + grp) * 64 + (e & 63)];
        big |= !(fabsf(mine[u].y) < kZLimit);
      }
      // the layout depends on the path, which the whole CTA has to agree on: H * 64 <= 2048 makes
      // this loop run once for H <= 32; for more heads the parameters are re-read below
      if (e0 == 0 && H * 64 <= 2048) break;
    }
    plain = __syncthreads_or(big) != 0;
    for (int e0 = 0; e0 < H * 64; e0 += 2048) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * 512 + tid;
        if (e < H * 64) {
          float2 sz = mine[u];
          if (H * 64 > 2048) sz = cur.kpar[((size_t)(e >> 6) * (cap >> 6) + grp) * 64 + (e & 63)];
          if (plain) {
            s_par[e] = sz;
          } else {
            const int h = e >> 6, ch = e & 63;
            sz.y = __fadd_rn(magic_val(ch & 7), sz.y);
            // [h][v = (ch & 7) >> 1][w = ch >> 3], two float2 per float4
            s_par[((h * 4 + ((ch & 7) >> 1)) * 8 + (ch >> 3)) * 2 + (ch & 1)] = sz;
          }
        }
      }
    }
  }
  if (MODE != 1 && tid < 64) s_w[tid] = qvec[tid];
  __syncthreads();
  const bool valid = i < r_old;
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  constexpr int kHB = (BITS == 4) ? 16 : 4;     // heads whose words are in flight together
  for (int h0 = 0; MODE != 2 && h0 < H; h0 += kHB) {
    uint32_t word[BITS == 4 ? kHB : 1];
    uint4 wide[BITS == 4 ? 1 : kHB];
#pragma unroll
    for (int u = 0; u < kHB; ++u) {
      const int h = h0 + u;
      if (BITS == 4) word[u] = 0u; else wide[u] = make_uint4(0, 0, 0, 0);
      if (valid && h < H) {
        if (BITS == 4) word[u] = *reinterpret_cast<const uint32_t*>(cur.k + ((size_t)h * cap + slot) * 32 + 4 * w);
        else wide[u] = *reinterpret_cast<const uint4*>(cur.k + ((size_t)h * cap + slot) * 128 + 16 * w);
      }
    }
#pragma unroll
    for (int u = 0; u < kHB; ++u) {
      const int h = h0 + u;
      if (h < H) {
        float x[8];
        if (BITS == 4) {
          if (plain) {
            dequant8_plain(word[BITS == 4 ? u : 0], s_par + h * 64 + 8 * w, x);
          } else {
            float2 par[8];
            const float4* pp = reinterpret_cast<const float4*>(s_par) + h * 32 + w;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              const float4 t = pp[v * 8];
              par[2 * v] = make_float2(t.x, t.y);
              par[2 * v + 1] = make_float2(t.z, t.w);
            }
            dequant8_magic(word[BITS == 4 ? u : 0], par, x);
          }
        } else {
          bf16x8_to_float(wide[BITS == 4 ? 0 : u], x);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = (h == 0) ? x[j] : __fadd_rn(acc[j], x[j]);
      }
    }
  }
  const float inv_h = __fdiv_rn(1.f, (float)H);
  float kb[8];
  if (MODE == 2) {
    const float4* src = reinterpret_cast<const float4*>(kbar + (size_t)(valid ? i : 0) * 64 + 8 * w);
    const float4 x = src[0], y = src[1];
    kb[0] = x.x; kb[1] = x.y; kb[2] = x.z; kb[3] = x.w; kb[4] = y.x; kb[5] = y.y; kb[6] = y.z; kb[7] = y.w;
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) kb[j] = __fmul_rn(acc[j], inv_h);
  }
  if (MODE == 1) {
    if (valid) {
      float4* dst = reinterpret_cast<float4*>(kbar + (size_t)i * 64 + 8 * w);
      dst[0] = make_float4(kb[0], kb[1], kb[2], kb[3]);
      dst[1] = make_float4(kb[4], kb[5], kb[6], kb[7]);
    }
    return;
  }
  float p[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) p[j] = __fmul_rn(kb[j], s_w[8 * w + j]);
  float t0 = __fadd_rn(p[0], p[1]), t1 = __fadd_rn(p[2], p[3]);
  float t2 = __fadd_rn(p[4], p[5]), t3 = __fadd_rn(p[6], p[7]);
  t0 = __fadd_rn(t0, t1);
  t2 = __fadd_rn(t2, t3);
  float s = __fadd_rn(t0, t2);
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
  if (valid && w == 0) {
    scores[i] = s;
    atomicAdd(&hist[order_key(s) >> 20], 1u);      // first digit of the selection (the select kernel clears it)
  }
}

cudaError_t launch_score(xkv_cache* c, int r_old, cudaStream_t st, bool from_kbar) {
  const int blocks = (r_old + 63) / 64;
  const size_t smem = (size_t)c->p.n_heads * 64 * sizeof(float2);
  LaunchScope ls(c, XKV_PROF_SCORE, st);
  const BufSet& b = c->buf[c->cur];
  const int H = c->p.n_heads;
  if (from_kbar) {
    if (c->p.kv_bits == 16)
      score_kernel<16, 2><<<blocks, 512, smem, st>>>(b, H, c->cap, c->rest_base, r_old, c->qvec, c->scores, c->sel_hist,
                                                     c->force_plain, c->kbar);
    else
      score_kernel<4, 2><<<blocks, 512, smem, st>>>(b, H, c->cap, c->rest_base, r_old, c->qvec, c->scores, c->sel_hist,
                                                    c->force_plain, c->kbar);
  } else if (c->p.kv_bits == 16) {
    score_kernel<16, 0><<<blocks, 512, smem, st>>>(b, H, c->cap, c->rest_base, r_old, c->qvec, c->scores, c->sel_hist,
                                                   c->force_plain, nullptr);
  } else {
    score_kernel<4, 0><<<blocks, 512, smem, st>>>(b, H, c->cap, c->rest_base, r_old, c->qvec, c->scores, c->sel_hist,
                                                  c->force_plain, nullptr);
  }
  return cudaGetLastError();
}

// Head means of the keys after the first frame, of the cache as it stands (after kv_quant_pack).
cudaError_t launch_kbar(xkv_cache* c, cudaStream_t st) {
  const int r = c->T - c->T_first;
  if (r <= 0) return cudaSuccess;
  const int blocks = (r + 63) / 64;
  const size_t smem = (size_t)c->p.n_heads * 64 * sizeof(float2);
  LaunchScope ls(c, XKV_PROF_KBAR, st);
  const BufSet& b = c->buf[c->cur];
  if (c->p.kv_bits == 16)
    score_kernel<16, 1><<<blocks, 512, smem, st>>>(b, c->p.n_heads, c->cap, c->rest_base, r, nullptr, nullptr, nullptr,
                                                   c->force_plain, c->kbar);
  else
    score_kernel<4, 1><<<blocks, 512, smem, st>>>(b, c->p.n_heads, c->cap, c->rest_base, r, nullptr, nullptr, nullptr,
                                                  c->force_plain, c->kbar);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Top-k of the scores (Sec. 3.2).  One CTA.  The order keys are held in shared
// memory when they fit.  The k-th largest key tau is found in two stages: the
// histogram of the top 12 bits (counted by the score kernel with global atomics)
// gives the bin that holds it; the keys of that bin, normally a few hundred, are
// collected and the remaining 20 bits are found by bisection on them.  Then a
// stable compaction keeps every key above tau and the first (k - #above) keys
// equal to it.  Each thread owns a run of consecutive positions.
// ---------------------------------------------------------------------------
constexpr int kSelThreads = 1024;
constexpr int kSelSmemKeys = 44 * 1024;   // keys held in shared memory (176 KB)
constexpr int kSelCand = 4096;            // candidates collected from the bin of tau

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

// sum of v over the block (all threads get it); s_acc must be zero on entry and is zero on exit
__device__ __forceinline__ unsigned int block_sum(unsigned int v, unsigned int* s_acc) {
  v = __reduce_add_sync(0xffffffffu, v);
  if ((threadIdx.x & 31) == 0 && v) atomicAdd(s_acc, v);
  __syncthreads();
  const unsigned int t = *s_acc;
  __syncthreads();
  if (threadIdx.x == 0) *s_acc = 0u;
  return t;
}

// KPT > 0: every thread's run has at most KPT keys and is held in registers after the first read.
template <bool IN_SMEM, int KPT>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int tp, int k, int32_t* __restrict__ kept,
              unsigned int* __restrict__ hist) {
  extern __shared__ uint32_t s_keys[];
  __shared__ uint32_t s_cand[kSelCand];
  __shared__ unsigned int s_warp[33];
  __shared__ unsigned int s_bin, s_need, s_ncand, s_acc;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  // ---- stage 1: the bin of tau from the 12-bit histogram (thread t owns 4 bins counted from the top) ----
  unsigned int hb[4], own = 0u;
  {
    const uint4 h4 = *reinterpret_cast<const uint4*>(hist + kSelBins - 4 - 4 * tid);   // bins 4095-4t-3 .. 4095-4t
    hb[0] = h4.w; hb[1] = h4.z; hb[2] = h4.y; hb[3] = h4.x;
  }
  if (IN_SMEM)
    for (int j = tid; j < tp; j += kSelThreads) s_keys[j] = order_key(scores[j]);
  if (tid == 0) { s_ncand = 0u; s_acc = 0u; }
  auto key_at = [&](int j) -> uint32_t { return IN_SMEM ? s_keys[j] : order_key(scores[j]); };
  *reinterpret_cast<uint4*>(hist + kSelBins - 4 - 4 * tid) = make_uint4(0u, 0u, 0u, 0u);   // ready for the next evicting step
#pragma unroll
  for (int u = 0; u < 4; ++u) own += hb[u];
  unsigned int total;
  unsigned int above = block_excl_scan(own, s_warp, total);   // keys in higher bins than this thread's
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (above < (unsigned int)k && (unsigned int)k <= above + hb[u]) {
      s_bin = (unsigned int)(kSelBins - 1 - (4 * tid + u));
      s_need = (unsigned int)k - above;
    }
    above += hb[u];
  }
  __syncthreads();
  const uint32_t bin = s_bin;
  const unsigned int need = s_need;                  // tau is the need-th largest key of its bin

  // ---- stage 2: collect the keys of that bin (each thread scans its run; a block scan places them) ----
  const int ipt = ((tp + kSelThreads - 1) / kSelThreads) | 1;   // odd run length: a warp's runs on different banks
  const int j0 = min(tid * ipt, tp), j1 = min(j0 + ipt, tp);
  constexpr int kR = KPT > 0 ? KPT : 1;
  uint32_t kr[kR];                                   // this thread's run (KPT > 0)
  if (KPT > 0) {
#pragma unroll
    for (int i = 0; i < kR; ++i) kr[i] = (j0 + i < j1) ? key_at(j0 + i) : 0u;
  }
  // key i of the run: from registers when the loop over i is unrolled, else from memory
#define XKV_RUN_LOOP(BODY)                                                              \
  if (KPT > 0) {                                                                        \
    _Pragma("unroll") for (int i = 0; i < kR; ++i) if (j0 + i < j1) { const int j = j0 + i; const uint32_t key = kr[i]; BODY } \
  } else {                                                                              \
    for (int j = j0; j < j1; ++j) { const uint32_t key = key_at(j); BODY }              \
  }
  unsigned int mine_n = 0u;
  XKV_RUN_LOOP({ (void)j; mine_n += ((key >> 20) == bin); })
  unsigned int ncand;
  unsigned int at = block_excl_scan(mine_n, s_warp, ncand);
  if (mine_n) {
    XKV_RUN_LOOP({ (void)j; if ((key >> 20) == bin) { if (at < (unsigned int)kSelCand) s_cand[at] = key; ++at; } })
  }
  __syncthreads();

  // ---- stage 3: the low 20 bits of tau by bisection on the candidates ----
  uint32_t prefix = bin << 20;
  unsigned int n_gt;                                 // candidates above tau
  if (ncand <= (unsigned int)kSelThreads) {
    const bool has = (unsigned int)tid < ncand;
    const uint32_t mine = has ? s_cand[tid] : 0u;
    for (int bit = 19; bit >= 0; --bit) {
      const uint32_t trial = prefix | (1u << bit);
      if ((unsigned int)__syncthreads_count(has && mine >= trial) >= need) prefix = trial;
    }
    n_gt = (unsigned int)__syncthreads_count(has && mine > prefix);
  } else {
    // rare (many equal or nearly equal scores): the same bisection over a list that does not fit
    // one candidate per thread, or over all keys of the bin when it overflowed the list
    const bool listed = ncand <= (unsigned int)kSelCand;
    auto count = [&](uint32_t trial, bool strict) -> unsigned int {
      unsigned int c = 0u;
      if (listed) {
        for (unsigned int i = tid; i < ncand; i += kSelThreads) c += strict ? (s_cand[i] > trial) : (s_cand[i] >= trial);
      } else {
        XKV_RUN_LOOP({ (void)j; if ((key >> 20) == bin) c += strict ? (key > trial) : (key >= trial); })
      }
      return block_sum(c, &s_acc);
    };
    for (int bit = 19; bit >= 0; --bit) {
      const uint32_t trial = prefix | (1u << bit);
      if (count(trial, false) >= need) prefix = trial;
    }
    n_gt = count(prefix, true);
  }
  const uint32_t tau = prefix;
  const unsigned int need_eq = need - n_gt;          // keys equal to tau that are kept (lowest positions)

  // ---- stage 4: stable compaction ----
  unsigned int cnt_eq = 0u, cnt_gt = 0u;
  XKV_RUN_LOOP({ (void)j; cnt_eq += (key == tau); cnt_gt += (key > tau); })
  const unsigned int eq_before = block_excl_scan(cnt_eq, s_warp, total);
  unsigned int take_eq = 0u;
  if (eq_before < need_eq) take_eq = min(cnt_eq, need_eq - eq_before);
  unsigned int out = block_excl_scan(cnt_gt + take_eq, s_warp, total);
  // The kept positions are listed in shared memory first (in the key array: a thread's keep flags
  // are taken before anything is overwritten) and copied out in full lines; written from the
  // runs directly, every store of a warp would touch 32 different sectors.
  unsigned int flags = 0u;                           // runs longer than 32 keys take the direct route
  const bool staged = IN_SMEM && ipt <= 32;
  if (staged) {
    XKV_RUN_LOOP({
      bool keep = key > tau;
      if (key == tau && take_eq > 0u) { keep = true; --take_eq; }
      flags |= (keep ? 1u : 0u) << (j - j0);
    })
    __syncthreads();
    int32_t* s_out = reinterpret_cast<int32_t*>(s_keys);
    if (KPT > 0) {
#pragma unroll
      for (int i = 0; i < kR; ++i)
        if ((flags >> i) & 1u) s_out[out++] = j0 + i;
    } else {
      for (int j = j0; j < j1; ++j)
        if ((flags >> (j - j0)) & 1u) s_out[out++] = j;
    }
    __syncthreads();
    for (int i = tid; i < k; i += kSelThreads) kept[i] = s_out[i];
  } else {
    XKV_RUN_LOOP({
      bool keep = key > tau;
      if (key == tau && take_eq > 0u) { keep = true; --take_eq; }
      if (keep) kept[out++] = j;
    })
  }
#undef XKV_RUN_LOOP
}

cudaError_t launch_select(xkv_cache* c, int r_old, int k, cudaStream_t st) {
  {
    // opt-in to large dynamic shared memory: a per-device function attribute, set once per device
    static std::mutex mu;
    static bool attr_set[64] = {false};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set[dev]) {
      e = cudaFuncSetAttribute(select_kernel<true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kSelSmemKeys * (int)sizeof(uint32_t));
      if (e != cudaSuccess) return e;
      e = cudaFuncSetAttribute(select_kernel<true, 17>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kSelSmemKeys * (int)sizeof(uint32_t));
      if (e != cudaSuccess) return e;
      attr_set[dev] = true;
    }
  }
  LaunchScope ls(c, XKV_PROF_SELECT, st);
  const size_t smem = (size_t)r_old * sizeof(uint32_t);
  const int ipt = ((r_old + kSelThreads - 1) / kSelThreads) | 1;
  if (r_old > kSelSmemKeys)
    select_kernel<false, 0><<<1, kSelThreads, 0, st>>>(c->scores, r_old, k, c->kept, c->sel_hist);
  else if (ipt <= 17)
    select_kernel<true, 17><<<1, kSelThreads, smem, st>>>(c->scores, r_old, k, c->kept, c->sel_hist);
  else
    select_kernel<true, 0><<<1, kSelThreads, smem, st>>>(c->scores, r_old, k, c->kept, c->sel_hist);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// kv_quant_pack, 4-bit.  One CTA per (new 64-slot key group, four heads); 128
// threads per head, thread = (8-channel word, four tokens 16 apart).
// Keys: survivors are dequantised with the parameters of the group they came
// from (Eq. 10), new keys come from the bf16 staging buffer; per-channel min/max
// over the group's tokens; new parameters and codes (Eq. 7-8).  A complete group
// whose 64 tokens all survive in place is copied.
// Values: the survivors' code rows and parameters, and the origins, move to
// their new slots in the other buffer set (they were quantised on arrival).
// ---------------------------------------------------------------------------
constexpr int kRgHeads = 4;

__global__ void __launch_bounds__(128 * kRgHeads, 2)
regroup_k_kernel(BufSet src, BufSet dst, BufSet dst2, bool two, int H, int cap, int max_n, int base_slot, int kk,
                 int r_new, const int32_t* __restrict__ kept, const __nv_bfloat16* __restrict__ kstage,
                 int force_plain) {
  __shared__ int s_old[64];                      // source position (rest-local) of each token, -1 = new key
  __shared__ float s_mn[kRgHeads][4][64];
  __shared__ float s_mx[kRgHeads][4][64];
  __shared__ float2 s_iz[kRgHeads][64];
  const int tid = threadIdx.x;
  const int gamma = blockIdx.x;
  const int hl = tid >> 7;                       // head within the CTA
  const int h = blockIdx.y * kRgHeads + hl;
  const int t = tid & 127;
  const int w = t & 7;
  const int tq = t >> 3;                         // tokens tq + 16 u
  const int wih = t >> 5;                        // warp within the head
  const bool head_ok = h < H;
  if (tid < 64) {
    const int i = gamma * 64 + tid;
    s_old[tid] = (i < kk) ? (kept ? kept[i] : i) : -1;
  }
  __syncthreads();

  // ---- values, parameters and origins of the survivors (first frame: nothing to move) ----
  if (kk > 0) {
    for (int e = tid; e < kRgHeads * 64 * 2; e += 128 * kRgHeads) {
      const int half = e & 1, tok = (e >> 1) & 63, hh = blockIdx.y * kRgHeads + (e >> 7);
      const int i = gamma * 64 + tok;
      if (hh < H && i < kk) {
        const size_t s_slot = (size_t)hh * cap + base_slot + s_old[tok];
        const size_t d_slot = (size_t)hh * cap + base_slot + i;
        *reinterpret_cast<uint4*>(dst.v + d_slot * 32 + 16 * half) =
            *reinterpret_cast<const uint4*>(src.v + s_slot * 32 + 16 * half);
        if (half == 0) dst.vpar[d_slot] = src.vpar[s_slot];
      }
    }
    if (blockIdx.y == 0 && tid < 64) {
      const int i = gamma * 64 + tid;
      if (i < kk) dst.origin[base_slot + i] = src.origin[base_slot + s_old[tid]];
    }
  }

  // ---- keys ----
  const int last = gamma * 64 + 63;
  const bool carried = (last < kk) && (s_old[63] == last);
  const size_t dgrp = ((size_t)h * (cap >> 6) + (base_slot >> 6) + gamma) * 64;
  if (carried) {
    if (head_ok) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const size_t dslot = (size_t)h * cap + base_slot + gamma * 64 + tq + 16 * u;
        const uint32_t word = *reinterpret_cast<const uint32_t*>(src.k + dslot * 32 + 4 * w);
        *reinterpret_cast<uint32_t*>(dst.k + dslot * 32 + 4 * w) = word;
        if (two) *reinterpret_cast<uint32_t*>(dst2.k + dslot * 32 + 4 * w) = word;
      }
      if (t < 64) {
        const float2 sz = src.kpar[dgrp + t];
        dst.kpar[dgrp + t] = sz;
        if (two) dst2.kpar[dgrp + t] = sz;
      }
    }
    return;
  }
  float x[4][8];
  uint32_t word[4];
  uint4 fresh[4];
  int old[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int tok = tq + 16 * u;
    const int i = gamma * 64 + tok;
    old[u] = (i < r_new) ? s_old[tok] : -2;      // -2: beyond the segment
    word[u] = 0u;
    fresh[u] = make_uint4(0, 0, 0, 0);
    if (head_ok && old[u] >= 0)
      word[u] = *reinterpret_cast<const uint32_t*>(src.k + ((size_t)h * cap + base_slot + old[u]) * 32 + 4 * w);
    else if (head_ok && old[u] == -1)
      fresh[u] = *reinterpret_cast<const uint4*>(kstage + ((size_t)h * max_n + (i - kk)) * 64 + 8 * w);
  }
  int par_grp = -1;
  float2 par[8];
  bool par_plain = false;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (old[u] >= 0) {
      const int g = (base_slot + old[u]) >> 6;
      if (g != par_grp && head_ok) {
        const float4* pp = reinterpret_cast<const float4*>(src.kpar + ((size_t)h * (cap >> 6) + g) * 64 + 8 * w);
        float zmax = 0.f;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const float4 q4 = __ldg(pp + v);
          par[2 * v] = make_float2(q4.x, q4.y);
          par[2 * v + 1] = make_float2(q4.z, q4.w);
          zmax = fmaxf(zmax, fmaxf(fabsf(q4.y), fabsf(q4.w)));
        }
        par_plain = !(zmax < kZLimit) || force_plain;
        if (!par_plain) {
#pragma unroll
          for (int j = 0; j < 8; ++j) par[j].y = __fadd_rn(magic_val(j), par[j].y);
        }
        par_grp = g;
      }
      if (par_plain) dequant8_plain(word[u], par, x[u]);
      else dequant8_magic(word[u], par, x[u]);
    } else {
      bf16x8_to_float(fresh[u], x[u]);
    }
  }
  float mn[8], mx[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) { mn[j] = INFINITY; mx[j] = -INFINITY; }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (old[u] != -2) {
#pragma unroll
      for (int j = 0; j < 8; ++j) { mn[j] = fminf(mn[j], x[u][j]); mx[j] = fmaxf(mx[j], x[u][j]); }
    }
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
  if ((t & 31) < 8) {
#pragma unroll
    for (int j = 0; j < 8; ++j) { s_mn[hl][wih][8 * w + j] = mn[j]; s_mx[hl][wih][8 * w + j] = mx[j]; }
  }
  __syncthreads();
  // one thread per channel finishes the reduction and derives the group's parameters
  int slow = force_plain;
  if (t < 64) {
    float a = s_mn[hl][0][t], b = s_mx[hl][0][t];
#pragma unroll
    for (int r = 1; r < 4; ++r) { a = fminf(a, s_mn[hl][r][t]); b = fmaxf(b, s_mx[hl][r][t]); }
    float sc, inv, z;
    quant_params(a, b, sc, inv, z);
    s_iz[hl][t] = make_float2(inv, z);
    if (head_ok) {
      dst.kpar[dgrp + t] = make_float2(sc, z);
      if (two) dst2.kpar[dgrp + t] = make_float2(sc, z);
      // the conversion-free quantiser needs |x * inv| < 2^21 and |z| < 2^22
      const float ymax = __fmul_rn(fmaxf(fabsf(a), fabsf(b)), inv);
      slow |= !(ymax < 2097152.f) || !(fabsf(z) < kZLimit);
    }
  }
  slow = __syncthreads_or(slow);
  if (!head_ok) return;
  float2 iz[8];
  int zadj[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    iz[j] = s_iz[hl][8 * w + j];
    zadj[j] = slow ? 0 : (int)iz[j].y - (int)0x4B400000;
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (old[u] == -2) continue;
    uint32_t packed;
    if (slow) {
      packed = 0u;
#pragma unroll
      for (int j = 0; j < 8; ++j) packed |= quant_code_call(x[u][j], iz[j].x, iz[j].y) << nib_shift(j);
    } else {
      packed = 0u;
#pragma unroll
      for (int j = 0; j < 8; ++j)   // the nibbles do not overlap: multiply-add places them
        packed = quant_code_magic(x[u][j], iz[j].x, zadj[j]) * (1u << nib_shift(j)) + packed;
    }
    const size_t dslot = (size_t)h * cap + base_slot + gamma * 64 + tq + 16 * u;
    *reinterpret_cast<uint32_t*>(dst.k + dslot * 32 + 4 * w) = packed;
    if (two) *reinterpret_cast<uint32_t*>(dst2.k + dslot * 32 + 4 * w) = packed;
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
    // one kernel: key regroup + survivor gather of values, value parameters and origins
    const int base = first ? 0 : c->rest_base;
    const int r_new = kk + n;
    const dim3 grid((r_new + 63) / 64, (H + kRgHeads - 1) / kRgHeads);
    LaunchScope ls(c, XKV_PROF_REGROUP, st);
    regroup_k_kernel<<<grid, 128 * kRgHeads, 0, st>>>(src, dst, src, first, H, c->cap, c->p.max_frame_tokens, base,
                                                     kk, r_new, kept, c->kstage, c->force_plain);
    return cudaGetLastError();
  }
  if (kk > 0) {
    LaunchScope ls(c, XKV_PROF_GATHER, st);
    const long long threads = (long long)H * kk * 8;
    gather_kernel<16><<<(int)((threads + 255) / 256), 256, 0, st>>>(src, dst, H, c->cap, c->rest_base, kk, kept);
  }
  return cudaGetLastError();
}

}  // namespace xkv
