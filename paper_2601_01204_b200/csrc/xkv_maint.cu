// Cache maintenance: append (+ per-token value quantisation), pooled query,
// importance scores, top-k selection, key regroup / re-quantisation and the
// survivor gather.  All bandwidth- or latency-bound; fp32 arithmetic whose every
// operation and order is fixed, because it decides integers (kept indices, 4-bit
// codes) that must be reproducible bit for bit.
//
// One persistent kernel, launched cooperatively with two thread blocks per SM,
// runs the phases that a call needs, separated by grid-wide barriers:
//
//   APPEND  values quantised per token (Eq. 7-9) into their final slot; keys staged
//           (4-bit) or copied (16-bit)                                 [kv_append]
//   POOL    pooled query rows, Eq. 2-3                                 [kv_score_evict]
//   KBAR    head means of the cached keys after the first frame, Eq. 4, when the
//           stored ones are stale
//   ---- barrier ----
//   SCORE   row mean of the pooled query, scores S = w . K-bar (Eq. 5-6), histogram
//           of the top 12 bits of the score keys
//   ---- barrier ----
//   SEL1    every block finds the histogram bin that holds the k-th largest key;
//           keys in higher bins are kept, keys in that bin become candidates
//   ---- barrier ----
//   SEL2    every block finds the k-th largest (key, position) among the candidates
//           by bisection and writes the kept positions of its own tokens in order
//   ---- barrier ----
//   PACK    16-bit caches: the survivor gather                          [kv_quant_pack]
//
// xkv_stream_step runs all of them in one launch; the per-call entry points launch
// the same kernel with the phases of that call.  The 4-bit kv_quant_pack (key regroup +
// re-quantisation, Eq. 7-9, fused with the survivor gather) is a kernel of its own,
// launched right behind.
#include <stdlib.h>

#include <mutex>

#include "xkv_internal.cuh"

namespace xkv {

namespace {

constexpr int kMT = 512;                 // threads per block
constexpr int kBlocksPerSM = 2;
constexpr uint32_t kBarSpin = 1u << 21;  // polls of a grid barrier before it gives up (about 0.1 s)

// ---------------------------------------------------------------------------
// Eq. 7-8, fixed-order fp32:  s = (max-min)/(2^b - 1) (1 if the range is 0),
// inv = 1/s, z = rint(-min*inv) + 0, q = clamp(rint(x*inv) + z, 0, 2^b - 1).  qmax = 2^b - 1.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void quant_params(float mn, float mx, float& s, float& inv, float& z, float qmax = 15.f) {
  const float r = __fsub_rn(mx, mn);
  s = (r == 0.f) ? 1.f : __fdiv_rn(r, qmax);
  inv = __fdiv_rn(1.f, s);
  z = __fadd_rn(rintf(__fmul_rn(-mn, inv)), 0.f);
}

__device__ __forceinline__ uint32_t quant_code(float x, float inv, float z, float qmax = 15.f) {
  float q = __fadd_rn(rintf(__fmul_rn(x, inv)), z);
  q = fminf(fmaxf(q, 0.f), qmax);
  return (uint32_t)q;
}

// 8-bit storage: the codes of channels 4i..4i+3 form the word c0 | c2<<8 | c1<<16 | c3<<24, so that
// the mask 0x00FF00FF yields the adjacent channels (0, 1) and, after a shift by 8, (2, 3).
__device__ __forceinline__ uint32_t pack4_bytes(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3) {
  return c0 | (c2 << 8) | (c1 << 16) | (c3 << 24);
}
__device__ __forceinline__ void unpack8_bytes(uint2 w, uint32_t (&c)[8]) {
  c[0] = w.x & 0xFFu; c[2] = (w.x >> 8) & 0xFFu; c[1] = (w.x >> 16) & 0xFFu; c[3] = w.x >> 24;
  c[4] = w.y & 0xFFu; c[6] = (w.y >> 8) & 0xFFu; c[5] = (w.y >> 16) & 0xFFu; c[7] = w.y >> 24;
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

// ---------------------------------------------------------------------------
// Conversion-free forms of Eq. 10 and Eq. 7.  They produce the same fp32 results
// as the plain forms whenever their preconditions hold (callers check them and
// take the plain forms otherwise), but use no int<->float conversion or round
// instruction, which issue at a quarter of the fp32 rate.
//
// A 4-bit code q sitting at bit 4i of a word, OR-ed into the mantissa of
// 2^(23-4i), is the float 2^(23-4i) + q.  Subtracting 2^(23-4i) + z (exact for
// integer |z| < 2^22) gives q - z exactly, like float(q) - z.
// ---------------------------------------------------------------------------
constexpr float kZLimit = 4194304.f;       // 2^22
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

// Two fp32 numbers in one 64-bit register and the packed forms of the IEEE operations (each half
// is rounded exactly like the scalar operation, so results do not change; one instruction does two).
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpk2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// dequant8_magic on channel pairs: s2[p] = (s of channel 2p, s of channel 2p + 1), mz2[p] the same
// for magic + z.
__device__ __forceinline__ void dequant8_magic2(uint32_t word, const uint64_t (&s2)[4], const uint64_t (&mz2)[4],
                                                float (&x)[8]) {
  const uint32_t hi = word >> 16;
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const uint32_t be = (word & (0xFu << (4 * p))) | magic_bits(2 * p);
    const uint32_t bo = (hi & (0xFu << (4 * p))) | magic_bits(2 * p);
    unpk2(mul2(s2[p], sub2(pk2(__uint_as_float(be), __uint_as_float(bo)), mz2[p])), x[2 * p], x[2 * p + 1]);
  }
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

// Unsigned key whose order is the total order of fp32 bit patterns (so that -0 < +0).
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const unsigned int* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

constexpr int kSelBins = 4096;       // histogram of the top 12 key bits
constexpr int kHistCopies = 4;       // copies of the histogram (a block adds to copy blockIdx mod 4: fewer collisions)
constexpr int kPoolRows = 120;       // pooled rows staged in shared memory at a time
constexpr int kCandSmem = 4096;      // candidates a block holds in shared memory
constexpr int kSubBins = 256;        // second histogram: the next 8 key bits of the candidates
constexpr int kSubList = 512;        // candidates of one sub-bin that a block lists in shared memory

// Shared memory of a block, one phase at a time.
union __align__(16) Smem {
  struct { float pooled[64 * 64]; } pool;                                          // [H <= 64][64]
  struct { float2 par[64 * 64]; } kbar;                                            // [H][64] key parameters of one group
  struct { float w[64]; float rows[kPoolRows * 64]; } score;
  struct { unsigned long long cand[kCandSmem]; unsigned long long list[kSubList]; } sel;   // (key << 32) | ~position
  struct { float mn[4][4][64]; float mx[4][4][64]; float2 iz[4][64]; } kq;          // quantise-once: one key group, 4 heads
};

struct Shared {
  Smem u;
  unsigned int warp[33];
  unsigned int acc;
  unsigned int bin, need;          // result of SEL1, used by SEL2
  unsigned int sub, need2, n_list; // SEL2: the sub-bin of the k-th largest key, its rank there, listed candidates
  float fsum[2];                   // SCORE: block sums of S and S^2
  int abort_flag;
};

__device__ __forceinline__ unsigned int block_excl_scan(unsigned int v, unsigned int* s_warp, unsigned int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;     // 16 warps
  unsigned int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) s_warp[warp] = x;
  __syncthreads();
  if (warp == 0) {
    const unsigned int t = (lane < kMT / 32) ? s_warp[lane] : 0u;
    unsigned int y = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int z = __shfl_up_sync(0xffffffffu, y, o);
      if (lane >= o) y += z;
    }
    s_warp[lane] = y - t;
    if (lane == 31) s_warp[32] = y;
  }
  __syncthreads();
  const unsigned int res = s_warp[warp] + x - v;
  total = s_warp[32];
  __syncthreads();
  return res;
}

// sum of v over the block (all threads get it); *s_acc must be zero on entry and is zero on exit
__device__ __forceinline__ unsigned int block_sum(unsigned int v, unsigned int* s_acc) {
  v = __reduce_add_sync(0xffffffffu, v);
  if ((threadIdx.x & 31) == 0 && v) atomicAdd(s_acc, v);
  __syncthreads();
  const unsigned int t = *s_acc;
  __syncthreads();
  if (threadIdx.x == 0) *s_acc = 0u;
  __syncthreads();
  return t;
}

// Grid-wide barrier.  Every block arrives once per barrier; the counter only grows (the host
// passes the value it had when the kernel was launched).  The wait is bounded: when it runs out
// the block records XKV_E_TIMEOUT and the kernel winds down without touching anything further.
__device__ __forceinline__ bool grid_barrier(const MaintArgs& a, uint32_t& epoch, Shared& sh) {
  __syncthreads();
  if (threadIdx.x == 0 && !sh.abort_flag) {
    __threadfence();
    atomicAdd(a.bar, 1u);
    const uint32_t target = a.bar_base + (epoch + 1u) * gridDim.x;
    uint32_t it = 0;
    while ((int)(ld_acquire_u32(a.bar) - target) < 0) {
      if (++it > kBarSpin) {
        sh.abort_flag = 1;
        atomicExch(a.status, (int)XKV_E_TIMEOUT);
        break;
      }
      __nanosleep(40);
    }
    __threadfence();
  }
  ++epoch;
  __syncthreads();
  return sh.abort_flag == 0;
}

// ---------------------------------------------------------------------------
// APPEND.  Thread = (head, token, 8-channel word).  Values: per-token min/max over
// the 64 channels by xor-shuffle inside the 8-lane group, then codes -> one 32-bit
// word per lane.  Keys: copied to the staging buffer (4-bit) or to their final
// slot (16-bit).
// ---------------------------------------------------------------------------
template <int BITS, bool ONCE>
__device__ __forceinline__ void phase_append(const MaintArgs& a) {
  const long long items = (long long)a.H * a.n * 8;
  const int passes = (int)((items + kMT - 1) / kMT);
  const BufSet& d0 = a.oth;
  const BufSet& d1 = a.cur;
  const bool two = a.first != 0;
  // pass p goes to block G - 1 - (p mod G): the blocks that hold no pooled row start first
  for (int p = (int)gridDim.x - 1 - (int)blockIdx.x; p < passes; p += gridDim.x) {
    const long long g = (long long)p * kMT + threadIdx.x;
    const int w = (int)(g & 7);
    const long long th = g >> 3;
    const bool valid = th < (long long)a.H * a.n;
    const int h = valid ? (int)(th / a.n) : 0;
    const int tok = valid ? (int)(th % a.n) : 0;
    const int64_t src = (int64_t)h * a.hs_kv + (int64_t)tok * a.ts_kv + 8 * w;
    const uint4 kv = *reinterpret_cast<const uint4*>(a.k + src);
    const uint4 vv = *reinterpret_cast<const uint4*>(a.v + src);
    const size_t slot = (size_t)h * a.cap + a.dst_slot + tok;
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
      constexpr float kQmax = (BITS == 8) ? 255.f : 15.f;
      float s, inv, z;
      quant_params(mn, mx, s, inv, z, kQmax);
      uint32_t c[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) c[j] = quant_code(x[j], inv, z, kQmax);
      if (valid) {
        if (BITS == 8) {
          const uint2 words = make_uint2(pack4_bytes(c[0], c[1], c[2], c[3]), pack4_bytes(c[4], c[5], c[6], c[7]));
          *reinterpret_cast<uint2*>(d0.v + slot * 64 + 8 * w) = words;
          if (two) *reinterpret_cast<uint2*>(d1.v + slot * 64 + 8 * w) = words;
        } else {
          const uint32_t word = pack8(c);
          *reinterpret_cast<uint32_t*>(d0.v + slot * 32 + 4 * w) = word;
          if (two) *reinterpret_cast<uint32_t*>(d1.v + slot * 32 + 4 * w) = word;
        }
        if (w == 0) d0.vpar[slot] = make_float2(s, z);
        if (two) {
          if (w == 0) d1.vpar[slot] = make_float2(s, z);
        }
        if (!ONCE) __stcg(reinterpret_cast<uint4*>(a.kstage + ((size_t)h * a.max_n + tok) * 64 + 8 * w), kv);
      }
    }
    if (valid && h == 0 && w == 0) {
      const int32_t o = (a.frame << 16) | tok;
      d0.origin[a.dst_slot + tok] = o;
      if (two) d1.origin[a.dst_slot + tok] = o;
    }
  }
}

// ---------------------------------------------------------------------------
// POOL.  Pooled query, Eq. 2-3.  Block b takes pooled rows b, b + G, ...; thread
// (c, hs) builds pooled[h][i][c] for heads h = hs, hs + 8, ... (sequential sum over
// the group's tokens, divided by the group size); threads with hs == 0 add the
// heads in order and scale by 1/H.  Loads are issued in batches ahead of the
// (ordered) additions.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void phase_pool(const MaintArgs& a, Shared& sh) {
  const int c = threadIdx.x & 63;
  const int hslot = threadIdx.x >> 6;      // 0..7
  for (int i = blockIdx.x; i < a.n_pooled; i += gridDim.x) {
    int ta, tb;
    if (i < a.n_special) { ta = i; tb = i + 1; }
    else { ta = a.n_special + (i - a.n_special) * a.pool_g; tb = min(ta + a.pool_g, a.n_q); }
    // heads h0 and h0 + 8 together: all loads of a batch (2 heads x 16 tokens) are issued before
    // the first (ordered) addition; an index past the group is clamped, its value unused
    for (int h0 = hslot; h0 < a.H; h0 += 16) {
      const bool has1 = h0 + 8 < a.H;
      const __nv_bfloat16* base0 = a.q + (int64_t)h0 * a.hs_q + c;
      const __nv_bfloat16* base1 = a.q + (int64_t)(has1 ? h0 + 8 : h0) * a.hs_q + c;
      float acc0 = 0.f, acc1 = 0.f;
      for (int t0 = ta; t0 < tb; t0 += 16) {
        float x0[16], x1[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int64_t off = (int64_t)min(t0 + u, tb - 1) * a.ts_q;
          x0[u] = __bfloat162float(base0[off]);
          x1[u] = __bfloat162float(base1[off]);
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          if (t0 + u < tb) {
            acc0 = (t0 + u == ta) ? x0[u] : __fadd_rn(acc0, x0[u]);
            acc1 = (t0 + u == ta) ? x1[u] : __fadd_rn(acc1, x1[u]);
          }
        }
      }
      if (i >= a.n_special) {
        acc0 = __fdiv_rn(acc0, (float)(tb - ta));
        acc1 = __fdiv_rn(acc1, (float)(tb - ta));
      }
      sh.u.pool.pooled[h0 * 64 + c] = acc0;
      if (has1) sh.u.pool.pooled[(h0 + 8) * 64 + c] = acc1;
    }
    __syncthreads();
    if (hslot == 0) {
      float acc = 0.f;
      for (int h0 = 0; h0 < a.H; h0 += 16) {
        float v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = (h0 + u < a.H) ? sh.u.pool.pooled[(h0 + u) * 64 + c] : 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u)
          if (h0 + u < a.H) acc = (h0 + u == 0) ? v[u] : __fadd_rn(acc, v[u]);
      }
      const float inv_h = __fdiv_rn(1.f, (float)a.H);
      __stcg(&a.qbar[i * 64 + c], __fmul_rn(acc, inv_h));
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------
// KBAR.  Head means of the keys, Eq. 4, for the rest-local positions [lo, hi) of the
// buffer set `b`: one pass per 64-slot key group (the rest segment starts on a
// 128-slot boundary, so the tokens of a pass share their quantisation parameters).
// Thread = (token, 8-channel word): dequantise the word of every head in order
// (Eq. 10), accumulate the head sum sequentially, scale by 1/H.  The words of
// sixteen heads (4-bit; four 16-byte pieces for 16-bit storage) are fetched ahead
// of their (ordered) use.
// ---------------------------------------------------------------------------
// One run of up to 64 consecutive slots whose keys share their quantisation parameters:
// slot0 = physical slot of the run's first token, i0 = its rest-local position, `count` tokens;
// the parameters of (head h, channel ch) are par[h * par_stride + ch].
template <int BITS>
__device__ __forceinline__ void kbar_run(const MaintArgs& a, Shared& sh, const BufSet& b, const float2* par,
                                         size_t par_stride, int slot0, int i0, int count) {
  const int tid = threadIdx.x;
  const int w = tid & 7;
  const int tok = tid >> 3;
  const int H = a.H, cap = a.cap;
  {
    const int i = i0 + tok;                       // rest-local index
    const int slot = slot0 + tok;
    bool plain = false;
    if (BITS == 4) {
      // Parameters of the key group.  Fast path: float4 [H][4][8] = (s, magic + z) of channels
      // 8w + 2v and 8w + 2v + 1 at [h][v][w], so that the eight lanes of a quarter-warp read
      // consecutive 16-byte chunks.  Plain path: float2 (s, z) [H][64].
      int big = a.force_plain;
      for (int e = tid; e < H * 64; e += kMT) {
        const float2 sz = __ldcg(&par[(size_t)(e >> 6) * par_stride + (e & 63)]);
        big |= !(fabsf(sz.y) < kZLimit);
      }
      plain = __syncthreads_or(big) != 0;
      for (int e = tid; e < H * 64; e += kMT) {
        float2 sz = __ldcg(&par[(size_t)(e >> 6) * par_stride + (e & 63)]);
        if (plain) {
          sh.u.kbar.par[e] = sz;
        } else {
          const int h = e >> 6, ch = e & 63;
          sz.y = __fadd_rn(magic_val(ch & 7), sz.y);
          sh.u.kbar.par[((h * 4 + ((ch & 7) >> 1)) * 8 + (ch >> 3)) * 2 + (ch & 1)] = sz;
        }
      }
      __syncthreads();
    }
    const bool valid = tok < count;
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
    if (BITS == 8) {
      // 8-bit codes: plain Eq. 10 per channel, parameters (s, z) [H][64] in shared memory
      __syncthreads();
      for (int e = tid; e < H * 64; e += kMT) sh.u.kbar.par[e] = __ldcg(&par[(size_t)(e >> 6) * par_stride + (e & 63)]);
      __syncthreads();
      for (int h0 = 0; h0 < H; h0 += 8) {
        uint2 wide8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          wide8[u] = make_uint2(0u, 0u);
          if (valid && h0 + u < H) wide8[u] = __ldcg(reinterpret_cast<const uint2*>(b.k + ((size_t)(h0 + u) * cap + slot) * 64 + 8 * w));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int h = h0 + u;
          if (h < H) {
            uint32_t c[8];
            unpack8_bytes(wide8[u], c);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float2 sz = sh.u.kbar.par[h * 64 + 8 * w + j];
              const float x = __fmul_rn(sz.x, __fsub_rn((float)c[j], sz.y));
              acc[j] = (h == 0) ? x : __fadd_rn(acc[j], x);
            }
          }
        }
      }
    }
    constexpr int kHB = (BITS == 4) ? 16 : 4;     // heads whose words are in flight together
    for (int h0 = 0; BITS != 8 && h0 < H; h0 += kHB) {
      uint32_t word[BITS == 4 ? kHB : 1];
      uint4 wide[BITS == 4 ? 1 : kHB];
#pragma unroll
      for (int u = 0; u < kHB; ++u) {
        const int h = h0 + u;
        if (BITS == 4) word[u] = 0u; else wide[u] = make_uint4(0, 0, 0, 0);
        if (valid && h < H) {
          if (BITS == 4) word[u] = __ldcg(reinterpret_cast<const uint32_t*>(b.k + ((size_t)h * cap + slot) * 32 + 4 * w));
          else wide[u] = __ldcg(reinterpret_cast<const uint4*>(b.k + ((size_t)h * cap + slot) * 128 + 16 * w));
        }
      }
#pragma unroll
      for (int u = 0; u < kHB; ++u) {
        const int h = h0 + u;
        if (h < H) {
          float x[8];
          if (BITS == 4) {
            if (plain) {
              dequant8_plain(word[BITS == 4 ? u : 0], sh.u.kbar.par + h * 64 + 8 * w, x);
            } else {
              float2 par[8];
              const float4* pp = reinterpret_cast<const float4*>(sh.u.kbar.par) + h * 32 + w;
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
    if (valid) {
      float4* dst = reinterpret_cast<float4*>(b.kbar + (size_t)i * 64 + 8 * w);
      __stcg(dst, make_float4(__fmul_rn(acc[0], inv_h), __fmul_rn(acc[1], inv_h), __fmul_rn(acc[2], inv_h),
                              __fmul_rn(acc[3], inv_h)));
      __stcg(dst + 1, make_float4(__fmul_rn(acc[4], inv_h), __fmul_rn(acc[5], inv_h), __fmul_rn(acc[6], inv_h),
                                  __fmul_rn(acc[7], inv_h)));
    }
    __syncthreads();       // the parameter table is rewritten by the next run
  }
}

// KBAR over the rest-local positions [0, hi) of the buffer set `b` (re-quantising mode and 16-bit):
// one run per 64-slot key group (the rest segment starts on a 128-slot boundary).
template <int BITS>
__device__ __forceinline__ void phase_kbar(const MaintArgs& a, Shared& sh, const BufSet& b, int lo, int hi) {
  const int g_lo = lo >> 6, g_hi = (hi + 63) >> 6;
  for (int gb = g_lo + blockIdx.x; gb < g_hi; gb += gridDim.x) {
    const int grp = (a.rest_base >> 6) + gb;
    kbar_run<BITS>(a, sh, b, b.kpar + (size_t)grp * 64, (size_t)(a.cap >> 6) * 64, a.rest_base + gb * 64, gb * 64,
                   min(64, hi - gb * 64));
  }
}

// ---------------------------------------------------------------------------
// Quantise-once mode, APPEND: the frame's keys are quantised here, per channel in groups of 64
// consecutive tokens of the frame (Eq. 7-9), and never again.  Item = (group, four heads); 128
// threads per head, thread = (8-channel word, four tokens 16 apart).  Each group takes a slot
// of the parameter table: fp32 (scale, zero) for the maintenance arithmetic and the constants
// of the attention's fp16 operand path.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

template <int BITS>
__device__ __forceinline__ void phase_quant_keys_once(const MaintArgs& a, Shared& sh) {
  constexpr float kQmax = (BITS == 8) ? 255.f : 15.f;
  const BufSet& d0 = a.oth;
  const BufSet& d1 = a.cur;
  const bool two = a.first != 0;
  const int H = a.H, cap = a.cap, n = a.n;
  const int tid = threadIdx.x;
  const int hl = tid >> 7, t = tid & 127, w = t & 7, tq = t >> 3, wih = t >> 5;
  const int n_groups = (n + 63) >> 6, n_quads = (H + 3) >> 2;
  const int items = n_groups * n_quads;
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int gamma = item / n_quads, quad = item - gamma * n_quads;
    const int h = quad * 4 + hl;
    const bool head_ok = h < H;
    // the group's table slot: the ring of free slots is read at places the host has counted out
    const uint32_t take = a.pop_base + (uint32_t)gamma;
    const int slot = __ldcg(&a.ring[take % (uint32_t)a.n_slots]);
    if (tid == 0 && quad == 0) {
      if ((int)(take - __ldcg(a.push_pos)) >= 0) atomicCAS(a.status, 0, (int)XKV_E_LIMIT);   // the table has run out
      a.ref[slot] = min(64, n - gamma * 64);
    }
    float x[4][8];
    bool live[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int tok = gamma * 64 + tq + 16 * u;
      live[u] = tok < n;
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (live[u] && head_ok) raw = *reinterpret_cast<const uint4*>(a.k + (int64_t)h * a.hs_kv + (int64_t)tok * a.ts_kv + 8 * w);
      bf16x8_to_float(raw, x[u]);
    }
    float mn[8], mx[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { mn[j] = INFINITY; mx[j] = -INFINITY; }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (live[u]) {
#pragma unroll
        for (int j = 0; j < 8; ++j) { mn[j] = fminf(mn[j], x[u][j]); mx[j] = fmaxf(mx[j], x[u][j]); }
      }
    }
#pragma unroll
    for (int o = 8; o < 32; o <<= 1) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        mn[j] = fminf(mn[j], __shfl_xor_sync(0xffffffffu, mn[j], o));
        mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], o));
      }
    }
    __syncthreads();                 // the previous item's parameters have been read
    if ((t & 31) < 8) {
#pragma unroll
      for (int j = 0; j < 8; ++j) { sh.u.kq.mn[hl][wih][8 * w + j] = mn[j]; sh.u.kq.mx[hl][wih][8 * w + j] = mx[j]; }
    }
    __syncthreads();
    if (t < 64) {                    // one thread per channel: the group's parameters (warps 0, 1 of the head)
      float lo = sh.u.kq.mn[hl][0][t], hi = sh.u.kq.mx[hl][0][t];
#pragma unroll
      for (int r = 1; r < 4; ++r) { lo = fminf(lo, sh.u.kq.mn[hl][r][t]); hi = fmaxf(hi, sh.u.kq.mx[hl][r][t]); }
      float sc, inv, z;
      quant_params(lo, hi, sc, inv, z, kQmax);
      sh.u.kq.iz[hl][t] = make_float2(inv, z);
      float zl, zh, cc;
      dequant_consts(sc, z, zl, zh, cc);
      const float zo = (BITS == 4 && (((t & 7) >> 1) & 1)) ? zh : zl;      // 8-bit codes all carry the bias 1024
      // the neighbouring channel's constants: pairs (2p, 2p + 1) share a word
      const float sc1 = __shfl_xor_sync(0xffffffffu, sc, 1), zo1 = __shfl_xor_sync(0xffffffffu, zo, 1);
      const float cc1 = __shfl_xor_sync(0xffffffffu, cc, 1);
      if (head_ok) {
        a.ktab32[((size_t)slot * H + h) * 64 + t] = make_float2(sc, z);
        if ((t & 1) == 0) {
          uint32_t* e = a.ktab16 + (((size_t)slot * H + h) * 8 + (t >> 3)) * 12 + ((t & 7) >> 1);
          e[0] = pack_half2(sc, sc1);
          e[4] = pack_half2(zo, zo1);
          e[8] = pack_half2(cc, cc1);
        }
        if (!(fabsf(sc) * (fabsf(z) + kQmax) <= 65504.f)) atomicCAS(a.status, 0, (int)XKV_E_RANGE);
      }
    }
    __syncthreads();
    if (head_ok) {
      float2 iz[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) iz[j] = sh.u.kq.iz[hl][8 * w + j];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (!live[u]) continue;
        uint32_t c[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) c[j] = quant_code(x[u][j], iz[j].x, iz[j].y, kQmax);
        const size_t dslot = (size_t)h * cap + a.dst_slot + gamma * 64 + tq + 16 * u;
        if (BITS == 8) {
          const uint2 words = make_uint2(pack4_bytes(c[0], c[1], c[2], c[3]), pack4_bytes(c[4], c[5], c[6], c[7]));
          *reinterpret_cast<uint2*>(d0.k + dslot * 64 + 8 * w) = words;
          if (two) *reinterpret_cast<uint2*>(d1.k + dslot * 64 + 8 * w) = words;
        } else {
          const uint32_t word = pack8(c);
          *reinterpret_cast<uint32_t*>(d0.k + dslot * 32 + 4 * w) = word;
          if (two) *reinterpret_cast<uint32_t*>(d1.k + dslot * 32 + 4 * w) = word;
        }
      }
    }
    if (quad == 0 && tid < 64 && gamma * 64 + tid < n) {
      d0.kslot[a.dst_slot + gamma * 64 + tid] = slot;
      if (two) d1.kslot[a.dst_slot + gamma * 64 + tid] = slot;
    }
  }
}

// Quantise-once mode: head means (Eq. 4) of the frame just quantised, into the destination's
// array: one run per arrival group, whose parameters sit in the group's table slot.
template <int BITS>
__device__ __forceinline__ void phase_kbar_new_once(const MaintArgs& a, Shared& sh) {
  const int n_groups = (a.n + 63) >> 6;
  const BufSet& d = a.oth;
  for (int gamma = blockIdx.x; gamma < n_groups; gamma += gridDim.x) {
    const int slot = __ldcg(&d.kslot[a.dst_slot + gamma * 64]);
    kbar_run<BITS>(a, sh, d, a.ktab32 + (size_t)slot * a.H * 64, 64, a.dst_slot + gamma * 64,
                   a.dst_slot - a.rest_base + gamma * 64, min(64, a.n - gamma * 64));
  }
}

// Quantise-once mode, PACK: the survivors' key and value code rows, value parameters, group
// references, origins and head means move to their new places in the other buffer set.
template <int BITS>
__device__ __forceinline__ void phase_gather_once(const MaintArgs& a) {
  constexpr int kRow = (BITS == 8) ? 64 : 32;       // bytes of a code row
  constexpr int kRC = kRow / 16;                    // 16-byte chunks of a row
  const BufSet& src = a.cur;
  const BufSet& dst = a.oth;
  const int32_t* kept = a.identity ? nullptr : a.kept;
  const long long stride = (long long)gridDim.x * kMT;
  const long long first = (long long)blockIdx.x * kMT + threadIdx.x;
  if (a.kk == 0) {
    // the budget leaves no room for the middle (k = 0): every token after the first frame leaves,
    // without a selection; their key groups give their table slots back
    for (long long i = first; i < a.r_old; i += stride) {
      const int slot = __ldcg(&src.kslot[a.rest_base + i]);
      if (atomicSub(&a.ref[slot], 1) == 1) a.ring[atomicAdd(a.push_pos, 1u) % (unsigned int)a.n_slots] = slot;
    }
    return;
  }
  // four items per thread and pass: the kept indices, then the rows, then the stores
  const long long items = (long long)a.H * a.kk * (2 * kRC);         // (head, survivor, 16-byte chunk of K | V codes)
  for (long long g0 = first; g0 < items; g0 += 4 * stride) {
    int old[4]; size_t so[4], dd[4]; int chn[4]; bool ok[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long g = g0 + u * stride;
      ok[u] = g < items;
      chn[u] = (int)(g % (2 * kRC));
      const long long r = ok[u] ? (g / (2 * kRC)) : 0;
      const int i = (int)(r % a.kk), h = (int)(r / a.kk);
      old[u] = kept ? __ldcg(&kept[i]) : i;
      dd[u] = (size_t)h * a.cap + a.rest_base + i;
      so[u] = (size_t)h * a.cap + a.rest_base;
    }
    uint4 row[4]; float2 vp[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const size_t s = so[u] + old[u];
      const uint8_t* base = chn[u] < kRC ? src.k : src.v;
      row[u] = ok[u] ? *reinterpret_cast<const uint4*>(base + s * kRow + 16 * (chn[u] % kRC)) : make_uint4(0, 0, 0, 0);
      vp[u] = (ok[u] && chn[u] == kRC) ? src.vpar[s] : make_float2(0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (!ok[u]) continue;
      uint8_t* base = chn[u] < kRC ? dst.k : dst.v;
      *reinterpret_cast<uint4*>(base + dd[u] * kRow + 16 * (chn[u] % kRC)) = row[u];
      if (chn[u] == kRC) dst.vpar[dd[u]] = vp[u];
    }
  }
  const long long rows = (long long)a.kk * 16;                       // (survivor, 16-byte chunk of its head-mean row)
  for (long long g0 = first; g0 < rows; g0 += 4 * stride) {
    int old[4]; bool ok[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long g = g0 + u * stride;
      ok[u] = g < rows;
      old[u] = ok[u] ? (kept ? __ldcg(&kept[(int)(g >> 4)]) : (int)(g >> 4)) : 0;
    }
    float4 row[4]; int org[4], ks[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long g = g0 + u * stride;
      const int ch = (int)(g & 15);
      row[u] = ok[u] ? __ldcg(reinterpret_cast<const float4*>(src.kbar + (size_t)old[u] * 64) + ch) : make_float4(0, 0, 0, 0);
      org[u] = (ok[u] && ch == 0) ? src.origin[a.rest_base + old[u]] : 0;
      ks[u] = (ok[u] && ch == 0) ? src.kslot[a.rest_base + old[u]] : 0;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long g = g0 + u * stride;
      if (!ok[u]) continue;
      const int ch = (int)(g & 15), i = (int)(g >> 4);
      reinterpret_cast<float4*>(dst.kbar + (size_t)i * 64)[ch] = row[u];
      if (ch == 0) { dst.origin[a.rest_base + i] = org[u]; dst.kslot[a.rest_base + i] = ks[u]; }
    }
  }
}

// ---------------------------------------------------------------------------
// SCORE.  w[c] = (sequential sum of the pooled rows) / N_pooled; S[j] = balanced
// tree over the 64 products w[c] * K-bar[j][c] (three levels inside the lane, three
// by xor-shuffle), Eq. 5-6.  Thread = (token, 8-channel word); block b takes the
// 64-token runs b, b + G, ...
// ---------------------------------------------------------------------------
__device__ __forceinline__ void phase_score(const MaintArgs& a, Shared& sh) {
  const int tid = threadIdx.x;
  const int n_runs = (a.r_old + 63) >> 6;
  if ((int)blockIdx.x >= n_runs && blockIdx.x != 0) return;
  // the pooled rows come through shared memory, 120 at a time (one round trip), and one thread
  // per channel adds them in order -- unless the caller supplied the row mean
  for (int r0 = 0; a.w_in == nullptr && r0 < a.n_pooled; r0 += kPoolRows) {
    const int rows = min(kPoolRows, a.n_pooled - r0);
    __syncthreads();
    for (int e = tid; e < rows * 64; e += kMT) sh.u.score.rows[e] = __ldcg(&a.qbar[r0 * 64 + e]);
    __syncthreads();
    if (tid < 64) {
      float acc = (r0 == 0) ? 0.f : sh.u.score.w[tid];
      for (int q0 = 0; q0 < rows; q0 += 16) {
        float v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = (q0 + u < rows) ? sh.u.score.rows[(q0 + u) * 64 + tid] : 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u)
          if (q0 + u < rows) acc = (r0 == 0 && q0 + u == 0) ? v[u] : __fadd_rn(acc, v[u]);
      }
      sh.u.score.w[tid] = acc;
    }
  }
  if (tid < 64) {
    const float wv = a.w_in ? a.w_in[tid] : __fdiv_rn(sh.u.score.w[tid], (float)a.n_pooled);
    sh.u.score.w[tid] = wv;
    if (blockIdx.x == 0) a.qvec[tid] = wv;
  }
  __syncthreads();
  const int w = tid & 7, tok = tid >> 3;
  float wq[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) wq[j] = sh.u.score.w[8 * w + j];
  for (int run = blockIdx.x; run < n_runs; run += gridDim.x) {
    const int i = run * 64 + tok;
    const bool valid = i < a.r_old;
    const float4* src = reinterpret_cast<const float4*>(a.cur.kbar + (size_t)(valid ? i : 0) * 64 + 8 * w);
    const float4 x = __ldcg(src), y = __ldcg(src + 1);
    const float kb[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
    float p[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) p[j] = __fmul_rn(kb[j], wq[j]);
    float t0 = __fadd_rn(p[0], p[1]), t1 = __fadd_rn(p[2], p[3]);
    float t2 = __fadd_rn(p[4], p[5]), t3 = __fadd_rn(p[6], p[7]);
    t0 = __fadd_rn(t0, t1);
    t2 = __fadd_rn(t2, t3);
    float s = __fadd_rn(t0, t2);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
    if (valid && w == 0) {
      __stcg(&a.scores[i], s);
      atomicAdd(&a.hist[(blockIdx.x & (kHistCopies - 1)) * kSelBins + (order_key(s) >> 20)], 1u);
    }
    // statistics of the scores (for budget policies): block sums, then one atomic per block
    float s1 = (valid && w == 0) ? s : 0.f, s2 = s1 * s1;
#pragma unroll
    for (int o = 8; o < 32; o <<= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
    if ((tid & 31) == 0) { atomicAdd(&sh.fsum[0], s1); atomicAdd(&sh.fsum[1], s2); }
    __syncthreads();
    if (tid == 0) { atomicAdd(&a.stats[0], sh.fsum[0]); atomicAdd(&a.stats[1], sh.fsum[1]); sh.fsum[0] = sh.fsum[1] = 0.f; }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------
// SEL1 / SEL2.  Top-k of the scores (Sec. 3.2), ties to the lower position, i.e.
// the k largest of the unique pairs (key, -position).  Every block that owns tokens
// repeats the global parts (histogram scan, bisection) for itself.
// ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long composite(uint32_t key, int pos) {
  return ((unsigned long long)key << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)pos);
}

__device__ __forceinline__ void phase_sel1(const MaintArgs& a, Shared& sh) {
  const int tid = threadIdx.x;
  const int n_runs = (a.r_old + 63) >> 6;
  if (blockIdx.x == gridDim.x - 1) {                 // the next selecting launch's counter and sub-histogram:
    if (tid == 0) *a.cand_count_next = 0u;           // nobody uses them in this launch
    if (tid < kSubBins) a.hist2_next[tid] = 0u;
    if (tid < 4) a.stats_next[tid] = 0.f;
  }
  if ((int)blockIdx.x >= n_runs) return;
  // thread t owns the bins 4095 - 8t - 7 .. 4095 - 8t; walked from the top
  unsigned int hb[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
  {
    uint4 lo4[kHistCopies], hi4[kHistCopies];
#pragma unroll
    for (int cpy = 0; cpy < kHistCopies; ++cpy) {
      const uint4* hp = reinterpret_cast<const uint4*>(a.hist + cpy * kSelBins + kSelBins - 8 - 8 * tid);
      lo4[cpy] = __ldcg(hp);
      hi4[cpy] = __ldcg(hp + 1);
    }
#pragma unroll
    for (int cpy = 0; cpy < kHistCopies; ++cpy) {
      hb[0] += hi4[cpy].w; hb[1] += hi4[cpy].z; hb[2] += hi4[cpy].y; hb[3] += hi4[cpy].x;
      hb[4] += lo4[cpy].w; hb[5] += lo4[cpy].z; hb[6] += lo4[cpy].y; hb[7] += lo4[cpy].x;
    }
  }
  unsigned int own = 0u;
#pragma unroll
  for (int u = 0; u < 8; ++u) own += hb[u];
  unsigned int total;
  unsigned int above = block_excl_scan(own, sh.warp, total);   // keys in higher bins than this thread's
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    if (above < (unsigned int)a.kk && (unsigned int)a.kk <= above + hb[u]) {
      sh.bin = (unsigned int)(kSelBins - 1 - (8 * tid + u));
      sh.need = (unsigned int)a.kk - above;                       // the k-th largest is the need-th largest of its bin
    }
    above += hb[u];
  }
  __syncthreads();
  const uint32_t bin = sh.bin;
  for (int run = blockIdx.x; run < n_runs; run += gridDim.x) {
    const int i = run * 64 + tid;
    bool hi = false;
    if (tid < 64 && i < a.r_old) {
      const uint32_t key = order_key(__ldcg(&a.scores[i]));
      hi = (key >> 20) > bin;
      if ((key >> 20) == bin) {
        const unsigned int at = atomicAdd(a.cand_count, 1u);
        __stcg(&a.cand[at], composite(key, i));
        atomicAdd(&a.hist2[(key >> 12) & (kSubBins - 1)], 1u);
      }
    }
    const int cnt = __syncthreads_count(hi);
    if (tid == 0) __stcg(&a.run_hi[run], (unsigned int)cnt);
  }
}

template <bool ONCE>
__device__ __forceinline__ void phase_sel2(const MaintArgs& a, Shared& sh) {
  const int tid = threadIdx.x;
  const int n_runs = (a.r_old + 63) >> 6;
  if (blockIdx.x == gridDim.x - 1) {                 // every block has read the histogram: ready for the next step
    for (int e = tid; e < kSelBins * kHistCopies; e += kMT) a.hist[e] = 0u;
  }
  if ((int)blockIdx.x >= n_runs) return;
  const uint32_t bin = sh.bin;
  const unsigned int need = sh.need;
  const unsigned int ncand = __ldcg(a.cand_count);
  const bool in_smem = ncand <= (unsigned int)kCandSmem;
  if (in_smem)
    for (unsigned int e = tid; e < ncand; e += kMT) sh.u.sel.cand[e] = __ldcg(&a.cand[e]);
  __syncthreads();
  auto cand_at = [&](unsigned int e) -> unsigned long long { return in_smem ? sh.u.sel.cand[e] : __ldcg(&a.cand[e]); };
  // the need-th largest candidate: its bin bits are known, the positions lie below 2^pbits
  int pbits = 1;
  while ((1 << pbits) < a.r_old) ++pbits;
  unsigned long long prefix = ((unsigned long long)bin << 52) | (unsigned long long)(0xFFFFFFFFu << pbits);
  // The candidates share the top 12 key bits; a second histogram over their next 8 bits (filled by
  // SEL1) narrows the k-th largest key down to one sub-bin, whose few members are listed and ranked.
  {
    const unsigned int h2 = (tid < kSubBins) ? __ldcg(&a.hist2[kSubBins - 1 - tid]) : 0u;   // thread t: sub-bin 255 - t
    unsigned int total;
    const unsigned int above2 = block_excl_scan(h2, sh.warp, total);
    if (tid == 0) sh.n_list = 0u;
    if (tid < kSubBins && above2 < need && need <= above2 + h2) { sh.sub = kSubBins - 1 - tid; sh.need2 = need - above2; }
    __syncthreads();
  }
  const uint32_t sub = sh.sub;
  const unsigned int need2 = sh.need2;
  if (in_smem) {
    for (unsigned int e = tid; e < ncand; e += kMT) {
      const unsigned long long cv = sh.u.sel.cand[e];
      if ((((uint32_t)(cv >> 32) >> 12) & (kSubBins - 1)) == sub) {
        const unsigned int at = atomicAdd(&sh.n_list, 1u);
        if (at < (unsigned int)kSubList) sh.u.sel.list[at] = cv;
      }
    }
  }
  __syncthreads();
  const unsigned int m = sh.n_list;
  if (in_smem && m <= 32u) {
    // every warp ranks the listed candidates by itself: lane l holds candidate l and counts the
    // larger ones; the one with need2 - 1 larger ones is the k-th largest of all
    const int lane = tid & 31;
    const unsigned long long mine = (unsigned int)lane < m ? sh.u.sel.list[lane] : 0ull;
    unsigned int larger = 0u;
    for (unsigned int j = 0; j < m; ++j) larger += __shfl_sync(0xffffffffu, mine, (int)j) > mine;
    const unsigned int hit = __ballot_sync(0xffffffffu, (unsigned int)lane < m && larger == need2 - 1u);
    prefix = __shfl_sync(0xffffffffu, mine, __ffs(hit) - 1);
  } else {
    // many candidates (many equal or nearly equal scores): the same bisection over the whole
    // 64-bit pair, block-wide, on the list in shared memory or, if it does not fit, in global memory
    for (int bit = 51; bit >= 0; --bit) {
      if (bit < 32 && bit >= pbits) continue;
      const unsigned long long trial = prefix | (1ull << bit);
      unsigned int c = 0u;
      for (unsigned int e = tid; e < ncand; e += kMT) c += cand_at(e) >= trial;
      if (block_sum(c, &sh.acc) >= need) prefix = trial;
    }
  }
  const unsigned long long tau = prefix;             // kept candidates: composite >= tau (exactly `need` of them)
  if (blockIdx.x == 0 && tid == 0) {                 // the k-th largest score itself, for the statistics
    const uint32_t key = (uint32_t)(tau >> 32);
    a.stats[2] = __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
  }
  for (int run = blockIdx.x; run < n_runs; run += gridDim.x) {
    // survivors before this run: the sure keeps of the runs before it plus the kept candidates at
    // lower positions
    unsigned int part = 0u;
    for (int r = tid; r < run; r += kMT) part += __ldcg(&a.run_hi[r]);
    const uint32_t below = 0xFFFFFFFFu - (uint32_t)(run * 64);         // position part of position run * 64
    for (unsigned int e = tid; e < ncand; e += kMT) {
      const unsigned long long cv = cand_at(e);
      part += (cv >= tau) && ((uint32_t)cv > below);                   // larger low word = lower position
    }
    const unsigned int base = block_sum(part, &sh.acc);
    const int i = run * 64 + tid;
    bool keep = false;
    if (tid < 64 && i < a.r_old) {
      const uint32_t key = order_key(__ldcg(&a.scores[i]));
      keep = (key >> 20) > bin || ((key >> 20) == bin && composite(key, i) >= tau);
    }
    if (tid < 64) {
      const unsigned int m = __ballot_sync(0xffffffffu, keep);
      if (tid == 31) sh.warp[0] = __popc(m);
      const unsigned int rank = __popc(m & ((1u << (tid & 31)) - 1u));
      asm volatile("bar.sync 2, 64;" ::: "memory");
      const unsigned int off = (tid >= 32) ? sh.warp[0] : 0u;
      if (keep) __stcg(&a.kept[base + off + rank], i);
      if (ONCE && i < a.r_old && !keep) {
        // the token leaves: its key group loses a member and gives its table slot back when empty
        const int slot = __ldcg(&a.cur.kslot[a.rest_base + i]);
        if (atomicSub(&a.ref[slot], 1) == 1) a.ring[atomicAdd(a.push_pos, 1u) % (unsigned int)a.n_slots] = slot;
      }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------
// kv_quant_pack, 4-bit: a kernel of its own (one thread block per item, placed by the
// hardware scheduler; the arithmetic needs more registers than the phases above).
// Item = (new 64-slot key group, four heads); 128 threads per head, thread =
// (8-channel word, four tokens 16 apart).
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

  // ---- values, parameters and origins of the survivors (first frame: nothing to move): the row is
  // fetched here and stored after the key loads below have been issued, so that the two round
  // trips overlap (thread = (head, token, half row): exactly one item per thread) ----
  uint4 v_row = make_uint4(0, 0, 0, 0);
  float2 v_par = make_float2(0.f, 0.f);
  int v_org = 0;
  size_t v_dst = 0;
  bool v_move = false, o_move = false;
  {
    const int half = tid & 1, tok = (tid >> 1) & 63, hh = blockIdx.y * kRgHeads + (tid >> 7);
    const int i = gamma * 64 + tok;
    if (kk > 0 && hh < H && i < kk) {
      const size_t s_slot = (size_t)hh * cap + base_slot + s_old[tok];
      v_dst = (size_t)hh * cap + base_slot + i;
      v_row = *reinterpret_cast<const uint4*>(src.v + s_slot * 32 + 16 * half);
      if (half == 0) v_par = src.vpar[s_slot];
      v_move = true;
    }
    if (kk > 0 && blockIdx.y == 0 && tid < 64 && gamma * 64 + tid < kk) {
      v_org = src.origin[base_slot + s_old[tid]];
      o_move = true;
    }
  }
  auto store_values = [&]() {
    if (v_move) {
      *reinterpret_cast<uint4*>(dst.v + v_dst * 32 + 16 * (tid & 1)) = v_row;
      if ((tid & 1) == 0) dst.vpar[v_dst] = v_par;
    }
    if (o_move) dst.origin[base_slot + gamma * 64 + tid] = v_org;
  };

  // ---- keys ----
  const int last = gamma * 64 + 63;
  const bool carried = (last < kk) && (s_old[63] == last);
  const size_t dgrp = ((size_t)h * (cap >> 6) + (base_slot >> 6) + gamma) * 64;
  if (carried) {
    store_values();
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
  store_values();
  int par_grp = -1;
  const float2* par_src = nullptr; // the group's (s, z) in global memory (the plain path reads them there)
  uint64_t s2[4], mz2[4];          // fast path: (s, s) and (magic + z, magic + z) of the channel pairs
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
          zmax = fmaxf(zmax, fmaxf(fabsf(q4.y), fabsf(q4.w)));
          s2[v] = pk2(q4.x, q4.z);
          mz2[v] = pk2(__fadd_rn(magic_val(2 * v), q4.y), __fadd_rn(magic_val(2 * v), q4.w));
        }
        par_plain = !(zmax < kZLimit) || force_plain;
        par_src = reinterpret_cast<const float2*>(pp);
        par_grp = g;
      }
      if (par_plain) dequant8_plain(word[u], par_src, x[u]);
      else dequant8_magic2(word[u], s2, mz2, x[u]);
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
  uint64_t inv2[4];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    iz[j] = s_iz[hl][8 * w + j];
    zadj[j] = slow ? 0 : (int)iz[j].y - (int)0x4B400000;
  }
#pragma unroll
  for (int p = 0; p < 4; ++p) inv2[p] = pk2(iz[2 * p].x, iz[2 * p + 1].x);
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
      for (int p = 0; p < 4; ++p) {
        // x * inv for two channels at once; the addition of 1.5 * 2^23 stays scalar: a packed
        // multiplication followed by a packed addition was observed to round once, like a fused
        // multiply-add, which breaks the ties of Eq. 7's rounding
        float te, to;
        unpk2(mul2(pk2(x[u][2 * p], x[u][2 * p + 1]), inv2[p]), te, to);
        te = __fadd_rn(te, kRoundMagic);
        to = __fadd_rn(to, kRoundMagic);
        int qe = (int)__float_as_uint(te) + zadj[2 * p], qo = (int)__float_as_uint(to) + zadj[2 * p + 1];
        asm("min.relu.s32 %0, %1, 15;" : "=r"(qe) : "r"(qe));
        asm("min.relu.s32 %0, %1, 15;" : "=r"(qo) : "r"(qo));
        // the nibbles do not overlap: multiply-add places them
        packed = (uint32_t)qe * (1u << nib_shift(2 * p)) + packed;
        packed = (uint32_t)qo * (1u << nib_shift(2 * p + 1)) + packed;
      }
    }
    const size_t dslot = (size_t)h * cap + base_slot + gamma * 64 + tq + 16 * u;
    *reinterpret_cast<uint32_t*>(dst.k + dslot * 32 + 4 * w) = packed;
    if (two) *reinterpret_cast<uint32_t*>(dst2.k + dslot * 32 + 4 * w) = packed;
  }
}

// ---------------------------------------------------------------------------
// PACK, 16-bit: rows of keys and values and the origins move from the current
// buffer set to the other, preserving order.  Thread-item = (head, survivor,
// 16-byte chunk).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void phase_gather16(const MaintArgs& a) {
  const BufSet& src = a.cur;
  const BufSet& dst = a.oth;
  const int32_t* kept = a.identity ? nullptr : a.kept;
  const long long items = (long long)a.H * a.kk * 8;
  for (long long g = (long long)blockIdx.x * kMT + threadIdx.x; g < items; g += (long long)gridDim.x * kMT) {
    const int ch = (int)(g & 7);
    const long long r = g >> 3;
    const int i = (int)(r % a.kk);
    const int h = (int)(r / a.kk);
    const int old = kept ? __ldcg(&kept[i]) : i;
    const size_t s = (size_t)h * a.cap + a.rest_base + old;
    const size_t d = (size_t)h * a.cap + a.rest_base + i;
    *reinterpret_cast<uint4*>(dst.v + d * 128 + 16 * ch) = *reinterpret_cast<const uint4*>(src.v + s * 128 + 16 * ch);
    *reinterpret_cast<uint4*>(dst.k + d * 128 + 16 * ch) = *reinterpret_cast<const uint4*>(src.k + s * 128 + 16 * ch);
    if (h == 0 && ch == 0) dst.origin[a.rest_base + i] = src.origin[a.rest_base + old];
  }
}

}  // namespace

// ---------------------------------------------------------------------------
// The kernel.
// ---------------------------------------------------------------------------
template <int BITS, bool ONCE>
__global__ void __launch_bounds__(kMT, kBlocksPerSM) maint_kernel(const __grid_constant__ MaintArgs a) {
  __shared__ Shared sh;
  if (threadIdx.x == 0) { sh.abort_flag = 0; sh.acc = 0u; sh.bin = 0u; sh.need = 0u; sh.fsum[0] = sh.fsum[1] = 0.f; }
  __syncthreads();
  uint32_t epoch = 0;
  const uint32_t ph = a.phases;
  bool ran = false;                 // something has run since the last barrier

  if (ph & kPhAppend) {
    phase_append<BITS, ONCE>(a);
    if (ONCE) phase_quant_keys_once<BITS>(a, sh);
    ran = true;
  }
  if (ph & kPhPool) { phase_pool(a, sh); ran = true; }
  if (ph & kPhKbar) { phase_kbar<BITS>(a, sh, a.kbar_on_other ? a.oth : a.cur, a.kbar_lo, a.kbar_hi); ran = true; }

  if (ph & (kPhScore | kPhKbarNew)) {
    if (ran && !grid_barrier(a, epoch, sh)) return;
    if (ONCE && (ph & kPhKbarNew)) phase_kbar_new_once<BITS>(a, sh);
    if (ph & kPhScore) phase_score(a, sh);
    ran = true;
  }
  if (ph & kPhSel) {
    if (ran && !grid_barrier(a, epoch, sh)) return;
    phase_sel1(a, sh);
    if (!grid_barrier(a, epoch, sh)) return;
    phase_sel2<ONCE>(a, sh);
    ran = true;
  }
  if (ph & kPhPack) {
    if (ran && !grid_barrier(a, epoch, sh)) return;
    if (ONCE) phase_gather_once<BITS>(a);
    else if (BITS == 16 && a.kk > 0) phase_gather16(a);
  }
}

// Quantise-once mode: the ring of free table slots starts full.
__global__ void once_init_kernel(int32_t* ring, unsigned int* push_pos, int n_slots) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_slots) ring[i] = i;
  if (i == 0) *push_pos = (unsigned int)n_slots;
}

cudaError_t launch_once_init(xkv_cache* c, cudaStream_t st) {
  once_init_kernel<<<(c->n_slots + 255) / 256, 256, 0, st>>>(c->ring, c->counters + 8, c->n_slots);
  return cudaGetLastError();
}

// Grid barriers that a launch with these phases goes through (the same decisions as in the kernel).
static int maint_barriers(uint32_t ph) {
  int nb = 0;
  bool ran = (ph & (kPhAppend | kPhPool | kPhKbar)) != 0;
  if (ph & (kPhScore | kPhKbarNew)) { nb += ran ? 1 : 0; ran = true; }
  if (ph & kPhSel) { nb += (ran ? 1 : 0) + 1; ran = true; }
  if (ph & kPhPack) nb += ran ? 1 : 0;
  return nb;
}

// Per device, on first use with that device current: how many blocks of the kernel can be
// resident at once (a cooperative launch needs the whole grid resident).
static std::mutex g_maint_mutex;
static int g_maint_grid[64] = {0};

static cudaError_t maint_grid(int* grid) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_maint_mutex);
  if (g_maint_grid[dev] == 0) {
    int sms = 0, per_sm = kBlocksPerSM;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const void* fns[4] = {(const void*)maint_kernel<4, false>, (const void*)maint_kernel<16, false>,
                          (const void*)maint_kernel<4, true>, (const void*)maint_kernel<8, true>};
    for (const void* fn : fns) {
      int nb = 0;
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, kMT, 0);
      if (e != cudaSuccess) return e;
      if (nb < per_sm) per_sm = nb;
    }
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    g_maint_grid[dev] = sms * per_sm;
  }
  *grid = g_maint_grid[dev];
  return cudaSuccess;
}

cudaError_t launch_regroup(xkv_cache* c, const MaintArgs& a, cudaStream_t st) {
  const dim3 grid((a.r_new + 63) / 64, (a.H + kRgHeads - 1) / kRgHeads);
  LaunchScope ls(c, XKV_PROF_PACK, st);
  regroup_k_kernel<<<grid, 128 * kRgHeads, 0, st>>>(a.cur, a.oth, a.cur, a.first != 0, a.H, a.cap, a.max_n,
                                                   a.first ? 0 : a.rest_base, a.kk, a.r_new,
                                                   a.identity ? nullptr : a.kept, a.kstage, a.force_plain);
  return cudaGetLastError();
}

cudaError_t launch_maint(xkv_cache* c, MaintArgs& a, int prof_cat, cudaStream_t st) {
  int grid = 0;
  cudaError_t e = maint_grid(&grid);
  if (e != cudaSuccess) return e;
  const int nb = maint_barriers(a.phases);
  a.bar = c->counters;
  a.bar_base = c->bar_base;
  a.status = c->status;
  a.cand_count = c->counters + 2 + c->sel_parity;
  a.cand_count_next = c->counters + 2 + (c->sel_parity ^ 1);
  a.hist2 = c->counters + 64 + 256 * c->sel_parity;
  a.hist2_next = c->counters + 64 + 256 * (c->sel_parity ^ 1);
  a.stats = reinterpret_cast<float*>(c->counters + 16 + 4 * c->sel_parity);
  a.stats_next = reinterpret_cast<float*>(c->counters + 16 + 4 * (c->sel_parity ^ 1));
  if (a.phases & kPhSel) c->stats_parity = c->sel_parity;
  if (a.phases & kPhSel) c->sel_parity ^= 1;
  LaunchScope ls(c, prof_cat, st);
  void* params[1] = {(void*)&a};
  a.push_pos = c->counters + 8;
  const void* fn = (c->p.kv_bits == 16) ? (const void*)maint_kernel<16, false>
                   : (c->p.kv_bits == 8) ? (const void*)maint_kernel<8, true>
                   : c->p.key_mode == XKV_KEYS_ONCE ? (const void*)maint_kernel<4, true>
                                                    : (const void*)maint_kernel<4, false>;
  if (nb > 0) {
    e = cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kMT), params, 0, st);
    c->bar_base += (uint32_t)nb * (uint32_t)grid;
  } else {
    e = cudaLaunchKernel(fn, dim3(grid), dim3(kMT), params, 0, st);
  }
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

}  // namespace xkv
