// Tensor-core attention over the packed cache (Eq. 1 with the dequantisation of
// Eq. 10) for sm_100a: tcgen05.mma with accumulators in tensor memory.
//
// One CTA = one tile of 128 queries of one head over a contiguous range of
// 128-slot key tiles (split-KV).  Warp roles:
//   warps 0-3  softmax: thread r owns query row r = TMEM lane r.  Reads S from
//              TMEM, online max/sum, writes P (16-bit) back to TMEM, rescales O
//              when the running maximum moved by more than 2^8, epilogue.
//   warps 4-7  operand producers: 4-bit codes -> fp16 (K~ per channel/group, V~
//              per token) written into shared memory in the 128-byte-swizzled
//              layouts the MMA descriptors expect.
//   warp  8    allocates tensor memory; one elected thread issues the MMAs:
//              S = Q K~^T (M128 N128 K64, both operands K-major in smem) and
//              O += P V~ (M128 N64 K128, A = P from TMEM, B = V~ MN-major).
// 4-bit caches multiply in fp16 (the dequantised keys are not bf16-representable:
// rounding them to bf16 alone costs ~1e-2 relative L2 with outlier channels);
// 16-bit caches hold bf16 and multiply in bf16.  Accumulation is fp32.
//
// Every mbarrier wait is bounded: when the bound is hit the thread records
// XKV_E_TIMEOUT in the cache's status word and carries on, so the kernel always
// terminates and frees its tensor memory.
#include <mutex>

#include "xkv_internal.cuh"

namespace xkv {

namespace {

constexpr int kMaxDevices = 64;
constexpr int kThreads = 288;
constexpr int kQRows = 128;
constexpr int kMaxSplits = 6;
constexpr uint32_t kSpinLimit = 1u << 22;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;                 // 16 KB  Q tile, K-major, SW128
constexpr int kOffK = 16384;             // 2 x 16 KB  K~ tiles
constexpr int kOffV = 16384 * 3;         // 2 x 16 KB  V~ tiles
constexpr int kOffBar = 16384 * 5;       // barriers + tmem base
constexpr int kSmemBytes = kOffBar + 256 + 1024;   // + alignment slack

// tensor memory columns
constexpr int kColS = 0;      // 128 fp32 columns
constexpr int kColP = 128;    // 64 columns of packed 16-bit pairs
constexpr int kColO = 192;    // 64 fp32 columns
constexpr int kTmemCols = 256;

struct Args {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  int n;
  int64_t ts, hs;
  const uint8_t* k;
  const float2* kpar;
  const uint8_t* v;
  const float2* vpar;
  int cap, t_first, rest_base, t_phys;
  float scale_log2;
  int n_tiles, tiles_per_split, n_splits;
  float* part_o;     // [split][H][n][64]
  float2* part_ml;   // [split][H][n]
  int* status;
};

// ---- PTX wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  On exhaustion the failure is recorded (device status word and a
// per-CTA flag); once the flag is up every later wait of the CTA gives up at once.
struct WaitCtx { int* status; volatile int* abort_flag; };
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& wc) {
  if (*wc.abort_flag) return;
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try(bar, parity)) return;
  *wc.abort_flag = 1;
  atomicExch(wc.status, (int)XKV_E_TIMEOUT);
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// packed fp32 pairs (two floats in one 64-bit register)
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float f2_lo(uint64_t v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float f2_hi(uint64_t v) { return __uint_as_float((uint32_t)(v >> 32)); }
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add_f2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul_f2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

#define XKV_TMEM_LD32(taddr, r)                                                                      \
  asm volatile(                                                                                      \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                      \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                      \
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                     \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), \
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),     \
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),   \
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),   \
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])                                                        \
      : "r"(taddr) : "memory")

#define XKV_TMEM_ST32(taddr, r)                                                                      \
  asm volatile(                                                                                      \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                                \
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"                                     \
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"                            \
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),     \
        "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), \
        "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]),          \
        "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]),          \
        "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory")

#define XKV_TMEM_ST16(taddr, r)                                                                      \
  asm volatile(                                                                                      \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "                                                \
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"                                    \
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),     \
        "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), \
        "r"(r[15]) : "memory")

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);        // start address
  d |= (uint64_t)1 << 16;                        // leading byte offset (unused with one swizzle span)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // SWIZZLE_128B
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulate, M = 128.
__device__ __forceinline__ uint32_t make_idesc(int n_dim, bool bf16, bool b_mn_major) {
  uint32_t d = 0;
  d |= 1u << 4;                                  // D format fp32
  d |= (bf16 ? 1u : 0u) << 7;                    // A format
  d |= (bf16 ? 1u : 0u) << 10;                   // B format
  d |= (b_mn_major ? 1u : 0u) << 16;             // B major
  d |= (uint32_t)(n_dim >> 3) << 17;
  d |= (uint32_t)(128 >> 4) << 24;
  return d;
}

__device__ __forceinline__ uint32_t swz_off(int row, int chunk) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk ^ (row & 7)) << 4));
}

__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf2(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t h2_sub(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

__device__ __forceinline__ uint32_t h2_mul(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// Eight 4-bit codes of one packed word -> four fp16 pairs s * (q - z)  (Eq. 10).
// (w & 0x000F000F) | 0x6400 is the fp16 number 1024 + q and (w & 0x00F000F0) | 0x5400 is 64 + q,
// so one subtraction of (1024 + z) resp. (64 + z) gives q - z exactly (z is an integer), and one
// multiplication by the fp16 scale follows.  zlo/zhi hold those two constants per channel pair:
// pairs 0 and 2 of a word use the 1024 offset, pairs 1 and 3 the 64 offset.
__device__ __forceinline__ uint4 dequant_word_h(uint32_t w, const uint32_t (&s2)[4], const uint32_t (&zo)[4]) {
  const uint32_t t = w >> 8;
  const uint32_t a0 = (w & 0x000F000Fu) | 0x64006400u;
  const uint32_t a1 = (w & 0x00F000F0u) | 0x54005400u;
  const uint32_t a2 = (t & 0x000F000Fu) | 0x64006400u;
  const uint32_t a3 = (t & 0x00F000F0u) | 0x54005400u;
  uint4 r;
  r.x = h2_mul(h2_sub(a0, zo[0]), s2[0]);
  r.y = h2_mul(h2_sub(a1, zo[1]), s2[1]);
  r.z = h2_mul(h2_sub(a2, zo[2]), s2[2]);
  r.w = h2_mul(h2_sub(a3, zo[3]), s2[3]);
  return r;
}

}  // namespace

template <int BITS>
__global__ void __launch_bounds__(kThreads, 2) attn_tc_kernel(const Args a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const uint32_t sQ = sbase + kOffQ, sK = sbase + kOffK, sV = sbase + kOffV;
  const uint32_t bar0 = sbase + kOffBar;
  // barrier slots (8 bytes each)
  const uint32_t b_kfull = bar0, b_kfree = bar0 + 16, b_vfull = bar0 + 32, b_vfree = bar0 + 48;
  const uint32_t b_sfull = bar0 + 64, b_sfree = bar0 + 72, b_pfull = bar0 + 80, b_pvdone = bar0 + 88;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sgen + kOffBar + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + kOffBar + 132);
  const WaitCtx wc{a.status, abort_flag};

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int h = blockIdx.y;
  const int q0 = blockIdx.x * kQRows;
  const int split = blockIdx.z;
  const int tile_lo = split * a.tiles_per_split;
  const int tile_hi = min(tile_lo + a.tiles_per_split, a.n_tiles);
  const int nt = tile_hi - tile_lo;
  constexpr bool kBf16 = (BITS == 16);

  if (tid == 0) {
    *abort_flag = (*reinterpret_cast<volatile int*>(a.status) != 0) ? 1 : 0;   // an earlier CTA already gave up
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_kfull + 8 * i, 128); mbar_init(b_kfree + 8 * i, 1);
      mbar_init(b_vfull + 8 * i, 128); mbar_init(b_vfree + 8 * i, 1);
    }
    mbar_init(b_sfull, 1); mbar_init(b_sfree, 128); mbar_init(b_pfull, 128); mbar_init(b_pvdone, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp < 4) {
    // Q tile: row r of this thread, bf16 -> operand type, into the swizzled K-major layout
    const int row = q0 + tid;
    uint4 u[8];
    if (row < a.n) {
      const __nv_bfloat16* qp = a.q + (int64_t)h * a.hs + (int64_t)row * a.ts;
#pragma unroll
      for (int c = 0; c < 8; ++c) u[c] = *reinterpret_cast<const uint4*>(qp + 8 * c);
    } else {
#pragma unroll
      for (int c = 0; c < 8; ++c) u[c] = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      uint4 o = u[c];
      if (!kBf16) {
        const uint32_t r[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
        uint32_t hh[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          hh[i] = pack_h2(__uint_as_float(r[i] << 16), __uint_as_float(r[i] & 0xFFFF0000u));
        o = make_uint4(hh[0], hh[1], hh[2], hh[3]);
      }
      *reinterpret_cast<uint4*>(sgen + kOffQ + swz_off(tid, c)) = o;
    }
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp < 4) {
    // =========================== softmax warps ===============================
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    float m_ref = -INFINITY;   // reference maximum (scaled, log2 units) used for the exponentials
    uint64_t l2 = 0ull;        // two partial row sums (packed fp32 pair)
    const int pad_tile = (a.t_first & 127) ? (a.t_first >> 7) : -1;
    for (int jj = 0; jj < nt; ++jj) {
      const int tile = tile_lo + jj;
      int lim_lo = 128, lim_hi = 128;   // columns [lim_lo, 128) of a first-segment pad tile, [lim_hi,128) of the tail are masked
      if (tile == pad_tile) lim_lo = a.t_first & 127;
      if (tile == a.n_tiles - 1) lim_hi = a.t_phys - tile * 128;
      const int lim = min(lim_lo, lim_hi);
      mbar_wait(b_sfull, jj & 1, wc);
      __syncwarp();
      tc_fence_after();
      // pass 1: row maximum
      float mx = -INFINITY;
      if (lim >= 128) {
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          XKV_TMEM_LD32(lane_addr + kColS + c0, r);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; i += 2) mx = max3(mx, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
        }
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          XKV_TMEM_LD32(lane_addr + kColS + c0, r);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float x = (c0 + i < lim) ? __uint_as_float(r[i]) : -INFINITY;
            mx = fmaxf(mx, x);
          }
        }
      }
      mx *= a.scale_log2;
      // decide whether the reference maximum moves (only when it grew by more than 2^8)
      float alpha = 1.f;
      const bool grow = mx > m_ref + 8.f;
      if (grow) {
        alpha = exp2f(m_ref - mx);      // 0 on the first tile (m_ref = -inf)
        m_ref = mx;
        l2 = mul_f2(l2, pack_f2(alpha, alpha));
      }
      if (jj > 0) {
        // P(jj-1) has been consumed and O is quiescent once PV(jj-1) completed
        mbar_wait(b_pvdone, (jj - 1) & 1, wc);
        __syncwarp();
        tc_fence_after();
        if (__any_sync(0xffffffffu, grow)) {
#pragma unroll 1
          for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t r[32];
            XKV_TMEM_LD32(lane_addr + kColO + c0, r);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            XKV_TMEM_ST32(lane_addr + kColO + c0, r);
          }
          tc_wait_st();
        }
      }
      // pass 2: exponentials, row sum, P -> TMEM (16-bit pairs)
      const uint64_t sc2 = pack_f2(a.scale_log2, a.scale_log2);
      const uint64_t nm2 = pack_f2(-m_ref, -m_ref);
      if (lim >= 128) {
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          XKV_TMEM_LD32(lane_addr + kColS + c0, r);
          tc_wait_ld();
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint64_t x2 = fma_f2(pack_f2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), sc2, nm2);
            const float p0 = fast_exp2(f2_lo(x2)), p1 = fast_exp2(f2_hi(x2));
            l2 = add_f2(l2, pack_f2(p0, p1));
            pk[i] = kBf16 ? pack_bf2(p0, p1) : pack_h2(p0, p1);
          }
          XKV_TMEM_ST16(lane_addr + kColP + (c0 >> 1), pk);
        }
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          XKV_TMEM_LD32(lane_addr + kColS + c0, r);
          tc_wait_ld();
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float p0 = fast_exp2(fmaf(__uint_as_float(r[2 * i]), a.scale_log2, -m_ref));
            float p1 = fast_exp2(fmaf(__uint_as_float(r[2 * i + 1]), a.scale_log2, -m_ref));
            if (c0 + 2 * i >= lim) p0 = 0.f;
            if (c0 + 2 * i + 1 >= lim) p1 = 0.f;
            l2 = add_f2(l2, pack_f2(p0, p1));
            pk[i] = kBf16 ? pack_bf2(p0, p1) : pack_h2(p0, p1);
          }
          XKV_TMEM_ST16(lane_addr + kColP + (c0 >> 1), pk);
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(b_sfree);
      mbar_arrive(b_pfull);
    }
    // epilogue
    mbar_wait(b_pvdone, (nt - 1) & 1, wc);
    __syncwarp();
    tc_fence_after();
    const int row = q0 + tid;
    const float l = f2_lo(l2) + f2_hi(l2);
    if (a.n_splits == 1) {
      const float inv_l = 1.f / l;
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t r[32];
        XKV_TMEM_LD32(lane_addr + kColO + c0, r);
        tc_wait_ld();
        if (row < a.n) {
          __nv_bfloat16* op = a.out + (int64_t)h * a.hs + (int64_t)row * a.ts + c0;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              o[i] = pack_bf2(__uint_as_float(r[8 * c + 2 * i]) * inv_l, __uint_as_float(r[8 * c + 2 * i + 1]) * inv_l);
            *reinterpret_cast<uint4*>(op + 8 * c) = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
      }
    } else {
      const size_t prow = ((size_t)split * gridDim.y + h) * a.n + row;
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t r[32];
        XKV_TMEM_LD32(lane_addr + kColO + c0, r);
        tc_wait_ld();
        if (row < a.n) {
          float4* dst = reinterpret_cast<float4*>(a.part_o + prow * 64 + c0);
#pragma unroll
          for (int c = 0; c < 8; ++c)
            dst[c] = make_float4(__uint_as_float(r[4 * c]), __uint_as_float(r[4 * c + 1]),
                                 __uint_as_float(r[4 * c + 2]), __uint_as_float(r[4 * c + 3]));
        }
      }
      if (row < a.n) a.part_ml[prow] = make_float2(m_ref, l);
    }
    tc_fence_before();
  } else if (warp < 8) {
    // =========================== operand producers ===========================
    const int t = tid - 128;
    const int w = t & 7;          // 16-byte chunk = 8 channels
    const int kb = t >> 3;        // keys kb + 16 i
    const uint32_t row_off = (uint32_t)((kb >> 3) * 1024 + (kb & 7) * 128 + ((w ^ (kb & 7)) << 4));
    const size_t head_slot = (size_t)h * a.cap;
    for (int jj = 0; jj < nt; ++jj) {
      const int tile = tile_lo + jj;
      const int b = jj & 1, u = jj >> 1;
      const int p0 = tile * 128 + kb;
      // ---- keys ----
      mbar_wait(b_kfree + 8 * b, (u & 1) ^ 1, wc);
      if (BITS == 4) {
        uint32_t wd[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          wd[i] = __ldg(reinterpret_cast<const uint32_t*>(a.k + (head_slot + p0 + 16 * i) * 32 + 4 * w));
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          const float2* par = a.kpar + ((size_t)h * (a.cap >> 6) + (tile * 2 + g)) * 64 + 8 * w;
          uint32_t s2[4], zo[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 p_a = __ldg(par + 2 * i), p_b = __ldg(par + 2 * i + 1);
            const float off = (i & 1) ? 64.f : 1024.f;
            s2[i] = pack_h2(p_a.x, p_b.x);
            zo[i] = pack_h2(off + p_a.y, off + p_b.y);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 o = dequant_word_h(wd[4 * g + i], s2, zo);
            *reinterpret_cast<uint4*>(sgen + kOffK + b * 16384 + row_off + (4 * g + i) * 2048) = o;
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 o = __ldg(reinterpret_cast<const uint4*>(a.k + (head_slot + p0 + 16 * i) * 128 + 16 * w));
          *reinterpret_cast<uint4*>(sgen + kOffK + b * 16384 + row_off + i * 2048) = o;
        }
      }
      fence_proxy_async();
      mbar_arrive(b_kfull + 8 * b);
      // ---- values ----
      mbar_wait(b_vfree + 8 * b, (u & 1) ^ 1, wc);
      if (BITS == 4) {
        uint32_t wd[8];
        float2 vp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          wd[i] = __ldg(reinterpret_cast<const uint32_t*>(a.v + (head_slot + p0 + 16 * i) * 32 + 4 * w));
          vp[i] = __ldg(a.vpar + head_slot + p0 + 16 * i);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint32_t s1 = pack_h2(vp[i].x, vp[i].x);
          const uint32_t z_lo = pack_h2(1024.f + vp[i].y, 1024.f + vp[i].y);
          const uint32_t z_hi = pack_h2(64.f + vp[i].y, 64.f + vp[i].y);
          const uint32_t s2[4] = {s1, s1, s1, s1}, zo[4] = {z_lo, z_hi, z_lo, z_hi};
          const uint4 o = dequant_word_h(wd[i], s2, zo);
          *reinterpret_cast<uint4*>(sgen + kOffV + b * 16384 + row_off + i * 2048) = o;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 o = __ldg(reinterpret_cast<const uint4*>(a.v + (head_slot + p0 + 16 * i) * 128 + 16 * w));
          *reinterpret_cast<uint4*>(sgen + kOffV + b * 16384 + row_off + i * 2048) = o;
        }
      }
      fence_proxy_async();
      mbar_arrive(b_vfull + 8 * b);
    }
  } else if (tid == 256) {
    // =========================== MMA issuer ===================================
    const uint32_t idesc_qk = make_idesc(128, kBf16, false);
    const uint32_t idesc_pv = make_idesc(64, kBf16, true);
    const uint64_t dq = make_desc(sQ);
    auto issue_pv = [&](int t) {
      const int b = t & 1, u = t >> 1;
      mbar_wait(b_vfull + 8 * b, u & 1, wc);
      mbar_wait(b_pfull, t & 1, wc);
      tc_fence_after();
      const uint64_t dv = make_desc(sV + b * 16384);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)   // 16 keys per step: 2 swizzle atoms = 2048 B of V~, 8 columns of P
        mma_ts(tmem + kColO, tmem + kColP + 8 * ks, dv + (uint64_t)((ks * 2048) >> 4), idesc_pv,
               (t > 0 || ks > 0) ? 1u : 0u);
      tc_commit(b_vfree + 8 * b);
      tc_commit(b_pvdone);
    };
    for (int jj = 0; jj < nt; ++jj) {
      const int b = jj & 1, u = jj >> 1;
      mbar_wait(b_kfull + 8 * b, u & 1, wc);
      mbar_wait(b_sfree, (jj & 1) ^ 1, wc);
      tc_fence_after();
      const uint64_t dk = make_desc(sK + b * 16384);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)   // 16 channels per step: 32 B inside the swizzle span
        mma_ss(tmem + kColS, dq + (uint64_t)(ks * 2), dk + (uint64_t)(ks * 2), idesc_qk, ks > 0 ? 1u : 0u);
      tc_commit(b_kfree + 8 * b);
      tc_commit(b_sfull);
      if (jj > 0) issue_pv(jj - 1);
    }
    issue_pv(nt - 1);
    // wait until the last MMAs are done before the CTA may free tensor memory
    mbar_wait(b_pvdone, (nt - 1) & 1, wc);
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 8) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------
// Split-KV combine: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.
// Thread = (head, row, 8-channel chunk).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
attn_combine_kernel(const float* __restrict__ part_o, const float2* __restrict__ part_ml, int n_splits, int H,
                    int n, __nv_bfloat16* __restrict__ out, int64_t ts, int64_t hs) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int ch = (int)(g & 7);
  const long long hr = g >> 3;
  if (hr >= (long long)H * n) return;
  float m = -INFINITY;
  for (int s = 0; s < n_splits; ++s) m = fmaxf(m, part_ml[(size_t)s * H * n + hr].x);
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  float l = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float2 ml = part_ml[(size_t)s * H * n + hr];
    const float wgt = exp2f(ml.x - m);
    l += wgt * ml.y;
    const float4* po = reinterpret_cast<const float4*>(part_o + ((size_t)s * H * n + hr) * 64 + 8 * ch);
    const float4 x = po[0], y = po[1];
    acc[0] += wgt * x.x; acc[1] += wgt * x.y; acc[2] += wgt * x.z; acc[3] += wgt * x.w;
    acc[4] += wgt * y.x; acc[5] += wgt * y.y; acc[6] += wgt * y.z; acc[7] += wgt * y.w;
  }
  const float inv = 1.f / l;
  const int h = (int)(hr / n), row = (int)(hr % n);
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = pack_bf2(acc[2 * i] * inv, acc[2 * i + 1] * inv);
  *reinterpret_cast<uint4*>(out + (int64_t)h * hs + (int64_t)row * ts + 8 * ch) = make_uint4(o[0], o[1], o[2], o[3]);
}

size_t attn_tc_scratch_bytes(const xkv_params* p) {
  const size_t rows = (size_t)kMaxSplits * p->n_heads * p->max_frame_tokens;
  return rows * 64 * sizeof(float) + rows * sizeof(float2) + 512;
}

// Splits are chosen so that the grid fills whole waves of (SMs x 2 resident CTAs).
static int choose_splits(int items, int n_tiles, int slots) {
  int best = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= kMaxSplits; ++s) {
    const int tps = (n_tiles + s - 1) / s;
    if (tps < 2 && s > 1) break;
    if ((s - 1) * tps >= n_tiles) continue;      // an empty split
    const long long ctas = (long long)items * s;
    const long long waves = (ctas + slots - 1) / slots;
    const double eff = (double)ctas / (double)(waves * slots) * ((double)n_tiles / (double)(tps * s));
    if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
  }
  return best;
}

// `part` holds the split-KV partials: accumulators float [rows_cap][64], then (max, sum) float2
// [rows_cap].  rows_cap = 0 means "as many rows as this launch needs" and `part_bytes` is then the
// room available: when it does not suffice nothing is launched and cudaErrorMemoryAllocation returns.
static cudaError_t launch_attn_tc_on(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                                     float scale, float* part, size_t rows_cap, size_t part_bytes,
                                     cudaStream_t st) {
  static int sm_count = 0;
  static bool attr_set = false;
  if (!attr_set) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  Args a;
  a.q = reinterpret_cast<const __nv_bfloat16*>(q);
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.n = n; a.ts = ts; a.hs = hs;
  const BufSet& b = c->buf[c->cur];
  a.k = b.k; a.kpar = b.kpar; a.v = b.v; a.vpar = b.vpar;
  a.cap = c->cap; a.t_first = c->T_first; a.rest_base = c->rest_base;
  a.t_phys = c->rest_base + (c->T - c->T_first);
  if (c->T == c->T_first) a.t_phys = c->T_first;          // only the first frame: no pad tile beyond it
  a.scale_log2 = scale * 1.4426950408889634f;
  a.n_tiles = (a.t_phys + 127) / 128;
  const int q_tiles = (n + kQRows - 1) / kQRows;
  const int H = c->p.n_heads;
  a.n_splits = choose_splits(q_tiles * H, a.n_tiles, sm_count * 2);
  a.tiles_per_split = (a.n_tiles + a.n_splits - 1) / a.n_splits;
  size_t rows = rows_cap;
  if (rows == 0) {
    rows = (size_t)a.n_splits * H * n;
    if (a.n_splits > 1 && rows * (64 * sizeof(float) + sizeof(float2)) > part_bytes) return cudaErrorMemoryAllocation;
  }
  a.part_o = part;
  a.part_ml = reinterpret_cast<float2*>(part + rows * 64);
  a.status = c->status;
  const dim3 grid(q_tiles, H, a.n_splits);
  {
    LaunchScope ls(c, XKV_PROF_ATTN, st);
    if (c->p.kv_bits == 16) attn_tc_kernel<16><<<grid, kThreads, kSmemBytes, st>>>(a);
    else attn_tc_kernel<4><<<grid, kThreads, kSmemBytes, st>>>(a);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (a.n_splits > 1) {
    LaunchScope ls(c, XKV_PROF_COMBINE, st);
    const long long threads = (long long)H * n * 8;
    attn_combine_kernel<<<(int)((threads + 255) / 256), 256, 0, st>>>(a.part_o, a.part_ml, a.n_splits, H, n, a.out, ts, hs);
  }
  return cudaGetLastError();
}

cudaError_t launch_attn_tc(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs, float scale,
                           cudaStream_t st) {
  return launch_attn_tc_on(c, q, out, n, ts, hs, scale, c->attn_part,
                           (size_t)kMaxSplits * c->p.n_heads * c->p.max_frame_tokens, c->attn_part_bytes, st);
}

// ---------------------------------------------------------------------------
// attn_packed_causal_static: the same attention with its split-KV partials in a
// fixed array that is part of the loaded library image instead of the caller's
// workspace.  See xkv.h for who needs this and for the rules of use.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_partials[XKV_STATIC_SCRATCH_BYTES];

// In host code `g_static_partials` only names the symbol; the device address has to be asked
// for, once per device, while that device is current.
static std::mutex g_static_mutex;
static void* g_static_addr[kMaxDevices] = {nullptr};

cudaError_t launch_attn_tc_static(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                                  float scale, cudaStream_t st) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  void* addr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_static_partials);
      if (e != cudaSuccess) return e;
      g_static_addr[dev] = p;
    }
    addr = g_static_addr[dev];
  }
  return launch_attn_tc_on(c, q, out, n, ts, hs, scale, reinterpret_cast<float*>(addr), 0,
                           (size_t)XKV_STATIC_SCRATCH_BYTES, st);
}

}  // namespace xkv
