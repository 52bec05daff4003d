// Tensor-core attention over the packed cache (Eq. 1 with the dequantisation of
// Eq. 10) for sm_100a: tcgen05.mma with accumulators in tensor memory, operands
// staged by bulk asynchronous copies (TMA) and dequantised in shared memory.
//
// Work.  An item is (head, pair of 128-query tiles); it meets every 128-slot key
// tile of the cache.  Items x key tiles are laid out on one line of steps, and the
// line is cut into equal pieces, one per CTA (one CTA per SM).  A piece that does
// not cover an item completely leaves partial results (accumulator, running max
// and sum) in a scratch slot; a second kernel merges them.
//
// One CTA.  The roles are the same in both forms of the kernel; the softmax comes in two:
//   softmax, 8 warps (SPLIT = false, 15 warps in all): warps 0-3 query tile 0, warps 4-7 query
//               tile 1; thread r owns query row r = TMEM lane r.  Reads S from tensor memory
//               chunk by chunk, online max/sum in one pass, writes P (16-bit) back to tensor
//               memory, rescales O only when the running maximum grew by more than 2^14.
//               Tensor memory: S 2 x 128 columns, P 2 x 64, O 2 x 64.
//   softmax, 16 warps (SPLIT = true, 24 warps in all): warps w and w + 8 share the rows of a
//               lane quarter, each takes 64 of the 128 key columns; a thread loads its half row
//               of scores into registers at once and releases the score columns, the maximum
//               is taken from the registers.  Registers move to these warps with setmaxnreg.
//               Tensor memory: ONE score buffer of 128 columns that the two tiles use in turn,
//               P 2 x 2 x 64 (two buffers per tile), O 2 x 64.
//   4 warps     operand producers: packed codes (raw, as copied by TMA) -> fp16 K~ (per channel
//               and key group) and V~ (per token) in the 128-byte-swizzled layouts the MMA
//               descriptors expect.  One dequantised tile serves both query tiles.
//   2 threads   (in warps of their own) issue the MMAs of query tile 0 resp. 1:
//               S_t = Q_t K~^T (M128 N128 K64) and O_t += P_t V~ (M128 N64 K128,
//               A = P from tensor memory).  A thread gets one tcgen05.mma through about every
//               125 cycles whatever its shape; a single issuing thread for both tiles was the
//               bottleneck of the CTA.
//   1 thread    issues the bulk copies of the raw tiles, several steps ahead; its warp owns the
//               tensor-memory allocation (all 512 columns).
// 4-bit caches multiply in fp16 (the dequantised keys are not bf16-representable:
// rounding them to bf16 alone costs ~1e-2 relative L2 with outlier channels);
// 16-bit caches hold bf16 and multiply in bf16.  Accumulation is fp32.
//
// Every mbarrier wait is bounded (one second of running time): when the bound is hit the thread records
// XKV_E_TIMEOUT in the cache's status word and carries on without waiting, so the
// kernel always terminates, drains its copies and frees its tensor memory.
#include <mutex>
#include <stdlib.h>

#include "xkv_internal.cuh"

namespace xkv {

namespace {

constexpr int kMaxDevices = 64;
constexpr int kThreads = 480;
// 16-warp form: registers per thread after the reallocation (softmax warps kSplitRegsSoftmax)
constexpr int kSplitRegsSoftmax = 96;
__host__ __device__ constexpr int split_regs_producers(bool once, bool tail) { return (once || tail) ? 56 : 40; }
__host__ __device__ constexpr int split_regs_misc(bool once, bool tail) { return (once || tail) ? 40 : 48; }   // MMA issuers, copy thread
constexpr int kThreadsSplit = 768;      // 16 softmax warps, 4 producers, 4 for the MMA issuers and the copies
constexpr int kQRows = 128;
constexpr int kMaxGrid = 160;                 // CTAs the scratch is sized for (>= SM count of the part)
constexpr uint32_t kSpinLimit = 1u << 22;
// The reference maximum of a row moves only when the row maximum exceeds it by more than 2^kGrow
// (log2 units).  Until then exponentials reach at most 2^14 = 16384, inside the fp16 range; the
// decision is taken per warp, so a low threshold would make some row of the 32 trip it at every
// few tiles.
constexpr float kGrow = 14.f;

// ring depths
constexpr int kNK = 3;                        // dequantised K~ tiles
constexpr int kNV = 3;                        // dequantised V~ tiles

template <int BITS> struct Cfg;
template <> struct Cfg<4> {
  static constexpr int kNR = 4;               // raw stages
  static constexpr int kRawK = 4096, kRawV = 4096, kRawKP = 1024, kRawVP = 1024;
  static constexpr int kRawStage = kRawK + kRawV + kRawKP + kRawVP;
};
template <> struct Cfg<8> {                    // 8-bit codes, keys quantised once: K, V rows of 64 bytes,
  static constexpr int kNR = 4;               // 128 group references (in the K-parameter region), V parameters
  static constexpr int kRawK = 8192, kRawV = 8192, kRawKP = 1024, kRawVP = 1024;
  static constexpr int kRawStage = kRawK + kRawV + kRawKP + kRawVP;
};
template <> struct Cfg<16> {
  static constexpr int kNR = 2;
  static constexpr int kRawK = 16384, kRawV = 16384, kRawKP = 0, kRawVP = 0;
  static constexpr int kRawStage = kRawK + kRawV;
};

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;                          // 2 x 16 KB  Q tiles, K-major, SW128
constexpr int kOffK = 32768;                      // kNK x 16 KB  K~ tiles
constexpr int kOffV = kOffK + kNK * 16384;        // kNV x 16 KB  V~ tiles
constexpr int kOffTab = kOffV + kNV * 16384;      // 2 x (K table 768 B + V table 2048 B) fp16 parameters
constexpr int kTabBytes = 768 + 2048;
constexpr int kOffBar = kOffTab + 2 * kTabBytes;  // barriers, tmem base, abort flag
constexpr int kBarBytes = 512;
constexpr int kOffRaw = kOffBar + kBarBytes;      // raw stages (16-byte aligned)
constexpr int kXchgBytes = 4096;                  // split softmax: values exchanged between the two halves of a row
template <int BITS, bool SPLIT = false> constexpr int smem_bytes() {
  return kOffRaw + Cfg<BITS>::kNR * Cfg<BITS>::kRawStage + (SPLIT ? kXchgBytes : 0) + 1024;
}

// tensor memory columns (all 512)
constexpr int kColS = 0;      // + 128 t : 128 fp32 columns per query tile
constexpr int kColP = 256;    // + 64 t  : 64 columns of packed 16-bit pairs
constexpr int kColO = 384;    // + 64 t  : 64 fp32 columns
// 16-warp form: one score buffer for both tiles, two P buffers per tile
constexpr int kColS1 = 0;     // 128 fp32 columns
constexpr int kColP2 = 128;   // + 128 t + 64 b
constexpr int kTmemCols = 512;

// one partial slot: two query tiles x 128 rows x (64 accumulators + max + sum)
constexpr size_t kSlotFloats = 2 * 128 * 64;
constexpr size_t kSlotBytes = kSlotFloats * sizeof(float) + 2 * 128 * sizeof(float2);

struct Args {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  int n;
  int64_t ts, hs;
  const uint8_t* k;
  const float2* kpar;
  const uint8_t* v;
  const float2* vpar;
  int cap, t_first, t_phys;
  float scale_log2;
  int n_tiles;          // key tiles of the cache
  int q_tiles;          // 128-row query tiles of the frame
  int n_pairs;          // ceil(q_tiles / 2)
  long long total;      // items * n_tiles
  float* part_o;        // [2 * grid][2][128][64]
  float2* part_ml;      // [2 * grid][2][128]
  int* status;
  // Newest frame unquantised (Eq. 1 read literally): when k_tail is set, the key slots
  // [tail_lo, t_phys) take K~, V~ from these bf16 tensors ([head][token][64] with the strides
  // below, token = slot - tail_lo) instead of the packed rows.
  const __nv_bfloat16* k_tail;
  const __nv_bfloat16* v_tail;
  int64_t tail_ts, tail_hs;
  int tail_lo;
  // Quantise-once mode: every token refers to the parameter-table slot of its key group
  // (kslot [cap]); ktab16 [slot][n_heads][8][12] holds, per 8-channel word, the four fp16 pairs
  // of scales, offsets and constants that dequant_word_h takes.
  const int32_t* kslot;
  const uint32_t* ktab16;
  int n_heads;
};

__device__ __forceinline__ long long piece_start(long long total, int grid, int b) {
  return (total * (long long)b) / (long long)grid;
}

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
constexpr uint32_t kSuspendNs = 2000;
// The same with a time the hardware may keep the thread suspended before it answers "not yet"
// (it answers at once when the phase completes).
__device__ __forceinline__ bool mbar_try_suspend(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
  return ok != 0;
}
// Up to 64 suspended tries in a loop of three instructions (try, branch out, count and branch back).
__device__ __forceinline__ bool mbar_try_many(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .pred q;\n\t.reg .u32 n;\n\t"
      "mov.u32 n, 64;\n\t"
      "XKV_TRY_%=:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "@p bra XKV_DONE_%=;\n\t"
      "sub.u32 n, n, 1;\n\t"
      "setp.ne.u32 q, n, 0;\n\t"
      "@q bra XKV_TRY_%=;\n\t"
      "XKV_DONE_%=:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  On exhaustion the failure is recorded (device status word and a
// per-CTA flag); once the flag is up every later wait of the CTA gives up at once.
struct WaitCtx { int* status; volatile int* abort_flag; };
// Threads on the critical chain (softmax warps, MMA issuers: SLEEP_NS below 128) retry at once, each
// try suspended by the hardware for a short while: their wake-up latency is part of every step.
// Threads that wait long and have slack (operand producers, the copy thread) sleep SLEEP_NS between
// tries, so that their polls (shared-memory instructions) do not take issue slots and queue space
// from the softmax warps.  The wait gives up after one second AND kWaitMinRounds rounds of tries
// (32 or 64 each): the rounds only count while the thread runs, so that a kernel that was
// descheduled for a while (a GPU shared between processes) does not time out on the clock alone.
constexpr uint64_t kWaitLimitNs = 1000000000ull;      // one second ...
constexpr uint32_t kWaitMinRounds = 1u << 12;         // ... and this many rounds, then XKV_E_TIMEOUT
template <int SLEEP_NS = 32>
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& wc) {
  if (mbar_try(bar, parity)) return;          // the common case costs one instruction
  if (*wc.abort_flag) return;
  const uint64_t t0 = global_ns();
  uint32_t rounds = 0;
  do {
    if (SLEEP_NS >= 128) {
#pragma unroll 1
      for (int it = 0; it < 32; ++it) {
        if (mbar_try_suspend(bar, parity, kSuspendNs)) return;
        __nanosleep(SLEEP_NS);
      }
    } else if (mbar_try_many(bar, parity)) {
      return;
    }
  } while (++rounds < kWaitMinRounds || global_ns() - t0 < kWaitLimitNs);
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

#define XKV_TMEM_LD16(taddr, r)                                                                      \
  asm volatile(                                                                                      \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                      \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"                              \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), \
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),     \
        "=r"(r[15])                                                                                  \
      : "r"(taddr) : "memory")

#define XKV_TMEM_ST8(taddr, r)                                                                       \
  asm volatile(                                                                                      \
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"                       \
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),     \
        "r"(r[7]) : "memory")

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


__device__ __forceinline__ uint32_t h2_fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

// Eight 4-bit codes of one packed word -> four fp16 pairs of s * (q - z)  (Eq. 10).
// (w & 0x000F000F) | 0x6400 is the fp16 number 1024 + q and (w & 0x00F000F0) | 0x5400 is 64 + q.
// Every pair is formed as  fma(biased - zo, s, c)  with the constants of dequant_consts.
// Pairs 0 and 2 of a word carry the bias 1024, pairs 1 and 3 the bias 64.
__device__ __forceinline__ uint4 dequant_word_h(uint32_t w, const uint32_t (&s2)[4], const uint32_t (&zo)[4],
                                                const uint32_t (&c2)[4]) {
  const uint32_t t = w >> 8;
  const uint32_t a0 = (w & 0x000F000Fu) | 0x64006400u;
  const uint32_t a1 = (w & 0x00F000F0u) | 0x54005400u;
  const uint32_t a2 = (t & 0x000F000Fu) | 0x64006400u;
  const uint32_t a3 = (t & 0x00F000F0u) | 0x54005400u;
  uint4 r;
  r.x = h2_fma(h2_sub(a0, zo[0]), s2[0], c2[0]);
  r.y = h2_fma(h2_sub(a1, zo[1]), s2[1], c2[1]);
  r.z = h2_fma(h2_sub(a2, zo[2]), s2[2], c2[2]);
  r.w = h2_fma(h2_sub(a3, zo[3]), s2[3], c2[3]);
  return r;
}

// The same for eight 8-bit codes (two words, channels 4i..4i+3 as c0 | c2<<8 | c1<<16 | c3<<24):
// (w & 0x00FF00FF) | 0x6400 is the fp16 pair (1024 + c0, 1024 + c1), the word shifted by 8 gives
// (1024 + c2, 1024 + c3); every pair carries the bias 1024.
__device__ __forceinline__ uint4 dequant_words8_h(uint2 w, const uint32_t (&s2)[4], const uint32_t (&zo)[4],
                                                  const uint32_t (&c2)[4]) {
  const uint32_t a0 = (w.x & 0x00FF00FFu) | 0x64006400u;
  const uint32_t a1 = ((w.x >> 8) & 0x00FF00FFu) | 0x64006400u;
  const uint32_t a2 = (w.y & 0x00FF00FFu) | 0x64006400u;
  const uint32_t a3 = ((w.y >> 8) & 0x00FF00FFu) | 0x64006400u;
  uint4 r;
  r.x = h2_fma(h2_sub(a0, zo[0]), s2[0], c2[0]);
  r.y = h2_fma(h2_sub(a1, zo[1]), s2[1], c2[1]);
  r.z = h2_fma(h2_sub(a2, zo[2]), s2[2], c2[2]);
  r.w = h2_fma(h2_sub(a3, zo[3]), s2[3], c2[3]);
  return r;
}

// fp16 can hold magnitudes up to 65504; anything beyond (or not a number) is reported.
__device__ __forceinline__ bool beyond_fp16(float x) { return !(fabsf(x) <= 65504.f); }
__device__ __noinline__ void report_range(int* status) { atomicCAS(status, 0, (int)XKV_E_RANGE); }

// true when one of the two fp16 numbers is an infinity or a NaN (all exponent bits set)
__device__ __forceinline__ bool h2_not_finite(uint32_t h) {
  return (h & 0x7C00u) == 0x7C00u || (h & 0x7C000000u) == 0x7C000000u;
}

// Eight bf16 values -> eight fp16 values (exact whenever the value is in fp16's range).
__device__ __forceinline__ uint4 bf16x8_to_h8(const uint4& u) {
  const uint32_t r[4] = {u.x, u.y, u.z, u.w};
  uint32_t h[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = pack_h2(__uint_as_float(r[i] << 16), __uint_as_float(r[i] & 0xFFFF0000u));
  return make_uint4(h[0], h[1], h[2], h[3]);
}

// Rows of the unquantised newest frame over the dequantised rows of a K~ or V~ tile: keys
// slot0 + 16 i of the tile that lie in [tail_lo, t_phys) are replaced by the caller's bf16 rows
// (src already points at this thread's head and 8-channel chunk).  A real call, so that the
// producers' loop carries none of this code.
__device__ __noinline__ void tail_rows_over(uint8_t* tile_row, const __nv_bfloat16* src, int64_t ts, int slot0,
                                            int tail_lo, int t_phys, int* status) {
  uint4 u[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int slot = slot0 + 16 * i;
    u[i] = make_uint4(0, 0, 0, 0);
    if (slot >= tail_lo && slot < t_phys) u[i] = *reinterpret_cast<const uint4*>(src + (int64_t)(slot - tail_lo) * ts);
  }
  uint32_t seen = 0u;       // exponent bits of everything written: all ones somewhere = beyond fp16
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int slot = slot0 + 16 * i;
    if (slot >= tail_lo && slot < t_phys) {
      const uint4 hv = bf16x8_to_h8(u[i]);
      *reinterpret_cast<uint4*>(tile_row + i * 2048) = hv;
      seen |= (h2_not_finite(hv.x) || h2_not_finite(hv.y) || h2_not_finite(hv.z) || h2_not_finite(hv.w)) ? 1u : 0u;
    }
  }
  if (seen) report_range(status);
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bulk asynchronous copy global -> this CTA's shared memory, completion counted on an mbarrier.
// Addresses 16-byte aligned, size a multiple of 16.  No multicast.
__device__ __forceinline__ void tma_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// O[row][0..63] *= alpha for the 32 rows (TMEM lanes) of the calling warp; a real call, to keep its
// registers out of the softmax loop.  Warp-collective.
__device__ __noinline__ void rescale_rows(uint32_t col_o, float alpha, int cols = 64) {
#pragma unroll 1
  for (int c0 = 0; c0 < cols; c0 += 32) {
    uint32_t ra[32];
    XKV_TMEM_LD32(col_o + c0, ra);
    tc_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) ra[i] = __float_as_uint(__uint_as_float(ra[i]) * alpha);
    XKV_TMEM_ST32(col_o + c0, ra);
  }
  tc_wait_st();
}
__device__ __forceinline__ void producer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

}  // namespace

// TAIL: the newest frame's keys and values come unquantised from Args::k_tail, v_tail (a separate
// instantiation, so that the kernel without a tail carries none of its code).
// ONCE: the keys' dequantisation constants are looked up per token (quantise-once mode) instead of
// per 64-slot run.
template <int BITS, bool TAIL = false, bool ONCE = false, bool SPLIT = false>
__global__ void __launch_bounds__(SPLIT ? kThreadsSplit : kThreads, 1) attn_tc_kernel(const Args a) {
  using C = Cfg<BITS>;
  constexpr int kSW = SPLIT ? 16 : 8;        // softmax warps
  constexpr uint32_t kRowThreads = SPLIT ? 256 : 128;   // threads that work on one query tile
  constexpr int kOffX = kOffRaw + C::kNR * C::kRawStage;   // exchange area of the split softmax
  constexpr int kRegProd = split_regs_producers(ONCE, TAIL), kRegMisc = split_regs_misc(ONCE, TAIL);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const uint32_t sQ = sbase + kOffQ, sK = sbase + kOffK, sV = sbase + kOffV, sRaw = sbase + kOffRaw;
  const uint32_t bar0 = sbase + kOffBar;
  // barrier slots (8 bytes each)
  const uint32_t b_kfull = bar0, b_kfree = bar0 + 8 * kNK;
  const uint32_t b_vfull = b_kfree + 8 * kNK, b_vfree = b_vfull + 8 * kNV;
  const uint32_t b_rfull = b_vfree + 8 * kNV, b_rfree = b_rfull + 8 * C::kNR;
  const uint32_t b_qfull = b_rfree + 8 * C::kNR;      // [2]
  const uint32_t b_sfull = b_qfull + 16, b_pfull = b_sfull + 16, b_pvdone = b_pfull + 16, b_sfree = b_pvdone + 16;
  const uint32_t b_pvdone2 = b_sfree + 16;             // [2 tiles][2 P buffers], 16-warp form
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sgen + kOffBar + kBarBytes - 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + kOffBar + kBarBytes - 12);
  const WaitCtx wc{a.status, abort_flag};

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  constexpr bool kBf16 = (BITS == 16);

  // this CTA's piece of the line of steps
  const long long step_lo = piece_start(a.total, gridDim.x, blockIdx.x);
  const long long step_hi = piece_start(a.total, gridDim.x, blockIdx.x + 1);

  if (tid == 0) {
    *abort_flag = (*reinterpret_cast<volatile int*>(a.status) == (int)XKV_E_TIMEOUT) ? 1 : 0;   // an earlier CTA already gave up
    for (int i = 0; i < kNK; ++i) { mbar_init(b_kfull + 8 * i, 128); mbar_init(b_kfree + 8 * i, 2); }
    for (int i = 0; i < kNV; ++i) { mbar_init(b_vfull + 8 * i, 128); mbar_init(b_vfree + 8 * i, 2); }
    for (int i = 0; i < C::kNR; ++i) { mbar_init(b_rfull + 8 * i, 1); mbar_init(b_rfree + 8 * i, 128); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(b_qfull + 8 * t, kRowThreads); mbar_init(b_sfull + 8 * t, 1);
      mbar_init(b_pfull + 8 * t, kRowThreads); mbar_init(b_pvdone + 8 * t, 1); mbar_init(b_sfree + 8 * t, kRowThreads);
      mbar_init(b_pvdone2 + 16 * t, 1); mbar_init(b_pvdone2 + 16 * t + 8, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kSW + 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (SPLIT) {
    // Registers move from the warps that need few to the softmax warps, which keep half a row of
    // scores in registers.  The pool is what the CTA was launched with (per scheduler 6 warps x 80
    // registers per lane = 480); afterwards 4 x 96 + 40 + 48 (or 56 + 40 where the producers look up
    // per-token constants) of them are in use: 472 or 480.
    if (warp < 16) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSplitRegsSoftmax));
    else if (warp < 20) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegProd));
    else asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegMisc));
  }

  if (SPLIT && warp < 16) {
    // ============== softmax warps, two per 32 rows of a query tile ==============
    // Warps w and w + 8 work on the same rows: each takes 64 of a key tile's 128 score columns, the
    // matching 32 columns of P and 32 of the accumulator.  A thread reads its half row of scores
    // into registers at once and releases the score columns, so that the next S = Q K~^T runs while
    // the exponentials are computed.  What the row needs as a whole (its maximum, its sum) the two
    // threads exchange through shared memory.
    const int t = (warp >> 2) & 1;           // query tile of the pair
    const int hf = warp >> 3;                // half of the key columns
    const int r = (warp & 3) * 32 + (tid & 31);   // row of the tile = TMEM lane
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    // tensor memory of this form: one score buffer that the two tiles use in turn (a tile holds it
    // only from its MMAs to its loads), two P buffers per tile, one accumulator per tile
    const uint32_t colS = lane_addr + kColS1 + 64 * hf, colP0 = lane_addr + kColP2 + 128 * t + 32 * hf;
    const uint32_t colO = lane_addr + kColO + 64 * t + 32 * hf;
    const uint32_t sfull = b_sfull + 8 * t, pfull = b_pfull + 8 * t, pvdone2 = b_pvdone2 + 16 * t;
    const int pad_tile = (a.t_first & 127) ? (a.t_first >> 7) : -1;
    const uint64_t sc2 = pack_f2(a.scale_log2, a.scale_log2);
    const int pair_bar = 2 + (warp & 7);     // named barrier of the two warps with these rows
    volatile float* xmine = reinterpret_cast<volatile float*>(sgen + kOffX) + ((t * 2 + hf) * 128 + r);
    volatile float* xpeer = reinterpret_cast<volatile float*>(sgen + kOffX) + ((t * 2 + (hf ^ 1)) * 128 + r);
    uint32_t xc = 0;
    // One value per thread to the thread of the other half with the same row.  Two buffers in turn:
    // a value is overwritten two exchanges later, after a barrier the reader has passed since.
    auto exchange = [&](float v) -> float {
      const uint32_t o = (xc++ & 1) * 512;
      xmine[o] = v;
      __syncwarp();
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      return xpeer[o];
    };
    uint32_t cnt = 0;                        // steps this tile has been through (barrier phases)
    uint32_t g_seg = 0;                      // uses of the score buffer (both tiles) before this segment
    int seg_idx = 0;
    for (long long pos = step_lo; pos < step_hi; ++seg_idx) {
      const int item = (int)(pos / a.n_tiles);
      const int tile_lo = (int)(pos - (long long)item * a.n_tiles);
      const int nt = (int)min((long long)(a.n_tiles - tile_lo), step_hi - pos);
      pos += nt;
      const int h = item / a.n_pairs, pair = item - h * a.n_pairs;
      const int qt = 2 * pair + t;
      const uint32_t per_step = (2 * pair + 1 < a.q_tiles) ? 2u : 1u;   // tiles that use the score buffer
      const uint32_t use0 = g_seg + (uint32_t)t;     // this tile's uses: use0 + jj * per_step
      g_seg += (uint32_t)nt * per_step;
      if (qt >= a.q_tiles) continue;          // the pair has no second tile
      // ---- Q tile: half of row r, bf16 -> operand type, into the swizzled K-major layout ----
      const int row = qt * kQRows + r;
      {
        uint4 u[4];
        if (row < a.n) {
          const __nv_bfloat16* qp = a.q + (int64_t)h * a.hs + (int64_t)row * a.ts + 32 * hf;
#pragma unroll
          for (int c = 0; c < 4; ++c) u[c] = *reinterpret_cast<const uint4*>(qp + 8 * c);
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) u[c] = make_uint4(0, 0, 0, 0);
        }
        bool q_bad = false;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 o = u[c];
          if (!kBf16) {
            const uint32_t rr[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
            uint32_t hh[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              hh[i] = pack_h2(__uint_as_float(rr[i] << 16), __uint_as_float(rr[i] & 0xFFFF0000u));
              q_bad |= h2_not_finite(hh[i]);
            }
            o = make_uint4(hh[0], hh[1], hh[2], hh[3]);
          }
          *reinterpret_cast<uint4*>(sgen + kOffQ + t * 16384 + swz_off(r, 4 * hf + c)) = o;
        }
        if (q_bad) report_range(a.status);
        fence_proxy_async();
        mbar_arrive(b_qfull + 8 * t);
      }
      float m_ref = -INFINITY;   // reference maximum of the row (scaled, log2 units; the same in both halves)
      uint64_t l2 = 0ull, l2b = 0ull;   // four partial sums of this half of the row (two packed fp32 pairs)
      for (int jj = 0; jj < nt; ++jj, ++cnt) {
        const int tile = tile_lo + jj;
        int lim = 128;           // columns [lim, 128) are masked (pad slots after the first frame, the tail)
        if (tile == pad_tile) lim = a.t_first & 127;
        if (tile == a.n_tiles - 1) lim = min(lim, a.t_phys - tile * 128);
        mbar_wait(sfull, cnt & 1, wc);
        __syncwarp();            // the waits may leave the warp diverged; tcgen05.ld/st are warp-collective
        tc_fence_after();
        // ---- this half of the scores (64 columns) into registers; after that the score columns
        // may take the next tile's scores ----
        uint32_t ra[32], rb[32];
        XKV_TMEM_LD32(colS, ra);
        XKV_TMEM_LD32(colS + 32, rb);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(b_sfree + 8 * ((use0 + (uint32_t)jj * per_step) & 1));    // uses alternate between two barriers
        if (lim < 128) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (64 * hf + i >= lim) ra[i] = 0xff800000u;           // -inf: exponential 0
            if (64 * hf + 32 + i >= lim) rb[i] = 0xff800000u;
          }
        }
        float mx1 = -INFINITY, mx2 = -INFINITY;      // two chains of 16, not one of 32
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          mx1 = max3(mx1, __uint_as_float(ra[i]), __uint_as_float(ra[i + 1]));
          mx2 = max3(mx2, __uint_as_float(rb[i]), __uint_as_float(rb[i + 1]));
        }
        float mx = fmaxf(mx1, mx2);
        mx = fmaxf(mx, exchange(mx)) * a.scale_log2;
        // The reference maximum moves only when the row maximum grew by more than 2^kGrow over it;
        // then the sums and (at the end of the step, when the registers are free) the accumulator
        // are rescaled.  Every tile has a column that is not masked, so mx is finite.
        float alpha = 1.f;
        const bool grow = mx > m_ref + kGrow;
        if (grow) {
          alpha = exp2f(m_ref - mx);      // 0 on the first tile (m_ref = -inf)
          m_ref = mx;
          l2 = mul_f2(l2, pack_f2(alpha, alpha));
          l2b = mul_f2(l2b, pack_f2(alpha, alpha));
        }
        const uint64_t nm2 = pack_f2(-m_ref, -m_ref);
        const uint32_t colP = colP0 + 64 * (cnt & 1);
        // exponentials of 16 columns against the reference; P (16-bit pairs) -> TMEM
        auto chunk16 = [&](const uint32_t* rr, int c) {
          uint64_t x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            x[i] = fma_f2(pack_f2(__uint_as_float(rr[2 * i]), __uint_as_float(rr[2 * i + 1])), sc2, nm2);
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = pack_f2(fast_exp2(f2_lo(x[i])), fast_exp2(f2_hi(x[i])));
          uint32_t pk[8];
#pragma unroll
          for (int i = 0; i < 8; i += 2) {
            l2 = add_f2(l2, x[i]);
            l2b = add_f2(l2b, x[i + 1]);
            pk[i] = kBf16 ? pack_bf2(f2_lo(x[i]), f2_hi(x[i])) : pack_h2(f2_lo(x[i]), f2_hi(x[i]));
            pk[i + 1] = kBf16 ? pack_bf2(f2_lo(x[i + 1]), f2_hi(x[i + 1])) : pack_h2(f2_lo(x[i + 1]), f2_hi(x[i + 1]));
          }
          if (c == 0 && cnt >= 2) {  // this P buffer's previous contents (two steps ago) consumed
            mbar_wait(pvdone2 + 8 * (cnt & 1), ((cnt >> 1) - 1) & 1, wc);
            __syncwarp();
            tc_fence_after();
          }
          XKV_TMEM_ST8(colP + 8 * c, pk);
        };
        chunk16(ra, 0);
        chunk16(ra + 16, 1);
        chunk16(rb, 2);
        chunk16(rb + 16, 3);
        if (jj > 0 && __any_sync(0xffffffffu, grow)) {
          // the accumulator is quiescent once the previous step's PV has completed
          mbar_wait(pvdone2 + 8 * ((cnt - 1) & 1), ((cnt - 1) >> 1) & 1, wc);
          __syncwarp();
          tc_fence_after();
          rescale_rows(colO, alpha, 32);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(pfull);
      }
      // ---- epilogue of the segment: 32 channels of the row per thread ----
      mbar_wait(pvdone2 + 8 * ((cnt - 1) & 1), ((cnt - 1) >> 1) & 1, wc);    // the last PV (they complete in order)
      __syncwarp();
      tc_fence_after();
      const float l_half = (f2_lo(l2) + f2_hi(l2)) + (f2_lo(l2b) + f2_hi(l2b));
      const float l_peer = exchange(l_half);
      const float l = hf ? (l_peer + l_half) : (l_half + l_peer);     // the same sum in both halves
      const bool whole = (tile_lo == 0 && nt == a.n_tiles);
      uint32_t ro[32];
      XKV_TMEM_LD32(colO, ro);
      tc_wait_ld();
      if (whole) {
        const float inv_l = 1.f / l;
        if (row < a.n) {
          __nv_bfloat16* op = a.out + (int64_t)h * a.hs + (int64_t)row * a.ts + 32 * hf;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              o[i] = pack_bf2(__uint_as_float(ro[8 * c + 2 * i]) * inv_l, __uint_as_float(ro[8 * c + 2 * i + 1]) * inv_l);
            *reinterpret_cast<uint4*>(op + 8 * c) = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
      } else {
        const size_t slot = (size_t)2 * blockIdx.x + (seg_idx == 0 ? 0 : 1);
        const size_t prow = (slot * 2 + t) * 128 + r;
        float4* dst = reinterpret_cast<float4*>(a.part_o + prow * 64 + 32 * hf);
#pragma unroll
        for (int c = 0; c < 8; ++c)
          dst[c] = make_float4(__uint_as_float(ro[4 * c]), __uint_as_float(ro[4 * c + 1]),
                               __uint_as_float(ro[4 * c + 2]), __uint_as_float(ro[4 * c + 3]));
        if (hf == 0) a.part_ml[prow] = make_float2(m_ref, l);
      }
      tc_fence_before();
    }
  } else if (!SPLIT && warp < 8) {
    // =========================== softmax warps ===============================
    const int t = warp >> 2;                 // query tile of the pair
    const int r = tid & 127;                 // row of the tile = TMEM lane
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t colS = lane_addr + kColS + 128 * t, colP = lane_addr + kColP + 64 * t;
    const uint32_t colO = lane_addr + kColO + 64 * t;
    const uint32_t sfull = b_sfull + 8 * t, pfull = b_pfull + 8 * t, pvdone = b_pvdone + 8 * t, sfree = b_sfree + 8 * t;
    const int pad_tile = (a.t_first & 127) ? (a.t_first >> 7) : -1;
    const uint64_t sc2 = pack_f2(a.scale_log2, a.scale_log2);
    uint32_t cnt = 0;                        // steps this tile has been through (barrier phases)
    int seg_idx = 0;
    for (long long pos = step_lo; pos < step_hi; ++seg_idx) {
      const int item = (int)(pos / a.n_tiles);
      const int tile_lo = (int)(pos - (long long)item * a.n_tiles);
      const int nt = (int)min((long long)(a.n_tiles - tile_lo), step_hi - pos);
      pos += nt;
      const int h = item / a.n_pairs, pair = item - h * a.n_pairs;
      const int qt = 2 * pair + t;
      if (qt >= a.q_tiles) continue;          // the pair has no second tile
      // ---- Q tile: row r, bf16 -> operand type, into the swizzled K-major layout ----
      const int row = qt * kQRows + r;
      {
        uint4 u[8];
        if (row < a.n) {
          const __nv_bfloat16* qp = a.q + (int64_t)h * a.hs + (int64_t)row * a.ts;
#pragma unroll
          for (int c = 0; c < 8; ++c) u[c] = *reinterpret_cast<const uint4*>(qp + 8 * c);
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c) u[c] = make_uint4(0, 0, 0, 0);
        }
        bool q_bad = false;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint4 o = u[c];
          if (!kBf16) {
            const uint32_t rr[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
            uint32_t hh[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              hh[i] = pack_h2(__uint_as_float(rr[i] << 16), __uint_as_float(rr[i] & 0xFFFF0000u));
              q_bad |= h2_not_finite(hh[i]);
            }
            o = make_uint4(hh[0], hh[1], hh[2], hh[3]);
          }
          *reinterpret_cast<uint4*>(sgen + kOffQ + t * 16384 + swz_off(r, c)) = o;
        }
        if (q_bad) report_range(a.status);
        fence_proxy_async();
        mbar_arrive(b_qfull + 8 * t);
      }
      float m_ref = -INFINITY;   // reference maximum (scaled, log2 units) used for the exponentials
      uint64_t l2 = 0ull;        // two partial row sums (packed fp32 pair)
      for (int jj = 0; jj < nt; ++jj, ++cnt) {
        const int tile = tile_lo + jj;
        int lim = 128;           // columns [lim, 128) are masked (pad slots after the first frame, the tail)
        if (tile == pad_tile) lim = a.t_first & 127;
        if (tile == a.n_tiles - 1) lim = min(lim, a.t_phys - tile * 128);
        mbar_wait(sfull, cnt & 1, wc);
        __syncwarp();            // the spin loops may leave the warp diverged; tcgen05.ld/st are warp-collective
        tc_fence_after();
        bool pv_waited = (jj == 0);   // P of the previous step consumed, O quiescent (its PV completed)
        auto wait_pv = [&]() {
          if (!pv_waited) {
            mbar_wait(pvdone, (cnt - 1) & 1, wc);
            __syncwarp();
            tc_fence_after();
            pv_waited = true;
          }
        };
        // The reference maximum m_ref moves only when the row maximum grew by more than 2^14 over
        // it: then the row sum and the accumulator are rescaled.
        auto apply_max = [&](float mx_scaled) {
          float alpha = 1.f;
          const bool grow = mx_scaled > m_ref + kGrow;
          if (grow) {
            alpha = exp2f(m_ref - mx_scaled);      // 0 on the first tile (m_ref = -inf)
            m_ref = mx_scaled;
            l2 = mul_f2(l2, pack_f2(alpha, alpha));
          }
          if (jj > 0) {
            wait_pv();
            if (__any_sync(0xffffffffu, grow)) rescale_rows(colO, alpha);
          }
        };
        if (lim >= 128) {
          // ---- full tile.  Exponentials against the current reference in one pass over S.  The
          // pass is valid when no exponential exceeded 2^kGrow; that is checked on the row sum of
          // the first 96 columns and the maximum of the last 32.  Otherwise (always on the first
          // tile of a segment, rarely afterwards) the row maximum is taken first, the reference
          // moves, and the pass is repeated. ----
          uint64_t lt2;
#pragma unroll 1
          for (int attempt = 0; attempt < 2; ++attempt) {
            if (jj == 0 || attempt == 1) {
              float mx = -INFINITY;
#pragma unroll 1
              for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t ra[32];
                XKV_TMEM_LD32(colS + c0, ra);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 2) mx = max3(mx, __uint_as_float(ra[i]), __uint_as_float(ra[i + 1]));
              }
              apply_max(mx * a.scale_log2);
            }
            const bool last_attempt = (jj == 0 || attempt == 1);
            const uint64_t nm2 = pack_f2(-m_ref, -m_ref);
            lt2 = 0ull;
            bool redo = false;
            uint32_t ra[32], rb[32];
            // exponentials of 32 columns against the reference; P (16-bit pairs) -> TMEM
            // Written in three sweeps over the chunk (scale and shift, exponentials, sums and
            // conversion), each of 16 or 32 independent operations, so that the latency of the
            // special-function unit is covered inside one warp.
            auto chunk = [&](uint32_t (&rr)[32], int c) {
              uint64_t x[16];
#pragma unroll
              for (int i = 0; i < 16; ++i)
                x[i] = fma_f2(pack_f2(__uint_as_float(rr[2 * i]), __uint_as_float(rr[2 * i + 1])), sc2, nm2);
#pragma unroll
              for (int i = 0; i < 16; ++i) x[i] = pack_f2(fast_exp2(f2_lo(x[i])), fast_exp2(f2_hi(x[i])));
              uint32_t pk[16];
              uint64_t s0 = 0ull, s1 = 0ull;
#pragma unroll
              for (int i = 0; i < 16; i += 2) {
                s0 = add_f2(s0, x[i]);
                s1 = add_f2(s1, x[i + 1]);
                pk[i] = kBf16 ? pack_bf2(f2_lo(x[i]), f2_hi(x[i])) : pack_h2(f2_lo(x[i]), f2_hi(x[i]));
                pk[i + 1] = kBf16 ? pack_bf2(f2_lo(x[i + 1]), f2_hi(x[i + 1])) : pack_h2(f2_lo(x[i + 1]), f2_hi(x[i + 1]));
              }
              lt2 = add_f2(lt2, add_f2(s0, s1));
              if (c == 0) wait_pv();
              XKV_TMEM_ST16(colP + 16 * c, pk);
            };
            XKV_TMEM_LD32(colS, ra);
            tc_wait_ld();
#pragma unroll 1
            for (int c = 0; c < 4; c += 2) {
              XKV_TMEM_LD32(colS + 32 * (c + 1), rb);          // in flight while chunk c is processed
              chunk(ra, c);
              tc_wait_ld();
              if (c == 0) {
                XKV_TMEM_LD32(colS + 64, ra);
              } else {
                // all of S is in registers: unless the pass has to be repeated, the score columns
                // can take the next tile's scores already
                if (!last_attempt) {
                  float mxl = -INFINITY;
#pragma unroll
                  for (int i = 0; i < 32; i += 2) mxl = max3(mxl, __uint_as_float(rb[i]), __uint_as_float(rb[i + 1]));
                  const float part = f2_lo(lt2) + f2_hi(lt2);
                  const bool bad = !(part < 16384.f) || (mxl * a.scale_log2 > m_ref + kGrow);
                  redo = __any_sync(0xffffffffu, bad);
                }
                if (!redo) { tc_fence_before(); mbar_arrive(sfree); }
              }
              chunk(rb, c + 1);
              if (c == 0) tc_wait_ld();
            }
            if (!redo) break;
            tc_wait_st();
          }
          l2 = add_f2(l2, lt2);
        } else {
          // ---- masked tile (pad slots after the first frame, the tail): two plain passes ----
          float mx = -INFINITY;
#pragma unroll 1
          for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t ra[32];
            XKV_TMEM_LD32(colS + c0, ra);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float x = (c0 + i < lim) ? __uint_as_float(ra[i]) : -INFINITY;
              mx = fmaxf(mx, x);
            }
          }
          apply_max(mx * a.scale_log2);
          wait_pv();
#pragma unroll 1
          for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t ra[32];
            XKV_TMEM_LD32(colS + c0, ra);
            tc_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float p0 = fast_exp2(fmaf(__uint_as_float(ra[2 * i]), a.scale_log2, -m_ref));
              float p1 = fast_exp2(fmaf(__uint_as_float(ra[2 * i + 1]), a.scale_log2, -m_ref));
              if (c0 + 2 * i >= lim) p0 = 0.f;
              if (c0 + 2 * i + 1 >= lim) p1 = 0.f;
              l2 = add_f2(l2, pack_f2(p0, p1));
              pk[i] = kBf16 ? pack_bf2(p0, p1) : pack_h2(p0, p1);
            }
            XKV_TMEM_ST16(colP + (c0 >> 1), pk);
          }
          tc_fence_before();
          mbar_arrive(sfree);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(pfull);
      }
      // ---- epilogue of the segment ----
      mbar_wait(pvdone, (cnt - 1) & 1, wc);
      __syncwarp();
      tc_fence_after();
      const float l = f2_lo(l2) + f2_hi(l2);
      const bool whole = (tile_lo == 0 && nt == a.n_tiles);
      if (whole) {
        const float inv_l = 1.f / l;
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t ra[32];
          XKV_TMEM_LD32(colO + c0, ra);
          tc_wait_ld();
          if (row < a.n) {
            __nv_bfloat16* op = a.out + (int64_t)h * a.hs + (int64_t)row * a.ts + c0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t o[4];
#pragma unroll
              for (int i = 0; i < 4; ++i)
                o[i] = pack_bf2(__uint_as_float(ra[8 * c + 2 * i]) * inv_l, __uint_as_float(ra[8 * c + 2 * i + 1]) * inv_l);
              *reinterpret_cast<uint4*>(op + 8 * c) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
        }
      } else {
        const size_t slot = (size_t)2 * blockIdx.x + (seg_idx == 0 ? 0 : 1);
        const size_t prow = (slot * 2 + t) * 128 + r;
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t ra[32];
          XKV_TMEM_LD32(colO + c0, ra);
          tc_wait_ld();
          float4* dst = reinterpret_cast<float4*>(a.part_o + prow * 64 + c0);
#pragma unroll
          for (int c = 0; c < 8; ++c)
            dst[c] = make_float4(__uint_as_float(ra[4 * c]), __uint_as_float(ra[4 * c + 1]),
                                 __uint_as_float(ra[4 * c + 2]), __uint_as_float(ra[4 * c + 3]));
        }
        a.part_ml[prow] = make_float2(m_ref, l);
      }
      tc_fence_before();
    }
  } else if (warp < kSW + 4) {
    // =========================== operand producers ===========================
    const int t = tid - 32 * kSW;
    const int w = t & 7;          // 16-byte chunk = 8 channels
    const int kb = t >> 3;        // keys kb + 16 i
    const uint32_t row_off = (uint32_t)((kb >> 3) * 1024 + (kb & 7) * 128 + ((w ^ (kb & 7)) << 4));
    uint32_t g = 0;               // steps so far (ring positions)
    for (long long pos = step_lo; pos < step_hi;) {
      const int item = (int)(pos / a.n_tiles);
      const int tile_lo = (int)(pos - (long long)item * a.n_tiles);
      const int nt = (int)min((long long)(a.n_tiles - tile_lo), step_hi - pos);
      pos += nt;
      const int h = item / a.n_pairs;
      for (int jj = 0; jj < nt; ++jj, ++g) {
        // keys of this tile that belong to the unquantised newest frame (none without a tail)
        const int slot0 = (tile_lo + jj) * 128 + kb;              // this thread's keys: slot0 + 16 i
        const bool tail_tile = TAIL && BITS == 4 && (tile_lo + jj) * 128 + 127 >= a.tail_lo;
        const int64_t tail_off = (int64_t)h * a.tail_hs + 8 * w;
        const uint32_t rs = g % C::kNR, ru = g / C::kNR;
        const uint32_t kbuf = g % kNK, ku = g / kNK;
        const uint32_t vbuf = g % kNV, vu = g / kNV;
        const uint8_t* raw = sgen + kOffRaw + rs * C::kRawStage;
        mbar_wait<256>(b_rfull + 8 * rs, ru & 1, wc);
        if (TAIL && BITS == 4 && (tile_lo + jj) * 128 >= a.tail_lo && (tile_lo + jj) * 128 + 127 < a.t_phys) {
          // ---- a tile that lies in the unquantised frame as a whole: K~ and V~ are the caller's
          // bf16 rows converted to fp16, the packed codes of the stage are not looked at ----
          bool bad = false;
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            const __nv_bfloat16* src = (kv ? a.v_tail : a.k_tail) + tail_off + (int64_t)(slot0 - a.tail_lo) * a.tail_ts;
            uint4 u[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) u[i] = *reinterpret_cast<const uint4*>(src + (int64_t)(16 * i) * a.tail_ts);
            if (kv == 0) mbar_wait<256>(b_kfree + 8 * kbuf, (ku & 1) ^ 1, wc);
            else mbar_wait<256>(b_vfree + 8 * vbuf, (vu & 1) ^ 1, wc);
            uint8_t* dst = sgen + (kv ? kOffV + vbuf * 16384 : kOffK + kbuf * 16384) + row_off;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint4 hv = bf16x8_to_h8(u[i]);
              bad |= h2_not_finite(hv.x) || h2_not_finite(hv.y) || h2_not_finite(hv.z) || h2_not_finite(hv.w);
              *reinterpret_cast<uint4*>(dst + i * 2048) = hv;
            }
            fence_proxy_async();
            mbar_arrive(kv ? b_vfull + 8 * vbuf : b_kfull + 8 * kbuf);
          }
          if (bad) report_range(a.status);
          mbar_arrive(b_rfree + 8 * rs);
          continue;
        }
        if (BITS == 4) {
          // ---- fp16 parameter tables of this tile (one (group, channel) and one key per thread) ----
          uint8_t* tab = sgen + kOffTab + (g & 1) * kTabBytes;
          {
            bool k_bad = false;
            if (!ONCE) {
              const float2 kp = *reinterpret_cast<const float2*>(raw + C::kRawK + C::kRawV + 8 * t);  // (group t>>6, channel t&63)
              float zl, zh, kc;
              dequant_consts(kp.x, kp.y, zl, zh, kc);
              __half* ks = reinterpret_cast<__half*>(tab);              // [2][64] scales, [2][64] offsets, [2][64] constants
              ks[t] = __float2half_rn(kp.x);
              ks[128 + t] = __float2half_rn((((t & 7) >> 1) & 1) ? zh : zl);
              ks[256 + t] = __float2half_rn(kc);
              k_bad = beyond_fp16(fabsf(kp.x) * (fabsf(kp.y) + 15.f));
            }
            const float2 vp = *reinterpret_cast<const float2*>(raw + C::kRawK + C::kRawV + C::kRawKP + 8 * t);   // key t
            float vl, vh, vc;
            dequant_consts(vp.x, vp.y, vl, vh, vc);
            *reinterpret_cast<uint4*>(tab + 768 + 16 * t) =
                make_uint4(pack_h2(vp.x, vp.x), pack_h2(vl, vl), pack_h2(vh, vh), pack_h2(vc, vc));
            // largest magnitude a code of this group / token can dequantise to
            if (k_bad || beyond_fp16(fabsf(vp.x) * (fabsf(vp.y) + 15.f))) report_range(a.status);
          }
          producer_sync();
          // ---- keys ----
          uint32_t wd[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) wd[i] = *reinterpret_cast<const uint32_t*>(raw + (kb + 16 * i) * 32 + 4 * w);
          if (ONCE) {
            // constants of each token's own key group, from the table in global memory (the tokens of
            // a group mostly sit next to each other, so the lines are shared); two tokens at a time,
            // the next two fetched while these are dequantised
            const uint8_t* slp = raw + C::kRawK + C::kRawV + 4 * kb;      // group references of keys kb + 16 i
            auto entry = [&](int i) {
              const int sl = *reinterpret_cast<const int*>(slp + 64 * i);
              return reinterpret_cast<const uint4*>(a.ktab16 + (((size_t)sl * a.n_heads + h) * 8 + w) * 12);
            };
            uint4 sv[2], zv[2], cv[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) { const uint4* e = entry(i); sv[i] = __ldg(e); zv[i] = __ldg(e + 1); cv[i] = __ldg(e + 2); }
            mbar_wait<256>(b_kfree + 8 * kbuf, (ku & 1) ^ 1, wc);
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) {
              uint4 o[2];
#pragma unroll
              for (int i = 0; i < 2; ++i) {
                const uint32_t s2[4] = {sv[i].x, sv[i].y, sv[i].z, sv[i].w}, zo[4] = {zv[i].x, zv[i].y, zv[i].z, zv[i].w};
                const uint32_t c2[4] = {cv[i].x, cv[i].y, cv[i].z, cv[i].w};
                o[i] = dequant_word_h(wd[2 * q2 + i], s2, zo, c2);
              }
              if (q2 < 3) {
#pragma unroll
                for (int i = 0; i < 2; ++i) { const uint4* e = entry(2 * q2 + 2 + i); sv[i] = __ldg(e); zv[i] = __ldg(e + 1); cv[i] = __ldg(e + 2); }
              }
#pragma unroll
              for (int i = 0; i < 2; ++i)
                *reinterpret_cast<uint4*>(sgen + kOffK + kbuf * 16384 + row_off + (2 * q2 + i) * 2048) = o[i];
            }
          } else {
          mbar_wait<256>(b_kfree + 8 * kbuf, (ku & 1) ^ 1, wc);
#pragma unroll
          for (int grp = 0; grp < 2; ++grp) {
            const uint4 sv = *reinterpret_cast<const uint4*>(tab + grp * 128 + 16 * w);
            const uint4 zv = *reinterpret_cast<const uint4*>(tab + 256 + grp * 128 + 16 * w);
            const uint4 cv = *reinterpret_cast<const uint4*>(tab + 512 + grp * 128 + 16 * w);
            const uint32_t s2[4] = {sv.x, sv.y, sv.z, sv.w}, zo[4] = {zv.x, zv.y, zv.z, zv.w};
            const uint32_t c2[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint4 o = dequant_word_h(wd[4 * grp + i], s2, zo, c2);
              *reinterpret_cast<uint4*>(sgen + kOffK + kbuf * 16384 + row_off + (4 * grp + i) * 2048) = o;
            }
          }
          }
          if (TAIL && tail_tile)
            tail_rows_over(sgen + kOffK + kbuf * 16384 + row_off, a.k_tail + tail_off, a.tail_ts, slot0, a.tail_lo, a.t_phys, a.status);
          fence_proxy_async();
          mbar_arrive(b_kfull + 8 * kbuf);
          // ---- values ----
#pragma unroll
          for (int i = 0; i < 8; ++i) wd[i] = *reinterpret_cast<const uint32_t*>(raw + C::kRawK + (kb + 16 * i) * 32 + 4 * w);
          mbar_wait<256>(b_vfree + 8 * vbuf, (vu & 1) ^ 1, wc);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 pv = *reinterpret_cast<const uint4*>(tab + 768 + 16 * (kb + 16 * i));
            const uint32_t s2[4] = {pv.x, pv.x, pv.x, pv.x}, zo[4] = {pv.y, pv.z, pv.y, pv.z};
            const uint32_t c2[4] = {pv.w, pv.w, pv.w, pv.w};
            const uint4 o = dequant_word_h(wd[i], s2, zo, c2);
            *reinterpret_cast<uint4*>(sgen + kOffV + vbuf * 16384 + row_off + i * 2048) = o;
          }
          if (TAIL && tail_tile)
            tail_rows_over(sgen + kOffV + vbuf * 16384 + row_off, a.v_tail + tail_off, a.tail_ts, slot0, a.tail_lo, a.t_phys, a.status);
          fence_proxy_async();
          mbar_arrive(b_vfull + 8 * vbuf);
          // The raw stage is released only here, after the words read from it have been used and
          // the fence above: released right after the loads, the refill of the stage was observed
          // to reach some of those loads when the wait in between was long.
          mbar_arrive(b_rfree + 8 * rs);
        } else if (BITS == 8) {
          // ---- 8-bit codes (keys quantised once): the same steps with rows of 64 bytes ----
          uint8_t* tab = sgen + kOffTab + (g & 1) * kTabBytes;
          {
            const float2 vp = *reinterpret_cast<const float2*>(raw + C::kRawK + C::kRawV + C::kRawKP + 8 * t);   // key t
            float vl, vh, vc;
            dequant_consts(vp.x, vp.y, vl, vh, vc);
            *reinterpret_cast<uint4*>(tab + 768 + 16 * t) = make_uint4(pack_h2(vp.x, vp.x), pack_h2(vl, vl), 0u, pack_h2(vc, vc));
            if (beyond_fp16(fabsf(vp.x) * (fabsf(vp.y) + 255.f))) report_range(a.status);
          }
          producer_sync();
          uint2 wd8[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) wd8[i] = *reinterpret_cast<const uint2*>(raw + (kb + 16 * i) * 64 + 8 * w);
          const uint8_t* slp = raw + C::kRawK + C::kRawV + 4 * kb;      // group references of keys kb + 16 i
          auto entry = [&](int i) {
            const int sl = *reinterpret_cast<const int*>(slp + 64 * i);
            return reinterpret_cast<const uint4*>(a.ktab16 + (((size_t)sl * a.n_heads + h) * 8 + w) * 12);
          };
          uint4 sv[2], zv[2], cv[2];
#pragma unroll
          for (int i = 0; i < 2; ++i) { const uint4* e = entry(i); sv[i] = __ldg(e); zv[i] = __ldg(e + 1); cv[i] = __ldg(e + 2); }
          mbar_wait<256>(b_kfree + 8 * kbuf, (ku & 1) ^ 1, wc);
#pragma unroll
          for (int q2 = 0; q2 < 4; ++q2) {
            uint4 o[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              const uint32_t s2[4] = {sv[i].x, sv[i].y, sv[i].z, sv[i].w}, zo[4] = {zv[i].x, zv[i].y, zv[i].z, zv[i].w};
              const uint32_t c2[4] = {cv[i].x, cv[i].y, cv[i].z, cv[i].w};
              o[i] = dequant_words8_h(wd8[2 * q2 + i], s2, zo, c2);
            }
            if (q2 < 3) {
#pragma unroll
              for (int i = 0; i < 2; ++i) { const uint4* e = entry(2 * q2 + 2 + i); sv[i] = __ldg(e); zv[i] = __ldg(e + 1); cv[i] = __ldg(e + 2); }
            }
#pragma unroll
            for (int i = 0; i < 2; ++i)
              *reinterpret_cast<uint4*>(sgen + kOffK + kbuf * 16384 + row_off + (2 * q2 + i) * 2048) = o[i];
          }
          fence_proxy_async();
          mbar_arrive(b_kfull + 8 * kbuf);
#pragma unroll
          for (int i = 0; i < 8; ++i) wd8[i] = *reinterpret_cast<const uint2*>(raw + C::kRawK + (kb + 16 * i) * 64 + 8 * w);
          mbar_wait<256>(b_vfree + 8 * vbuf, (vu & 1) ^ 1, wc);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 pv = *reinterpret_cast<const uint4*>(tab + 768 + 16 * (kb + 16 * i));
            const uint32_t s2[4] = {pv.x, pv.x, pv.x, pv.x}, zo[4] = {pv.y, pv.y, pv.y, pv.y};
            const uint32_t c2[4] = {pv.w, pv.w, pv.w, pv.w};
            const uint4 o = dequant_words8_h(wd8[i], s2, zo, c2);
            *reinterpret_cast<uint4*>(sgen + kOffV + vbuf * 16384 + row_off + i * 2048) = o;
          }
          fence_proxy_async();
          mbar_arrive(b_vfull + 8 * vbuf);
          mbar_arrive(b_rfree + 8 * rs);
        } else {
          uint4 rowk[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) rowk[i] = *reinterpret_cast<const uint4*>(raw + (kb + 16 * i) * 128 + 16 * w);
          mbar_wait<256>(b_kfree + 8 * kbuf, (ku & 1) ^ 1, wc);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint4*>(sgen + kOffK + kbuf * 16384 + row_off + i * 2048) = rowk[i];
          fence_proxy_async();
          mbar_arrive(b_kfull + 8 * kbuf);
#pragma unroll
          for (int i = 0; i < 8; ++i) rowk[i] = *reinterpret_cast<const uint4*>(raw + C::kRawK + (kb + 16 * i) * 128 + 16 * w);
          mbar_wait<256>(b_vfree + 8 * vbuf, (vu & 1) ^ 1, wc);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint4*>(sgen + kOffV + vbuf * 16384 + row_off + i * 2048) = rowk[i];
          fence_proxy_async();
          mbar_arrive(b_vfull + 8 * vbuf);
          mbar_arrive(b_rfree + 8 * rs);
        }
      }
    }
  } else if (SPLIT && (tid == 32 * (kSW + 4) || tid == 32 * (kSW + 6))) {
    // =========================== MMA issuers, 16-warp form ====================
    // One thread per query tile, products in program order (S of step j, then P V~ of step j - 1).
    // The two tiles share one score buffer: its uses are numbered in the order tile 0, tile 1,
    // tile 0, ... (tile 0 alone where the item has no second tile), and use G is issued once the
    // softmax warps have loaded use G - 1.  Even and odd uses are released on two barriers: the
    // barrier of use G - 1 cannot complete again before use G + 1 has been issued, and a thread
    // waits for uses that are at most two apart, so a parity wait is never two phases off.
    const int t = (tid == 32 * (kSW + 6)) ? 1 : 0;
    const uint32_t idesc_qk = make_idesc(128, kBf16, false);
    const uint32_t idesc_pv = make_idesc(64, kBf16, true);
    const uint64_t dq = make_desc(sQ + t * 16384);
    const uint32_t d_s = tmem + kColS1, d_p0 = tmem + kColP2 + 128 * t, d_o = tmem + kColO + 64 * t;
    uint32_t g = 0, cp = 0, segq = 0;
    uint32_t g_seg = 0;              // score-buffer uses before this segment
    for (long long pos = step_lo; pos < step_hi;) {
      const int item = (int)(pos / a.n_tiles);
      const int tile_lo = (int)(pos - (long long)item * a.n_tiles);
      const int nt = (int)min((long long)(a.n_tiles - tile_lo), step_hi - pos);
      pos += nt;
      const int pair = item % a.n_pairs;
      const bool active = 2 * pair + t < a.q_tiles;
      const uint32_t per_step = (2 * pair + 1 < a.q_tiles) ? 2u : 1u;     // tiles that use the score buffer
      auto issue_pv = [&](uint32_t gv, bool first_of_segment) {
        mbar_wait(b_vfull + 8 * (gv % kNV), (gv / kNV) & 1, wc);
        if (active) {
          mbar_wait(b_pfull + 8 * t, cp & 1, wc);               // P_t of that step written
          tc_fence_after();
          const uint64_t dv = make_desc(sV + (gv % kNV) * 16384);
          const uint32_t d_p = d_p0 + 64 * (cp & 1);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)   // 16 keys per step: 2 swizzle atoms = 2048 B of V~, 8 columns of P
            mma_ts(d_o, d_p + 8 * ks, dv + (uint64_t)((ks * 2048) >> 4), idesc_pv,
                   (!first_of_segment || ks > 0) ? 1u : 0u);
          tc_commit(b_pvdone2 + 16 * t + 8 * (cp & 1));
          ++cp;
        }
        tc_commit(b_vfree + 8 * (gv % kNV));
      };
      for (int jj = 0; jj < nt; ++jj, ++g) {
        mbar_wait(b_kfull + 8 * (g % kNK), (g / kNK) & 1, wc);
        if (active) {
          const uint32_t use = g_seg + (uint32_t)jj * per_step + (uint32_t)t;
          if (use > 0) mbar_wait(b_sfree + 8 * ((use - 1) & 1), ((use - 1) >> 1) & 1, wc);   // use - 1 is in registers
          if (jj == 0) mbar_wait(b_qfull + 8 * t, segq & 1, wc);
          tc_fence_after();
          const uint64_t dk = make_desc(sK + (g % kNK) * 16384);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)   // 16 channels per step: 32 B inside the swizzle span
            mma_ss(d_s, dq + (uint64_t)(ks * 2), dk + (uint64_t)(ks * 2), idesc_qk, ks > 0 ? 1u : 0u);
          tc_commit(b_sfull + 8 * t);
        } else {
          // An item without a second tile: this thread follows the other tile's uses of the score
          // buffer one by one.  A parity wait is only sound while the waiter is at most one
          // completion ahead of the barrier, so no use may be skipped.
          const uint32_t use = g_seg + (uint32_t)jj;
          if (use > 0) mbar_wait(b_sfree + 8 * ((use - 1) & 1), ((use - 1) >> 1) & 1, wc);
        }
        tc_commit(b_kfree + 8 * (g % kNK));
        if (jj > 0) issue_pv(g - 1, jj == 1);
      }
      issue_pv(g - 1, nt == 1);           // the last PV of the segment
      g_seg += (uint32_t)nt * per_step;
      if (active) ++segq;
    }
    tc_fence_before();
  } else if (!SPLIT && (tid == 32 * (kSW + 4) || tid == 32 * (kSW + 6))) {
    // =========================== MMA issuers ==================================
    // One thread per query tile.  Both release the K~/V~ stages (two arrivals each), also for an
    // item that has no second tile: then the second thread only follows the rings.
    const int t = (tid == 32 * (kSW + 6)) ? 1 : 0;
    const uint32_t idesc_qk = make_idesc(128, kBf16, false);
    const uint32_t idesc_pv = make_idesc(64, kBf16, true);
    const uint64_t dq = make_desc(sQ + t * 16384);
    const uint32_t d_s = tmem + kColS + 128 * t, d_p = tmem + kColP + 64 * t, d_o = tmem + kColO + 64 * t;
    uint32_t g = 0, cnt = 0, segq = 0;
    for (long long pos = step_lo; pos < step_hi;) {
      const int item = (int)(pos / a.n_tiles);
      const int tile_lo = (int)(pos - (long long)item * a.n_tiles);
      const int nt = (int)min((long long)(a.n_tiles - tile_lo), step_hi - pos);
      pos += nt;
      const int pair = item % a.n_pairs;
      const bool active = 2 * pair + t < a.q_tiles;
      auto issue_pv = [&](uint32_t gv, bool first_of_segment) {
        mbar_wait(b_vfull + 8 * (gv % kNV), (gv / kNV) & 1, wc);
        if (active) {
          mbar_wait(b_pfull + 8 * t, (cnt - 1) & 1, wc);        // P_t of that step written
          tc_fence_after();
          const uint64_t dv = make_desc(sV + (gv % kNV) * 16384);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)   // 16 keys per step: 2 swizzle atoms = 2048 B of V~, 8 columns of P
            mma_ts(d_o, d_p + 8 * ks, dv + (uint64_t)((ks * 2048) >> 4), idesc_pv,
                   (!first_of_segment || ks > 0) ? 1u : 0u);
          tc_commit(b_pvdone + 8 * t);
        }
        tc_commit(b_vfree + 8 * (gv % kNV));
      };
      for (int jj = 0; jj < nt; ++jj, ++g) {
        mbar_wait(b_kfull + 8 * (g % kNK), (g / kNK) & 1, wc);
        if (active) {
          if (jj == 0) mbar_wait(b_qfull + 8 * t, segq & 1, wc);
          else mbar_wait(b_sfree + 8 * t, (cnt - 1) & 1, wc);   // S_t of the previous step has been read
          tc_fence_after();
          const uint64_t dk = make_desc(sK + (g % kNK) * 16384);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)   // 16 channels per step: 32 B inside the swizzle span
            mma_ss(d_s, dq + (uint64_t)(ks * 2), dk + (uint64_t)(ks * 2), idesc_qk, ks > 0 ? 1u : 0u);
          tc_commit(b_sfull + 8 * t);
        }
        tc_commit(b_kfree + 8 * (g % kNK));
        if (jj > 0) issue_pv(g - 1, jj == 1);
        if (active) ++cnt;
      }
      issue_pv(g - 1, nt == 1);           // the last PV of the segment
      if (active) ++segq;
    }
    // all MMAs must be done before the CTA may free tensor memory: the softmax warps have waited
    // for every PV (pvdone) before their epilogues, and every QK (sfull) before that.
    tc_fence_before();
  } else if (tid == 32 * (kSW + 5)) {
    // =========================== TMA loader ===================================
    uint32_t g = 0;
    for (long long pos = step_lo; pos < step_hi;) {
      const int item = (int)(pos / a.n_tiles);
      const int tile_lo = (int)(pos - (long long)item * a.n_tiles);
      const int nt = (int)min((long long)(a.n_tiles - tile_lo), step_hi - pos);
      pos += nt;
      const int h = item / a.n_pairs;
      const size_t head_slot = (size_t)h * a.cap;
      for (int jj = 0; jj < nt; ++jj, ++g) {
        const int tile = tile_lo + jj;
        const uint32_t rs = g % C::kNR, ru = g / C::kNR;
        mbar_wait<256>(b_rfree + 8 * rs, (ru & 1) ^ 1, wc);
        const uint32_t dst = sRaw + rs * C::kRawStage, bar = b_rfull + 8 * rs;
        const uint32_t kp_bytes = ONCE ? 512u : (uint32_t)C::kRawKP;    // 128 group references instead of 2 x 64 parameters
        mbar_expect_tx(bar, C::kRawStage - C::kRawKP + kp_bytes);
        const size_t slot0 = head_slot + (size_t)tile * 128;
        if (BITS == 4) {
          tma_load_1d(dst, a.k + slot0 * 32, C::kRawK, bar);
          tma_load_1d(dst + C::kRawK, a.v + slot0 * 32, C::kRawV, bar);
          if (ONCE) tma_load_1d(dst + C::kRawK + C::kRawV, a.kslot + (size_t)tile * 128, kp_bytes, bar);
          else tma_load_1d(dst + C::kRawK + C::kRawV, a.kpar + ((size_t)h * (a.cap >> 6) + 2 * tile) * 64, C::kRawKP, bar);
          tma_load_1d(dst + C::kRawK + C::kRawV + C::kRawKP, a.vpar + slot0, C::kRawVP, bar);
        } else if (BITS == 8) {
          tma_load_1d(dst, a.k + slot0 * 64, C::kRawK, bar);
          tma_load_1d(dst + C::kRawK, a.v + slot0 * 64, C::kRawV, bar);
          tma_load_1d(dst + C::kRawK + C::kRawV, a.kslot + (size_t)tile * 128, kp_bytes, bar);
          tma_load_1d(dst + C::kRawK + C::kRawV + C::kRawKP, a.vpar + slot0, C::kRawVP, bar);
        } else {
          tma_load_1d(dst, a.k + slot0 * 128, C::kRawK, bar);
          tma_load_1d(dst + C::kRawK, a.v + slot0 * 128, C::kRawV, bar);
        }
      }
    }
    // Drain: every copy this thread started has landed once the last use of each stage completed
    // (bounded, and not cut short by the abort flag, so that nothing is in flight at exit).
    const uint32_t issued = g;
    for (uint32_t i = 0; i < (uint32_t)C::kNR && i < issued; ++i) {
      const uint32_t gi = issued - 1 - i;
      const uint32_t rs = gi % C::kNR, ru = gi / C::kNR;
      for (uint32_t it = 0; it < kSpinLimit; ++it)
        if (mbar_try(b_rfull + 8 * rs, ru & 1)) break;
    }
  }
  __syncthreads();
  if (warp == kSW + 5) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------
// Merge of the partial results of the items that were cut between CTAs:
// out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.  Thread = (item, query
// tile, row, 8-channel chunk); items that one CTA covered alone were written by it.
// ---------------------------------------------------------------------------
// IDX = uint32_t when total * grid fits 32 bits (the divisions are then cheap), else uint64_t.
template <typename IDX>
__global__ void __launch_bounds__(256)
attn_combine_kernel(const float* __restrict__ part_o, const float2* __restrict__ part_ml, int grid_i, long long total_ll,
                    int n_tiles, int n_pairs, int q_tiles, int n, __nv_bfloat16* __restrict__ out, int64_t ts,
                    int64_t hs) {
  const IDX grid = (IDX)grid_i, total = (IDX)total_ll;
  const long long gidx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int ch = (int)(gidx & 7);
  const int r = (int)((gidx >> 3) & 127);
  const int t = (int)((gidx >> 10) & 1);
  const IDX item = (IDX)(gidx >> 11);
  if ((long long)item * n_tiles >= total_ll) return;
  const int h = (int)(item / (IDX)n_pairs), pair = (int)(item - (IDX)h * (IDX)n_pairs);
  const int qt = 2 * pair + t;
  const int row = qt * 128 + r;
  if (qt >= q_tiles || row >= n) return;
  const IDX lo = item * (IDX)n_tiles, hi = lo + (IDX)n_tiles;
  // CTA that holds step x: the largest b with piece_start(b) <= x
  const int b_first = (int)(((lo + 1) * grid - 1) / total);
  const int b_last = (int)((hi * grid - 1) / total);
  if (b_first == b_last) return;                 // one CTA covered the whole item and wrote the result
  // a piece's first segment (slot 0) is this item iff the piece starts inside it: only the first
  // piece of the item can start before it
  const bool first_is_second_slot = (total * (IDX)b_first) / grid < lo;
  // The partials are fetched four at a time, all loads before the first use (an item is cut into
  // two or three pieces unless the cache is very long); the running maximum and the weights are
  // those of the online softmax, in the fixed order of the pieces.
  float m = -INFINITY, l = 0.f;
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  for (int b0 = b_first; b0 <= b_last; b0 += 4) {
    float2 ml[4];
    float4 x[4], y[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int b = b0 + j;
      ml[j] = make_float2(-INFINITY, 0.f);
      x[j] = y[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (b <= b_last) {
        const size_t slot = (size_t)2 * b + ((b == b_first && first_is_second_slot) ? 1 : 0);
        const size_t prow = (slot * 2 + t) * 128 + r;
        ml[j] = part_ml[prow];
        const float4* po = reinterpret_cast<const float4*>(part_o + prow * 64 + 8 * ch);
        x[j] = po[0];
        y[j] = po[1];
      }
    }
    const float mc = fmaxf(fmaxf(m, fmaxf(ml[0].x, ml[1].x)), fmaxf(ml[2].x, ml[3].x));
    const float sc = exp2f(m - mc);                // 0 for the first group (m = -inf)
    m = mc;
    l *= sc;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] *= sc;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float wgt = exp2f(ml[j].x - m);        // 0 for an absent piece
      l += wgt * ml[j].y;
      acc[0] += wgt * x[j].x; acc[1] += wgt * x[j].y; acc[2] += wgt * x[j].z; acc[3] += wgt * x[j].w;
      acc[4] += wgt * y[j].x; acc[5] += wgt * y[j].y; acc[6] += wgt * y[j].z; acc[7] += wgt * y[j].w;
    }
  }
  const float inv = 1.f / l;
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = pack_bf2(acc[2 * i] * inv, acc[2 * i + 1] * inv);
  *reinterpret_cast<uint4*>(out + (int64_t)h * hs + (int64_t)row * ts + 8 * ch) = make_uint4(o[0], o[1], o[2], o[3]);
}

size_t attn_tc_scratch_bytes(const xkv_params*) { return (size_t)2 * kMaxGrid * kSlotBytes + 512; }

// `part` holds the partial slots: accumulators float [slots][2][128][64], then (max, sum) float2
// [slots][2][128], slots = part_bytes / kSlotBytes.  The grid is the SM count, capped by the slots
// available (two per CTA) and by the number of steps.
struct TailArgs { const void* k; const void* v; int64_t ts, hs; };

// Per device, on first use with that device current: the SM count, and the opt-in to more than
// 48 KB of dynamic shared memory for the attention kernels (a per-device function attribute).
static std::mutex g_setup_mutex;
static int g_sm_count[kMaxDevices] = {0};       // 0: not set up yet

// The 16-warp form moves registers between its warps with setmaxnreg; the pool they move in is
// what the CTA was launched with.  If a compiler ever gave the kernel fewer registers at launch
// than the reallocation needs, setmaxnreg.inc would wait for ever: refuse to run instead.
template <typename K>
static cudaError_t check_register_pool(K kernel, bool once, bool tail) {
  cudaFuncAttributes fa;
  const cudaError_t e = cudaFuncGetAttributes(&fa, kernel);
  if (e != cudaSuccess) return e;
  const int warps_per_scheduler = kThreadsSplit / 32 / 4;
  return (fa.numRegs * warps_per_scheduler >= 4 * kSplitRegsSoftmax + split_regs_producers(once, tail) + split_regs_misc(once, tail)) ? cudaSuccess
                                                                                    : cudaErrorLaunchOutOfResources;
}

static cudaError_t attn_device_setup(int* sm_count) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_sm_count[dev] == 0) {
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<4, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<4, true>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<16, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<16, true>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<4, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<4, true>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<4, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<4>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<4, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<4>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<8, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<8>());
    if (e != cudaSuccess) return e;
    e = check_register_pool(attn_tc_kernel<4, false, false, true>, false, false);
    if (e != cudaSuccess) return e;
    e = check_register_pool(attn_tc_kernel<16, false, false, true>, false, false);
    if (e != cudaSuccess) return e;
    e = check_register_pool(attn_tc_kernel<4, true, false, true>, false, true);
    if (e != cudaSuccess) return e;
    g_sm_count[dev] = sms;
  }
  *sm_count = g_sm_count[dev];
  return cudaSuccess;
}

static cudaError_t launch_attn_tc_on(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                                     float scale, float* part, size_t part_bytes, cudaStream_t st,
                                     const TailArgs* tail = nullptr, int prefix = 0) {
  int sm_count = 0;
  {
    const cudaError_t e = attn_device_setup(&sm_count);
    if (e != cudaSuccess) return e;
  }
  Args a;
  a.q = reinterpret_cast<const __nv_bfloat16*>(q);
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.n = n; a.ts = ts; a.hs = hs;
  const BufSet& b = c->buf[c->cur];
  a.k = b.k; a.kpar = b.kpar; a.v = b.v; a.vpar = b.vpar;
  a.cap = c->cap; a.t_first = c->T_first;
  a.t_phys = c->rest_base + (c->T - c->T_first);
  if (c->T == c->T_first) a.t_phys = c->T_first;          // only the first frame: no pad tile beyond it
  if (prefix > 0 && prefix < c->T) {
    // a prefix of the cache in logical order: inside the first frame it ends the first segment,
    // after it the rest segment
    if (prefix <= c->T_first) { a.t_first = prefix; a.t_phys = prefix; }
    else a.t_phys = c->rest_base + (prefix - c->T_first);
  }
  a.scale_log2 = scale * 1.4426950408889634f;
  a.n_tiles = (a.t_phys + 127) / 128;
  a.q_tiles = (n + kQRows - 1) / kQRows;
  a.n_pairs = (a.q_tiles + 1) / 2;
  const int H = c->p.n_heads;
  a.total = (long long)H * a.n_pairs * a.n_tiles;
  const size_t slots = part_bytes / kSlotBytes;
  long long grid = sm_count;
  if (grid > (long long)(slots / 2)) grid = (long long)(slots / 2);
  if (c->attn_max_blocks > 0 && grid > c->attn_max_blocks) grid = c->attn_max_blocks;
  if (grid > a.total) grid = a.total;
  if (grid < 1) return cudaErrorMemoryAllocation;
  a.part_o = part;
  a.part_ml = reinterpret_cast<float2*>(part + slots * kSlotFloats);
  a.status = c->status;
  a.kslot = b.kslot; a.ktab16 = c->ktab16; a.n_heads = H;
  a.k_tail = a.v_tail = nullptr;
  a.tail_ts = a.tail_hs = 0;
  a.tail_lo = a.t_phys;
  if (tail && c->p.kv_bits == 8) return cudaErrorNotSupported;      // (the unquantised tail is built for 4-bit caches)
  if (tail && c->p.kv_bits == 4) {      // a 16-bit cache holds the frame exactly as it arrived
    a.k_tail = reinterpret_cast<const __nv_bfloat16*>(tail->k);
    a.v_tail = reinterpret_cast<const __nv_bfloat16*>(tail->v);
    a.tail_ts = tail->ts;
    a.tail_hs = tail->hs;
    a.tail_lo = a.t_phys - n;           // the newest frame holds the last n slots
  }
  {
    LaunchScope ls(c, XKV_PROF_ATTN, st);
    const bool once = c->p.key_mode == XKV_KEYS_ONCE;
    // The 16-warp softmax where the producers have registers to spare for it; with per-token
    // constants (keys quantised once, 8-bit codes) the producers need theirs and the 8-warp
    // softmax measured faster.
    const int T = kThreadsSplit;
    if (c->p.kv_bits == 16) attn_tc_kernel<16, false, false, true><<<(int)grid, T, smem_bytes<16, true>(), st>>>(a);
    else if (c->p.kv_bits == 8) attn_tc_kernel<8, false, true><<<(int)grid, kThreads, smem_bytes<8>(), st>>>(a);
    else if (a.k_tail && once) attn_tc_kernel<4, true, true><<<(int)grid, kThreads, smem_bytes<4>(), st>>>(a);
    else if (a.k_tail) attn_tc_kernel<4, true, false, true><<<(int)grid, T, smem_bytes<4, true>(), st>>>(a);
    else if (once) attn_tc_kernel<4, false, true><<<(int)grid, kThreads, smem_bytes<4>(), st>>>(a);
    else attn_tc_kernel<4, false, false, true><<<(int)grid, T, smem_bytes<4, true>(), st>>>(a);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  {
    LaunchScope ls(c, XKV_PROF_COMBINE, st);
    const long long threads = (long long)H * a.n_pairs * 2048;
    const int blocks = (int)((threads + 255) / 256);
    if ((a.total + 1) * grid < (1ll << 31))
      attn_combine_kernel<uint32_t><<<blocks, 256, 0, st>>>(a.part_o, a.part_ml, (int)grid, a.total, a.n_tiles,
                                                            a.n_pairs, a.q_tiles, n, a.out, ts, hs);
    else
      attn_combine_kernel<uint64_t><<<blocks, 256, 0, st>>>(a.part_o, a.part_ml, (int)grid, a.total, a.n_tiles,
                                                            a.n_pairs, a.q_tiles, n, a.out, ts, hs);
  }
  return cudaGetLastError();
}

cudaError_t launch_attn_tc(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs, float scale,
                           cudaStream_t st, int prefix) {
  return launch_attn_tc_on(c, q, out, n, ts, hs, scale, c->attn_part, c->attn_part_bytes, st, nullptr, prefix);
}

cudaError_t launch_attn_tc_tail(xkv_cache* c, const void* q, const void* k_t, const void* v_t, void* out, int n,
                                int64_t ts, int64_t hs, float scale, cudaStream_t st) {
  const TailArgs tail{k_t, v_t, ts, hs};
  return launch_attn_tc_on(c, q, out, n, ts, hs, scale, c->attn_part, c->attn_part_bytes, st, &tail);
}

// ---------------------------------------------------------------------------
// attn_packed_causal_static: the same attention with its partial slots in a
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
      e = cudaGetSymbolAddress((void**)&p, g_static_partials);
      if (e != cudaSuccess) return e;
      g_static_addr[dev] = p;
    }
    addr = g_static_addr[dev];
  }
  return launch_attn_tc_on(c, q, out, n, ts, hs, scale, reinterpret_cast<float*>(addr),
                           (size_t)XKV_STATIC_SCRATCH_BYTES, st);
}

// ---------------------------------------------------------------------------
// Test hook: the bounded wait of the attention kernel on a barrier that nothing completes.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(32) timeout_probe_kernel(int* status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const WaitCtx wc{status, &abort_flag};
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, wc);     // phase 0 never completes: runs into the limit
  __syncthreads();
  mbar_wait(smem_u32(&bar), 0, wc);                           // the flag is up: every later wait returns at once
}

cudaError_t launch_timeout_probe(xkv_cache* c, cudaStream_t st) {
  timeout_probe_kernel<<<1, 32, 0, st>>>(c->status);
  c->launches++;
  return cudaGetLastError();
}

}  // namespace xkv
