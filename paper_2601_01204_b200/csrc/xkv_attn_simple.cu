// Simple CUDA-core attention over the packed cache (Eq. 1 with Eq. 10).
// One thread per query row, fp32 throughout, tiles of 32 key slots dequantised
// into shared memory.  Kept as an independent cross-check of the tensor-core
// kernel (impl = 1); never the default.
#include "xkv_internal.cuh"

namespace xkv {

constexpr int kSimpleTile = 32;

__device__ __forceinline__ int nib_shift_s(int j) { return ((j >> 1) << 2) + ((j & 1) << 4); }

// ktab: quantise-once mode, the key parameter table [slot][H][64] that buf.kslot refers to
// (null otherwise: the parameters of a 64-slot run are in buf.kpar).
template <int BITS>
__global__ void __launch_bounds__(128)
attn_simple_kernel(const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out, int n, int64_t ts,
                   int64_t hs, BufSet buf, int cap, int t_first, int rest_base, int t_phys,
                   float scale_log2, const float2* __restrict__ ktab, int H) {
  __shared__ __align__(16) float s_k[kSimpleTile][64];
  __shared__ __align__(16) float s_v[kSimpleTile][64];
  const int tid = threadIdx.x;
  const int h = blockIdx.y;
  const int row = blockIdx.x * 128 + tid;
  const bool valid = row < n;
  float qf[64];
  {
    const __nv_bfloat16* qp = q + (int64_t)h * hs + (int64_t)(valid ? row : 0) * ts;
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {
      const uint4 u = *reinterpret_cast<const uint4*>(qp + 8 * c8);
      const uint32_t r[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        qf[8 * c8 + 2 * i] = __uint_as_float(r[i] << 16) * scale_log2;
        qf[8 * c8 + 2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u) * scale_log2;
      }
    }
  }
  float acc[64];
#pragma unroll
  for (int c = 0; c < 64; ++c) acc[c] = 0.f;
  float m = -INFINITY, l = 0.f;

  for (int t0 = 0; t0 < t_phys; t0 += kSimpleTile) {
    // cooperative dequantisation of the tile
    for (int item = tid; item < kSimpleTile * 8; item += 128) {
      const int key = item >> 3, w = item & 7;
      const int p = t0 + key;
      float kx[8], vx[8];
      if (p < t_phys) {
        const size_t slot = (size_t)h * cap + p;
        if (BITS == 4) {
          const uint32_t kw = *reinterpret_cast<const uint32_t*>(buf.k + slot * 32 + 4 * w);
          const uint32_t vw = *reinterpret_cast<const uint32_t*>(buf.v + slot * 32 + 4 * w);
          const float2* kp = ktab ? ktab + ((size_t)buf.kslot[p] * H + h) * 64 + 8 * w
                                  : buf.kpar + ((size_t)h * (cap >> 6) + (p >> 6)) * 64 + 8 * w;
          const float2 vp = buf.vpar[slot];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float2 sz = kp[j];
            kx[j] = sz.x * ((float)((kw >> nib_shift_s(j)) & 0xFu) - sz.y);
            vx[j] = vp.x * ((float)((vw >> nib_shift_s(j)) & 0xFu) - vp.y);
          }
        } else if (BITS == 8) {
          // 8-bit codes (keys quantised once): bytes of channels (0, 2, 1, 3) per word
          const uint2 kw = *reinterpret_cast<const uint2*>(buf.k + slot * 64 + 8 * w);
          const uint2 vw = *reinterpret_cast<const uint2*>(buf.v + slot * 64 + 8 * w);
          const float2* kp = ktab + ((size_t)buf.kslot[p] * H + h) * 64 + 8 * w;
          const float2 vp = buf.vpar[slot];
          const uint32_t kws[2] = {kw.x, kw.y}, vws[2] = {vw.x, vw.y};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int sh = ((j & 3) == 0) ? 0 : ((j & 3) == 1) ? 16 : ((j & 3) == 2) ? 8 : 24;
            const float2 sz = kp[j];
            kx[j] = sz.x * ((float)((kws[j >> 2] >> sh) & 0xFFu) - sz.y);
            vx[j] = vp.x * ((float)((vws[j >> 2] >> sh) & 0xFFu) - vp.y);
          }
        } else {
          const uint4 ku = *reinterpret_cast<const uint4*>(buf.k + slot * 128 + 16 * w);
          const uint4 vu = *reinterpret_cast<const uint4*>(buf.v + slot * 128 + 16 * w);
          const uint32_t kr[4] = {ku.x, ku.y, ku.z, ku.w};
          const uint32_t vr[4] = {vu.x, vu.y, vu.z, vu.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            kx[2 * i] = __uint_as_float(kr[i] << 16);
            kx[2 * i + 1] = __uint_as_float(kr[i] & 0xFFFF0000u);
            vx[2 * i] = __uint_as_float(vr[i] << 16);
            vx[2 * i + 1] = __uint_as_float(vr[i] & 0xFFFF0000u);
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) { kx[j] = 0.f; vx[j] = 0.f; }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) { s_k[key][8 * w + j] = kx[j]; s_v[key][8 * w + j] = vx[j]; }
    }
    __syncthreads();

    float s[kSimpleTile];
    float tmax = -INFINITY;
#pragma unroll
    for (int key = 0; key < kSimpleTile; ++key) {
      float d0 = 0.f, d1 = 0.f;
#pragma unroll
      for (int c4 = 0; c4 < 16; ++c4) {
        const float4 kv = *reinterpret_cast<const float4*>(&s_k[key][4 * c4]);
        d0 = fmaf(qf[4 * c4], kv.x, d0);
        d1 = fmaf(qf[4 * c4 + 1], kv.y, d1);
        d0 = fmaf(qf[4 * c4 + 2], kv.z, d0);
        d1 = fmaf(qf[4 * c4 + 3], kv.w, d1);
      }
      const int p = t0 + key;
      const bool masked = (p >= t_phys) || (p >= t_first && p < rest_base);
      s[key] = masked ? -INFINITY : (d0 + d1);
      tmax = fmaxf(tmax, s[key]);
    }
    const float m_new = fmaxf(m, tmax);
    if (m_new > -INFINITY) {
      const float corr = exp2f(m - m_new);
      l *= corr;
#pragma unroll
      for (int c = 0; c < 64; ++c) acc[c] *= corr;
#pragma unroll
      for (int key = 0; key < kSimpleTile; ++key) {
        const float pj = exp2f(s[key] - m_new);
        l += pj;
#pragma unroll
        for (int c4 = 0; c4 < 16; ++c4) {
          const float4 vv = *reinterpret_cast<const float4*>(&s_v[key][4 * c4]);
          acc[4 * c4] = fmaf(pj, vv.x, acc[4 * c4]);
          acc[4 * c4 + 1] = fmaf(pj, vv.y, acc[4 * c4 + 1]);
          acc[4 * c4 + 2] = fmaf(pj, vv.z, acc[4 * c4 + 2]);
          acc[4 * c4 + 3] = fmaf(pj, vv.w, acc[4 * c4 + 3]);
        }
      }
      m = m_new;
    }
    __syncthreads();
  }
  if (valid) {
    const float inv_l = 1.f / l;
    __nv_bfloat16* op = out + (int64_t)h * hs + (int64_t)row * ts;
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {
      uint32_t r[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 b = __floats2bfloat162_rn(acc[8 * c8 + 2 * i] * inv_l, acc[8 * c8 + 2 * i + 1] * inv_l);
        r[i] = *reinterpret_cast<const uint32_t*>(&b);
      }
      *reinterpret_cast<uint4*>(op + 8 * c8) = make_uint4(r[0], r[1], r[2], r[3]);
    }
  }
}

cudaError_t launch_attn_simple(xkv_cache* c, const void* q, void* out, int n, int64_t ts, int64_t hs,
                               float scale, cudaStream_t st) {
  const dim3 grid((n + 127) / 128, c->p.n_heads);
  const int t_phys = c->rest_base + (c->T - c->T_first);
  const float scale_log2 = scale * 1.4426950408889634f;
  auto qq = reinterpret_cast<const __nv_bfloat16*>(q);
  auto oo = reinterpret_cast<__nv_bfloat16*>(out);
  LaunchScope ls(c, XKV_PROF_ATTN, st);
  if (c->p.kv_bits == 8)
    attn_simple_kernel<8><<<grid, 128, 0, st>>>(qq, oo, n, ts, hs, c->buf[c->cur], c->cap, c->T_first,
                                                c->rest_base, t_phys, scale_log2, c->ktab32, c->p.n_heads);
  else if (c->p.kv_bits == 16)
    attn_simple_kernel<16><<<grid, 128, 0, st>>>(qq, oo, n, ts, hs, c->buf[c->cur], c->cap, c->T_first,
                                                 c->rest_base, t_phys, scale_log2, nullptr, c->p.n_heads);
  else
    attn_simple_kernel<4><<<grid, 128, 0, st>>>(qq, oo, n, ts, hs, c->buf[c->cur], c->cap, c->T_first,
                                                c->rest_base, t_phys, scale_log2,
                                                c->p.key_mode == XKV_KEYS_ONCE ? c->ktab32 : nullptr, c->p.n_heads);
  return cudaGetLastError();
}

}  // namespace xkv
