// Bucket staging shared by the quantizer, the histogram and the fused encoder: one CTA holds one
// bucket in registers (V4 quads of four coordinates per thread, quad q = j * blockDim.x + tid, so
// that a warp reads 512 contiguous bytes per load), reduces its norm, and then visits its quads.
#pragma once

#include "qgx_common.cuh"

namespace qgx {

// threads per CTA for a bucket of `bucket` coordinates held V4 quads per thread
inline int bucket_threads(int bucket, int v4) {
  const int quads = (bucket + kQuad - 1) / kQuad;
  int t = (quads + v4 - 1) / v4;
  t = ((t + kWarp - 1) / kWarp) * kWarp;
  return t < kWarp ? kWarp : t;
}
// quads per thread chosen so that CTAs have 128..1024 threads
inline int bucket_v4(int bucket) {
  if (bucket <= 512) return 1;
  if (bucket <= 2048) return 2;
  if (bucket <= 8192) return 4;
  return 8;
}

// Source of a dual vector's coordinates: v alone, or a + u (V_k = A(x) + U_k of Eq. "oracle",
// one fp32 addition), or a * u (relative noise, Assumption 3: one fp32 multiplication), or a alone when u is null.
struct DualSource {
  const float* v;        // [K][d] plain vectors, or the noise U; may be null when a is given
  const float* a;        // [d] operator value A(x) shared by all workers; null for plain vectors
  size_t ld;             // distance between workers' rows of v in floats; 0 means d
  int mul;               // with both arrays: 0 the sum a + v, 1 the product a * v (relative noise: v holds scales)
};

__device__ __forceinline__ float dual_combine(float a, float v, int mul) { return mul ? __fmul_rn(a, v) : __fadd_rn(a, v); }
__device__ __forceinline__ float4 dual_combine(float4 a, float4 v, int mul) {
  return mul ? make_float4(__fmul_rn(a.x, v.x), __fmul_rn(a.y, v.y), __fmul_rn(a.z, v.z), __fmul_rn(a.w, v.w))
             : make_float4(__fadd_rn(a.x, v.x), __fadd_rn(a.y, v.y), __fadd_rn(a.z, v.z), __fadd_rn(a.w, v.w));
}

__device__ __forceinline__ float dual_value(const DualSource& s, size_t k, size_t d, size_t i) {
  const size_t ld = s.ld ? s.ld : d;
  if (s.a == nullptr) return s.v[k * ld + i];
  return s.v ? dual_combine(s.a[i], s.v[k * ld + i], s.mul) : s.a[i];
}

template <int V4>
struct BucketRegs {
  float4 x[V4];
};

// Loads bucket [lo, lo + len) of worker k.  vec_ok: every base pointer is 16-byte aligned and d is
// a multiple of 4, so full quads can be fetched as one 128-bit load.
template <int V4>
__device__ __forceinline__ void load_bucket(BucketRegs<V4>& r, const DualSource& s, size_t k, size_t d,
                                            size_t lo, int len, bool vec_ok) {
  const size_t ld = s.ld ? s.ld : d;
#pragma unroll
  for (int j = 0; j < V4; ++j) {
    const int e = (j * (int)blockDim.x + (int)threadIdx.x) * kQuad;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e + kQuad <= len && vec_ok) {
      if (s.a == nullptr) {
        x = __ldcs(reinterpret_cast<const float4*>(s.v + k * ld + lo + e));
      } else {
        const float4 a = __ldg(reinterpret_cast<const float4*>(s.a + lo + e));
        if (s.v) {
          const float4 u = __ldcs(reinterpret_cast<const float4*>(s.v + k * ld + lo + e));
          x = dual_combine(a, u, s.mul);
        } else {
          x = a;
        }
      }
    } else {
      if (e + 0 < len) x.x = dual_value(s, k, d, lo + e + 0);
      if (e + 1 < len) x.y = dual_value(s, k, d, lo + e + 1);
      if (e + 2 < len) x.z = dual_value(s, k, d, lo + e + 2);
      if (e + 3 < len) x.w = dual_value(s, k, d, lo + e + 3);
    }
    r.x[j] = x;
  }
}

// Norm of the bucket held by the CTA.  L2: fp64 sum of squares (per-thread, then warp shuffles,
// then across warps through shared memory), one square root, one rounding to fp32.
// L-infinity: largest magnitude (NaN is reported as NaN).  red: >= 34 doubles of shared memory.
template <int V4>
__device__ __forceinline__ float bucket_norm(const BucketRegs<V4>& r, int norm_type, double* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  double acc = 0.0;
  if (norm_type == QGX_NORM_L2) {
#pragma unroll
    for (int j = 0; j < V4; ++j) {
      const double a = r.x[j].x, b = r.x[j].y, c = r.x[j].z, e = r.x[j].w;
      acc = fma(a, a, acc); acc = fma(b, b, acc); acc = fma(c, c, acc); acc = fma(e, e, acc);
    }
    acc = warp_sum(acc);
  } else {
    float m = 0.0f;
    bool bad = false;
#pragma unroll
    for (int j = 0; j < V4; ++j) {
      const float4 x = r.x[j];
      bad = bad || (x.x != x.x) || (x.y != x.y) || (x.z != x.z) || (x.w != x.w);
      m = fmaxf(m, fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w))));
    }
    m = warp_max(m);
    bad = __any_sync(0xffffffffu, bad);
    acc = bad ? (double)__int_as_float(0x7fc00000) : (double)m;
  }
  __syncthreads();                       // red may still be read by the previous bucket
  if (lane == 0) red[warp] = acc;
  __syncthreads();
  if (warp == 0) {
    double t = lane < nwarps ? red[lane] : 0.0;
    if (norm_type == QGX_NORM_L2) {
      t = warp_sum(t);
      if (lane == 0) red[32] = (double)(float)sqrt(t);
    } else {
      // max over warps; a NaN partial must survive
      bool bad = __any_sync(0xffffffffu, t != t);
      float m = warp_max((float)t);
      if (lane == 0) red[32] = bad ? (double)__int_as_float(0x7fc00000) : (double)m;
    }
  }
  __syncthreads();
  return (float)red[32];
}

}  // namespace qgx
