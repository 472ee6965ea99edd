// Sufficient statistics of the level refit (Sec. 3.3): the histogram of normalized magnitudes,
// each coordinate weighted by its bucket's squared norm (the weights lambda_j of Eq. QAda), and
// qgx_update_levels, which feeds it to the host-side fit and code builders.
#include "qgx_bucket.cuh"

#include <algorithm>
#include <vector>

namespace qgx {

constexpr int kMaxBins = 4096;

// Bin of one coordinate: floor(fl(fl(|x| / norm) * nbins)), clamped to the last bin -- the definition, in IEEE
// operations.
__device__ __forceinline__ int bin_exact(float x, float norm, float nbf, int nbins) {
  float u = (norm > 0.0f) ? __fdiv_rn(fabsf(x), norm) : 0.0f;
  u = fminf(u, 1.0f);
  return min((int)floorf(__fmul_rn(u, nbf)), nbins - 1);
}

// floor(t) of t = min(|x| * c, nbins), c = fl(nbins / norm), read from the mantissa of t + (2^23 - 1/2) -- one exact
// rounding to the nearest integer of t - 1/2 (which is -1/2, read as bin 0, while t < 1/4) -- and whether it is
// safely the bin of x: t differs from the defining product T by less than 4.0001 * 2^-24 * T < 2^-21.9 * t (four
// roundings), so floor(t) = floor(T) whenever t keeps a distance of 2^-21 * t from the integers.  A t that is not
// finite, or that reaches nbins, is never safe.
struct FastBin { int bin; bool safe; };
__device__ __forceinline__ FastBin fast_bin(float x, float c, float nbf) {
  const float kMagic = 8388607.5f;                                    // 2^23 - 1/2
  const float tt = fminf(__fmul_rn(fabsf(x), c), nbf);
  const float m = __fadd_rn(tt, kMagic);
  FastBin f;
  f.bin = max((int)__float_as_uint(m) - 0x4B000000, 0);
  const float dist = __fsub_rn(tt, __fsub_rn(m, kMagic));             // t - (floor(t) + 1/2)
  f.safe = fabsf(dist) <= __fmaf_rn(tt, -4.76837158203125e-07f, 0.5f);
  return f;
}

// Persistent CTAs: bucket t of the launch (b = t / K, k = t % K, so that CTAs working side by side share the
// operator's bucket in L2) belongs to CTA t mod gridDim.x.  Counts per bin of one bucket in shared memory, folded
// after each bucket into the CTA's own fp64 histogram (count * weight); one fp64 atomic per occupied bin and CTA at
// the end.
//
// A coordinate whose bin fast_bin cannot vouch for (a few in a million for bins of small index) takes the defining
// operations after the thread's other coordinates.
template <int V4>
__global__ void __launch_bounds__(512, 2) k_histogram(DualSource src, size_t d, int bucket, size_t nb, int K, int norm_type,
                                                      int nbins, int weighted, bool vec_ok, double* __restrict__ hist,
                                                      DevStatus* st) {
  extern __shared__ __align__(8) unsigned char s_raw[];
  double* s_hist = reinterpret_cast<double*>(s_raw);                 // [nbins]
  uint32_t* s_cnt = reinterpret_cast<uint32_t*>(s_hist + nbins);      // [nbins + 1]
  __shared__ double s_red[34];
  for (int i = threadIdx.x; i < nbins; i += blockDim.x) { s_hist[i] = 0.0; s_cnt[i] = 0u; }
  const float nbf = (float)nbins;
  const unsigned long long total = (unsigned long long)nb * (unsigned long long)K;
  for (unsigned long long t = blockIdx.x; t < total; t += gridDim.x) {
    const size_t b = (size_t)(t / (unsigned long long)K), k = (size_t)(t % (unsigned long long)K);
    const size_t lo = b * (size_t)bucket;
    const int len = (int)min((size_t)bucket, d - lo);
    BucketRegs<V4> r;
    load_bucket<V4>(r, src, k, d, lo, len, vec_ok);
    const float norm = bucket_norm<V4>(r, norm_type, s_red);   // contains __syncthreads: the fold of the last bucket is done
    const bool finite = (norm - norm) == 0.0f;
    if (!finite) {
      if (threadIdx.x == 0) latch_error(st, QGX_ERR_NONFINITE);
    } else {
      if (len == (int)blockDim.x * V4 * kQuad) {                   // every thread's quads lie inside the bucket
        const float c = (norm > 0.0f) ? __fdiv_rn(nbf, norm) : 0.0f;
        bool redo = false;                                         // one of this thread's coordinates is not safe
#pragma unroll
        for (int j = 0; j < V4; ++j) {
          const float x[kQuad] = {r.x[j].x, r.x[j].y, r.x[j].z, r.x[j].w};
#pragma unroll
          for (int q = 0; q < kQuad; ++q) {
            const FastBin f = fast_bin(x[q], c, nbf);
            redo = redo || !f.safe;
            atomicAdd(&s_cnt[f.safe ? f.bin : nbins], 1u);         // entry nbins collects the unsafe ones and is never read
          }
        }
        if (redo) {                                                // rare: the thread's coordinates are read again
          for (int j = 0; j < V4; ++j) {
            const size_t e = lo + (size_t)(j * (int)blockDim.x + (int)threadIdx.x) * kQuad;
            for (int q = 0; q < kQuad; ++q) {
              const float xq = dual_value(src, k, d, e + q);
              if (!fast_bin(xq, c, nbf).safe) atomicAdd(&s_cnt[bin_exact(xq, norm, nbf, nbins)], 1u);
            }
          }
        }
      } else {                                                     // a short last bucket: the defining operations
#pragma unroll
        for (int j = 0; j < V4; ++j) {
          const int e = (j * (int)blockDim.x + (int)threadIdx.x) * kQuad;
          const float x[kQuad] = {r.x[j].x, r.x[j].y, r.x[j].z, r.x[j].w};
#pragma unroll
          for (int q = 0; q < kQuad; ++q)
            if (e + q < len) atomicAdd(&s_cnt[bin_exact(x[q], norm, nbf, nbins)], 1u);
        }
      }
    }
    __syncthreads();
    if (finite) {
      const double wgt = weighted ? (double)norm * (double)norm : 1.0;
      for (int i = threadIdx.x; i < nbins; i += blockDim.x) {
        const uint32_t n = s_cnt[i];
        if (n) { s_hist[i] += (double)n * wgt; s_cnt[i] = 0u; }
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < nbins; i += blockDim.x) {
    const double h = s_hist[i];
    if (h != 0.0) atomicAdd(&hist[i], h);
  }
}

qgx_status launch_histogram(qgx_ctx* c, DualSource src, int K, size_t d, int bucket, int norm_type, int nbins, int weighted,
                            double* hist) {
  if (!c || !hist || K < 1 || K > 65535 || d < 1 || bucket < kQuad || bucket > QGX_MAX_BUCKET || bucket % kQuad != 0 ||
      nbins < 1 || nbins > kMaxBins || (norm_type != QGX_NORM_L2 && norm_type != QGX_NORM_LINF))
    return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  if (cudaMemsetAsync(hist, 0, sizeof(double) * (size_t)nbins, c->stream) != cudaSuccess) return QGX_ERR_CUDA;
  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  const bool vec_ok = (d % kQuad == 0) && ((reinterpret_cast<uintptr_t>(src.v) & 15u) == 0) &&
                      ((reinterpret_cast<uintptr_t>(src.a) & 15u) == 0);
  const int v4 = bucket_v4(bucket);
  const int threads = bucket_threads(bucket, v4);
  const size_t smem = (sizeof(double) + sizeof(uint32_t)) * (size_t)nbins + 16;
  const unsigned long long total = (unsigned long long)nb * (unsigned long long)K;
  ScopedKernelTimer timer(c, QGX_KERNEL_HISTOGRAM);
#define QGX_LAUNCH_H(V)                                                                                              \
  do {                                                                                                               \
    int per_sm = 1;                                                                                                  \
    if (smem > 40u * 1024u) cudaFuncSetAttribute(k_histogram<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_histogram<V>, threads, smem);                           \
    const unsigned grid = (unsigned)std::min<unsigned long long>(total, (unsigned long long)c->num_sms * (unsigned long long)std::max(per_sm, 1)); \
    k_histogram<V><<<grid, threads, smem, c->stream>>>(src, d, bucket, nb, K, norm_type, nbins, weighted, vec_ok, hist, c->dstatus); \
  } while (0)
  switch (v4) {
    case 1: QGX_LAUNCH_H(1); break;
    case 2: QGX_LAUNCH_H(2); break;
    case 4: QGX_LAUNCH_H(4); break;
    default: QGX_LAUNCH_H(8); break;
  }
#undef QGX_LAUNCH_H
  count_launch(c);
  return cuda_status(cudaGetLastError());
}

// histogram -> host; levels refit; code rebuilt.  Synchronizes the stream.
qgx_status refit_from_source(qgx_ctx* c, DualSource src, int K, size_t d, qgx_quant_cfg* cfg, int refit, double* hist,
                             double* hist_host) {
  if (!cfg || refit == QGX_REFIT_NONE) return QGX_ERR_INVALID_ARG;
  if (cfg->nlev < 2 || cfg->nlev > QGX_MAX_LEVELS) return QGX_ERR_BAD_LEVELS;
  qgx_status rc = launch_histogram(c, src, K, d, cfg->bucket, cfg->norm_type, cfg->nbins, 1, hist);
  if (rc != QGX_OK) return rc;
  std::vector<double> h((size_t)cfg->nbins);
  if (cudaMemcpyAsync(h.data(), hist, sizeof(double) * h.size(), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaStreamSynchronize(c->stream) != cudaSuccess)
    return QGX_ERR_CUDA;
  rc = qgx_fit_levels(h.data(), cfg->nbins, cfg->levels, cfg->nlev, refit == QGX_REFIT_FIRST ? 1 : 0);
  if (rc != QGX_OK) return rc;
  const int sub = cfg->cb.subblock;
  if (cfg->code_type == QGX_CODE_HUFFMAN) {
    double p[QGX_MAX_LEVELS];
    rc = qgx_symbol_pmf(h.data(), cfg->nbins, cfg->levels, cfg->nlev, p);
    if (rc != QGX_OK) return rc;
    rc = qgx_build_codebook_huffman(p, cfg->nlev, sub, &cfg->cb);
  } else if (cfg->code_type == QGX_CODE_ELIAS) {
    rc = qgx_build_codebook_elias(cfg->nlev, sub, &cfg->cb);
  } else {
    rc = qgx_build_codebook_fixed(cfg->nlev, sub, &cfg->cb);
  }
  if (hist_host)
    for (int j = 0; j < cfg->nbins; ++j) hist_host[j] = h[(size_t)j];
  return rc;
}

}  // namespace qgx

using namespace qgx;

extern "C" {

qgx_status qgx_histogram(qgx_ctx* c, const float* v, int K, size_t d, int bucket, int norm_type, int nbins, int weighted,
                         double* hist) {
  if (!v) return QGX_ERR_INVALID_ARG;
  DualSource src{v, nullptr, 0, 0};
  return launch_histogram(c, src, K, d, bucket, norm_type, nbins, weighted, hist);
}

qgx_status qgx_update_levels(qgx_ctx* c, const float* v, int K, size_t d, qgx_quant_cfg* cfg, int refit, double* hist,
                             double* hist_host) {
  if (!v) return QGX_ERR_INVALID_ARG;
  DualSource src{v, nullptr, 0, 0};
  return refit_from_source(c, src, K, d, cfg, refit, hist, hist_host);
}

}  // extern "C"
