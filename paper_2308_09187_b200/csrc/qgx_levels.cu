// Sufficient statistics of the level refit (Sec. 3.3): the histogram of normalized magnitudes,
// each coordinate weighted by its bucket's squared norm (the weights lambda_j of Eq. QAda), and
// qgx_update_levels, which feeds it to the host-side fit and code builders.
#include "qgx_bucket.cuh"

#include <vector>

namespace qgx {

constexpr int kMaxBins = 4096;

// One CTA per (bucket, worker): counts per bin in shared memory, then one fp64 atomic per
// occupied bin adds count * weight to the global histogram.
template <int V4>
__global__ void __launch_bounds__(512) k_histogram(DualSource src, size_t d, int bucket, int norm_type, int nbins, int weighted,
                                                   bool vec_ok, double* __restrict__ hist, DevStatus* st) {
  extern __shared__ uint32_t s_cnt[];
  __shared__ double s_red[34];
  const size_t b = blockIdx.x, k = blockIdx.y;
  const size_t lo = b * (size_t)bucket;
  const int len = (int)min((size_t)bucket, d - lo);
  for (int i = threadIdx.x; i < nbins; i += blockDim.x) s_cnt[i] = 0;

  BucketRegs<V4> r;
  load_bucket<V4>(r, src, k, d, lo, len, vec_ok);
  const float norm = bucket_norm<V4>(r, norm_type, s_red);     // contains __syncthreads
  if (!((norm - norm) == 0.0f)) {
    if (threadIdx.x == 0) latch_error(st, QGX_ERR_NONFINITE);
    return;
  }
  const float nbf = (float)nbins;
#pragma unroll
  for (int j = 0; j < V4; ++j) {
    const int e = (j * (int)blockDim.x + (int)threadIdx.x) * kQuad;
    const float x[kQuad] = {r.x[j].x, r.x[j].y, r.x[j].z, r.x[j].w};
#pragma unroll
    for (int c = 0; c < kQuad; ++c) {
      if (e + c < len) {
        float u = (norm > 0.0f) ? __fdiv_rn(fabsf(x[c]), norm) : 0.0f;
        u = fminf(u, 1.0f);
        const int bin = min((int)floorf(__fmul_rn(u, nbf)), nbins - 1);
        atomicAdd(&s_cnt[bin], 1u);
      }
    }
  }
  __syncthreads();
  const double wgt = weighted ? (double)norm * (double)norm : 1.0;
  for (int i = threadIdx.x; i < nbins; i += blockDim.x) {
    const uint32_t n = s_cnt[i];
    if (n) atomicAdd(&hist[i], (double)n * wgt);
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
  const dim3 grid((unsigned)nb, (unsigned)K);
  const size_t smem = sizeof(uint32_t) * (size_t)nbins;
  ScopedKernelTimer timer(c, QGX_KERNEL_HISTOGRAM);
  switch (v4) {
    case 1: k_histogram<1><<<grid, threads, smem, c->stream>>>(src, d, bucket, norm_type, nbins, weighted, vec_ok, hist, c->dstatus); break;
    case 2: k_histogram<2><<<grid, threads, smem, c->stream>>>(src, d, bucket, norm_type, nbins, weighted, vec_ok, hist, c->dstatus); break;
    case 4: k_histogram<4><<<grid, threads, smem, c->stream>>>(src, d, bucket, norm_type, nbins, weighted, vec_ok, hist, c->dstatus); break;
    default: k_histogram<8><<<grid, threads, smem, c->stream>>>(src, d, bucket, norm_type, nbins, weighted, vec_ok, hist, c->dstatus); break;
  }
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
