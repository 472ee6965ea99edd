// qgx_eg_step: one iteration of Algorithm 1 in its dual-extrapolation instance -- operator
// evaluation (coalesced GEMV with fp64 accumulation), two fused exchanges whose decode epilogues
// apply the half step and the dual step of Eq. (Q-GenX), and the adaptive step size of Theorem 3.
#include "qgx_bucket.cuh"

namespace qgx {

// declared in qgx_exchange.cu / qgx_levels.cu
qgx_status exchange_impl(qgx_ctx* c, DualSource src, int K, size_t d, const qgx_quant_cfg* cfg, uint32_t xid, int slot,
                         float* mean_out, uint64_t* total_bits_out, const ExchangeUpdate* upd, int sym_mode, double* sum_sq,
                         uint64_t coord_base);
qgx_status refit_from_source(qgx_ctx* c, DualSource src, int K, size_t d, qgx_quant_cfg* cfg, int refit, double* hist,
                             double* hist_host);
enum { WS_OPVAL = 15, WS_MEAN = 16, WS_HIST = 17 };

// sum_j m[j] x[j] of one row by one warp: fp64 accumulation, four partial sums per lane, the lanes' sums added by
// shuffles; every lane returns the total
__device__ __forceinline__ double gemv_row(const float* __restrict__ m, size_t ncols, const float* __restrict__ x, int lane, bool vec_ok) {
  double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
  if (vec_ok) {
    // four loads of the row in flight, added in index order
    constexpr int kAhead = 4;
    for (size_t j0 = (size_t)lane * 4; j0 < ncols; j0 += 128 * kAhead) {
      float4 mv[kAhead], xv[kAhead];
#pragma unroll
      for (int u = 0; u < kAhead; ++u) {
        const size_t j = j0 + 128 * (size_t)u;
        if (j < ncols) {
          mv[u] = __ldcs(reinterpret_cast<const float4*>(m + j));
          xv[u] = __ldg(reinterpret_cast<const float4*>(x + j));
        }
      }
#pragma unroll
      for (int u = 0; u < kAhead; ++u) {
        if (j0 + 128 * (size_t)u < ncols) {
          a0 = fma((double)mv[u].x, (double)xv[u].x, a0);
          a1 = fma((double)mv[u].y, (double)xv[u].y, a1);
          a2 = fma((double)mv[u].z, (double)xv[u].z, a2);
          a3 = fma((double)mv[u].w, (double)xv[u].w, a3);
        }
      }
    }
  } else {
    for (size_t j = lane; j < ncols; j += 32) a0 = fma((double)m[j], (double)x[j], a0);
  }
  return warp_sum((a0 + a1) + (a2 + a3));
}

// out[row] = sign * (sum_j mat[row][j] x[j] + bias[row]); one warp per row, fp64 accumulation,
// one rounding to fp32
__global__ void __launch_bounds__(256) k_gemv_rows(const float* __restrict__ mat, size_t nrows, size_t ncols,
                                                   const float* __restrict__ x, const float* __restrict__ bias,
                                                   float* __restrict__ out, bool vec_ok) {
  const int lane = threadIdx.x & 31;
  const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const size_t nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
  for (size_t row = warp; row < nrows; row += nwarps) {
    const double s = gemv_row(mat + row * ncols, ncols, x, lane, vec_ok);
    if (lane == 0) out[row] = (float)(bias ? s + (double)bias[row] : s);
  }
}

// The bilinear operator in one launch, z = (x, y): out = (M y, -M^T x).  Blocks of 32 x 32 threads; the first
// ceil(n / 32) blocks take 32 columns each (out[n + col] = -(sum_i mat[i][col] x[i]): rows strided over the 32 row
// lanes, partial sums combined in row-lane order), the others 32 rows each (one warp per row, as k_gemv_rows).
__global__ void __launch_bounds__(1024) k_bilinear(const float* __restrict__ mat, size_t n, const float* __restrict__ z,
                                                   float* __restrict__ out_all, bool vec_ok) {
  __shared__ double s_part[32][33];
  const int cx = threadIdx.x, ry = threadIdx.y;
  const size_t col_blocks = (n + 31) / 32;
  if (blockIdx.x >= col_blocks) {
    const size_t row = ((size_t)blockIdx.x - col_blocks) * 32 + (size_t)ry;
    if (row < n) {
      const double s = gemv_row(mat + row * n, n, z + n, cx, vec_ok);
      if (cx == 0) out_all[row] = (float)s;
    }
    return;
  }
  const float* x = z;
  float* out = out_all + n;
  const size_t col = (size_t)blockIdx.x * 32 + cx;
  double acc = 0.0;
  if (col < n) {
    // eight loads of the column in flight, added in index order
    constexpr int kAhead = 8;
    for (size_t i0 = ry; i0 < n; i0 += 32 * kAhead) {
      float mv[kAhead], xv[kAhead];
#pragma unroll
      for (int u = 0; u < kAhead; ++u) {
        const size_t i = i0 + 32 * (size_t)u;
        if (i < n) { mv[u] = mat[i * n + col]; xv[u] = x[i]; }
      }
#pragma unroll
      for (int u = 0; u < kAhead; ++u)
        if (i0 + 32 * (size_t)u < n) acc = fma((double)mv[u], (double)xv[u], acc);
    }
  }
  s_part[ry][cx] = acc;
  __syncthreads();
  if (ry == 0 && col < n) {
    double s = 0.0;
    for (int r = 0; r < 32; ++r) s += s_part[r][cx];
    out[col] = (float)(-s);
  }
}

__global__ void __launch_bounds__(256) k_diag(const float* __restrict__ D, const float* __restrict__ x, float* __restrict__ out, size_t d) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (size_t)gridDim.x * blockDim.x)
    out[i] = __fmul_rn(D[i], x[i]);
}

__global__ void __launch_bounds__(256) k_eg_init(float* X, float* Y, float* Xbar, const float* anchor, double* scalars, size_t d, int K) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (size_t)gridDim.x * blockDim.x) {
    X[i] = anchor[i];
    Y[i] = 0.0f;
    Xbar[i] = 0.0f;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) { scalars[0] = 0.0; scalars[1] = (double)K; }
}

// gamma_{t+1} = K / sqrt(1 + sum); X_{t+1} = anchor + gamma_{t+1} Y_{t+1}; Xbar += (X_{t+1/2} - Xbar) / t
__global__ void __launch_bounds__(256) k_eg_finish(float* __restrict__ X, const float* __restrict__ Y, float* __restrict__ Xbar,
                                                   const float* __restrict__ Xhalf, const float* __restrict__ anchor,
                                                   double* scalars, size_t d, int K, int t) {
  const float gamma = (float)((double)K / sqrt(1.0 + scalars[0]));
  const float tf = (float)t;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (size_t)gridDim.x * blockDim.x) {
    X[i] = __fadd_rn(anchor[i], __fmul_rn(gamma, Y[i]));
    const float xb = Xbar[i];
    Xbar[i] = __fadd_rn(xb, __fdiv_rn(__fsub_rn(Xhalf[i], xb), tf));
  }
  // scalars[1] is not read by this kernel, so one thread may replace it
  if (blockIdx.x == 0 && threadIdx.x == 0) scalars[1] = (double)gamma;
}

// X_{t+1/2} = X_t - gamma_t * m (optimistic dual averaging: m is the mean of the previous iteration's quantized vectors)
__global__ void __launch_bounds__(256) k_half_from_mean(const float* __restrict__ X, const float* __restrict__ m,
                                                        const double* __restrict__ scalars, float* __restrict__ Xhalf, size_t d) {
  const float gamma = (float)scalars[1];
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (size_t)gridDim.x * blockDim.x)
    Xhalf[i] = __fsub_rn(X[i], __fmul_rn(gamma, m[i]));
}

static unsigned grid_for(const qgx_ctx* c, size_t n, int threads) {
  return (unsigned)std::max<size_t>(1, std::min<size_t>((n + threads - 1) / threads, (size_t)c->num_sms * 8));
}

qgx_status apply_operator_impl(qgx_ctx* c, const qgx_operator* op, const float* x, float* out) {
  if (!c || !op || !x || !out || !op->mat || op->d < 1) return QGX_ERR_INVALID_ARG;
  const size_t d = op->d;
  ScopedKernelTimer timer(c, QGX_KERNEL_OPERATOR);
  if (op->kind == QGX_OP_DENSE_AFFINE) {
    const bool vec_ok = (d % 4 == 0) && ((reinterpret_cast<uintptr_t>(op->mat) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(x) & 15u) == 0);
    k_gemv_rows<<<grid_for(c, d * 32, 256), 256, 0, c->stream>>>(op->mat, d, d, x, op->bias, out, vec_ok);
    count_launch(c);
  } else if (op->kind == QGX_OP_BILINEAR) {
    if (d % 2) return QGX_ERR_INVALID_ARG;
    const size_t n = d / 2;
    const bool vec_ok = (n % 4 == 0) && ((reinterpret_cast<uintptr_t>(op->mat) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(x + n) & 15u) == 0);
    k_bilinear<<<(unsigned)(2 * ((n + 31) / 32)), dim3(32, 32), 0, c->stream>>>(op->mat, n, x, out, vec_ok);
    count_launch(c);
  } else if (op->kind == QGX_OP_DIAGONAL) {
    k_diag<<<grid_for(c, d, 256), 256, 0, c->stream>>>(op->mat, x, out, d);
    count_launch(c);
  } else {
    return QGX_ERR_INVALID_ARG;
  }
  return cuda_status(cudaGetLastError());
}

}  // namespace qgx

using namespace qgx;

extern "C" {

qgx_status qgx_apply_operator(qgx_ctx* c, const qgx_operator* op, const float* x, float* out) {
  if (c && cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  return apply_operator_impl(c, op, x, out);
}

qgx_status qgx_eg_init(qgx_ctx* c, qgx_eg_state* st) {
  if (!c || !st || !st->X || !st->Y || !st->Xbar || !st->Xhalf || !st->anchor || !st->scalars || st->d < 1 || st->K < 1)
    return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  k_eg_init<<<grid_for(c, st->d, 256), 256, 0, c->stream>>>(st->X, st->Y, st->Xbar, st->anchor, st->scalars, st->d, st->K);
  count_launch(c);
  st->t = 1;
  return cuda_status(cudaGetLastError());
}

// cfg_half == cfg: one level table and code for both exchanges; otherwise each exchange has its own, refitted on
// its own dual vectors
static qgx_status eg_step_impl(qgx_ctx* c, qgx_eg_state* st, const qgx_operator* op, const float* noise_t, const float* noise_half,
                               qgx_quant_cfg* cfg, qgx_quant_cfg* cfg_half, int refit, uint64_t* bits) {
  if (!c || !st || !op || !cfg || !cfg_half || !st->X || !st->Y || !st->Xbar || !st->Xhalf || !st->anchor || !st->scalars || st->t < 1 ||
      op->d != st->d || st->K < 1)
    return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  const size_t d = st->d;
  const int K = st->K;
  float* a = (float*)ws_get(c, WS_OPVAL, sizeof(float) * d);
  float* mean = (float*)ws_get(c, WS_MEAN, sizeof(float) * d);
  if (!a || !mean) return QGX_ERR_CUDA;

  qgx_status rc = apply_operator_impl(c, op, st->X, a);                      // A(X_t)
  if (rc != QGX_OK) return rc;
  const int mul = op->noise_model == QGX_NOISE_RELATIVE ? 1 : 0;
  DualSource src{noise_t, a, 0, mul};                                           // V_{k,t} = A(X_t) + U_{k,t}  (or .* S_{k,t})
  if (refit != QGX_REFIT_NONE) {
    double* hist = (double*)ws_get(c, WS_HIST, sizeof(double) * (size_t)std::max(cfg->nbins, 1));
    if (!hist) return QGX_ERR_CUDA;
    rc = refit_from_source(c, src, K, d, cfg, refit, hist, nullptr);
    if (rc != QGX_OK) return rc;
  }
  const uint32_t xid = 2u * (uint32_t)st->t;
  ExchangeUpdate half{1, st->X, st->Xhalf, st->scalars};                      // X_{t+1/2} = X_t - gamma_t * mean
  rc = exchange_impl(c, src, K, d, cfg, xid, 0, mean, bits, &half, 1, nullptr, 0);
  if (rc != QGX_OK) return rc;
  rc = apply_operator_impl(c, op, st->Xhalf, a);                              // A(X_{t+1/2})
  if (rc != QGX_OK) return rc;
  DualSource src2{noise_half, a, 0, mul};
  if (cfg_half != cfg && refit != QGX_REFIT_NONE) {
    double* hist = (double*)ws_get(c, WS_HIST, sizeof(double) * (size_t)std::max(cfg_half->nbins, 1));
    if (!hist) return QGX_ERR_CUDA;
    rc = refit_from_source(c, src2, K, d, cfg_half, refit, hist, nullptr);
    if (rc != QGX_OK) return rc;
  }
  ExchangeUpdate dual{2, st->Y, st->Y, st->scalars};                          // Y_{t+1} = Y_t - mean
  rc = exchange_impl(c, src2, K, d, cfg_half, xid + 1u, 1, mean, bits ? bits + K : nullptr, &dual, 2, st->scalars, 0);
  if (rc != QGX_OK) return rc;
  {
    ScopedKernelTimer timer(c, QGX_KERNEL_FINISH);
    k_eg_finish<<<grid_for(c, d, 256), 256, 0, c->stream>>>(st->X, st->Y, st->Xbar, st->Xhalf, st->anchor, st->scalars, d, K, st->t);
  }
  count_launch(c);
  st->t += 1;
  return cuda_status(cudaGetLastError());
}

qgx_status qgx_eg_step(qgx_ctx* c, qgx_eg_state* st, const qgx_operator* op, const float* noise_t, const float* noise_half,
                       qgx_quant_cfg* cfg, int refit, uint64_t* bits) {
  return eg_step_impl(c, st, op, noise_t, noise_half, cfg, cfg, refit, bits);
}

qgx_status qgx_eg_step_two_tables(qgx_ctx* c, qgx_eg_state* st, const qgx_operator* op, const float* noise_t,
                                  const float* noise_half, qgx_quant_cfg* cfg_t, qgx_quant_cfg* cfg_half, int refit,
                                  uint64_t* bits) {
  if (!cfg_t || !cfg_half || cfg_t == cfg_half) return QGX_ERR_INVALID_ARG;
  // the decode pass compares sub-block by sub-block: both exchanges need the same bucket and sub-block sizes
  if (cfg_t->bucket != cfg_half->bucket || eff_subblock(cfg_t->bucket, cfg_t->cb.subblock) != eff_subblock(cfg_half->bucket, cfg_half->cb.subblock))
    return QGX_ERR_INVALID_ARG;
  return eg_step_impl(c, st, op, noise_t, noise_half, cfg_t, cfg_half, refit, bits);
}

qgx_status qgx_family_step(qgx_ctx* c, qgx_eg_state* st, int method, const qgx_operator* op, const float* noise,
                           qgx_quant_cfg* cfg, int refit, float* mean_prev, uint64_t* bits) {
  if (!c || !st || !op || !cfg || !st->X || !st->Y || !st->Xbar || !st->Xhalf || !st->anchor || !st->scalars || st->t < 1 ||
      op->d != st->d || st->K < 1)
    return QGX_ERR_INVALID_ARG;
  if (method != QGX_METHOD_DA && method != QGX_METHOD_OPTDA) return QGX_ERR_INVALID_ARG;
  if (method == QGX_METHOD_OPTDA && !mean_prev) return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  const size_t d = st->d;
  const int K = st->K;
  float* a = (float*)ws_get(c, WS_OPVAL, sizeof(float) * d);
  float* mean = method == QGX_METHOD_OPTDA ? mean_prev : (float*)ws_get(c, WS_MEAN, sizeof(float) * d);
  if (!a || !mean) return QGX_ERR_CUDA;

  if (method == QGX_METHOD_OPTDA && st->t > 1) {
    ScopedKernelTimer timer(c, QGX_KERNEL_FINISH);
    k_half_from_mean<<<grid_for(c, d, 256), 256, 0, c->stream>>>(st->X, mean_prev, st->scalars, st->Xhalf, d);   // g_{k,t-1/2}
    count_launch(c);
  } else {                                                                       // no earlier feedback: X_{t+1/2} = X_t
    if (cudaMemcpyAsync(st->Xhalf, st->X, sizeof(float) * d, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
      return QGX_ERR_CUDA;
  }
  qgx_status rc = apply_operator_impl(c, op, st->Xhalf, a);                    // A(X_{t+1/2})
  if (rc != QGX_OK) return rc;
  DualSource src{noise, a, 0, op->noise_model == QGX_NOISE_RELATIVE ? 1 : 0};
  if (refit != QGX_REFIT_NONE) {
    double* hist = (double*)ws_get(c, WS_HIST, sizeof(double) * (size_t)std::max(cfg->nbins, 1));
    if (!hist) return QGX_ERR_CUDA;
    rc = refit_from_source(c, src, K, d, cfg, refit, hist, nullptr);
    if (rc != QGX_OK) return rc;
  }
  // the symbol modes of the decode pass: dual averaging adds the squared vectors themselves; the optimistic variant
  // compares with the vectors kept by the previous iteration (none in the first) and keeps the new ones
  const int sym_mode = method == QGX_METHOD_DA ? 4 : (st->t == 1 ? 5 : 3);
  const int slot = st->t & 1;                                                    // the kept norms live in the other slot
  ExchangeUpdate dual{2, st->Y, st->Y, st->scalars};                            // Y_{t+1} = Y_t - mean
  rc = exchange_impl(c, src, K, d, cfg, 2u * (uint32_t)st->t + 1u, slot, mean, bits, &dual, sym_mode, st->scalars, 0);
  if (rc != QGX_OK) return rc;
  {
    ScopedKernelTimer timer(c, QGX_KERNEL_FINISH);
    k_eg_finish<<<grid_for(c, d, 256), 256, 0, c->stream>>>(st->X, st->Y, st->Xbar, st->Xhalf, st->anchor, st->scalars, d, K, st->t);
  }
  count_launch(c);
  st->t += 1;
  return cuda_status(cudaGetLastError());
}

}  // extern "C"
