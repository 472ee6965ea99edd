// qgx_quantize (Definition 1 per bucket) and qgx_average (the aggregation of Algorithm 1).
#include "qgx_bucket.cuh"

namespace qgx {

// One CTA per (bucket, worker).  The bucket stays in registers between the norm reduction and
// the rounding pass, so v is read from HBM exactly once.
template <int V4>
__global__ void __launch_bounds__(512) k_quantize(DualSource src, size_t d, int bucket, const __grid_constant__ LevelTable lt,
                                                   const __grid_constant__ PhiloxKey key, const __grid_constant__ RoundTable rt,
                                                   uint32_t xid, int norm_type, int norms_supplied, bool vec_ok,
                                                   float* __restrict__ norms, uint8_t* __restrict__ sym, DevStatus* st) {
  __shared__ float s_lev[QGX_MAX_LEVELS];
  __shared__ float4 s_bin[kBinEntries];
  fill_bin_table(s_bin, rt);
  __shared__ double s_red[34];
  const size_t b = blockIdx.x, k = blockIdx.y;
  const size_t nb = gridDim.x;
  const size_t lo = b * (size_t)bucket;
  const int len = (int)min((size_t)bucket, d - lo);
  if (threadIdx.x < QGX_MAX_LEVELS) s_lev[threadIdx.x] = threadIdx.x < lt.nlev ? lt.lev[threadIdx.x] : 1.0f;

  BucketRegs<V4> r;
  load_bucket<V4>(r, src, k, d, lo, len, vec_ok);
  float norm;
  if (norms_supplied) {
    norm = norms[k * nb + b];
    __syncthreads();
  } else {
    norm = bucket_norm<V4>(r, norm_type, s_red);
    if (threadIdx.x == 0) norms[k * nb + b] = norm;
  }
  const bool finite = (norm - norm) == 0.0f;
  if (!finite && threadIdx.x == 0) latch_error(st, QGX_ERR_NONFINITE);
  const RoundConsts rc = round_consts(rt, norm);

  uint8_t* out = sym + k * d + lo;
  const bool sym_vec = vec_ok;            // d % 4 == 0 and bucket % 4 == 0: every quad is 4-byte aligned
#pragma unroll
  for (int j = 0; j < V4; ++j) {
    const int q = j * (int)blockDim.x + (int)threadIdx.x;
    const int e = q * kQuad;
    if (e >= len) continue;
    uint32_t packed = 0;
    if (finite && norm != 0.0f) {
      const uint64_t ctr = (uint64_t)(lo >> 2) + (uint64_t)q;      // (coordinate index) / 4
      const uint4 w = philox4x32_10((uint32_t)ctr, (uint32_t)(ctr >> 32), (uint32_t)k, xid, key);
      const float4 x = r.x[j];
      const uint32_t code4 = quantize_quad_codes(x, w, rc, norm, s_bin, s_lev, lt.nlev);
      packed = (code4 & 0x1f1f1f1fu) | ((code4 & 0x20202020u) << 2);      // symbol bytes: level | sign << 7
    }
    if (e + kQuad <= len && sym_vec) {
      *reinterpret_cast<uint32_t*>(out + e) = packed;
    } else {
      for (int c = 0; c < kQuad && e + c < len; ++c) out[e + c] = (uint8_t)(packed >> (8 * c));
    }
  }
}

// out[i] = (sum_k vhat[k][i]) / K, the sum taken in the order k = 0..K-1; one thread per quad.
__global__ void __launch_bounds__(256) k_average(const float* __restrict__ norms, const uint8_t* __restrict__ sym, int K,
                                                 size_t d, int bucket, size_t nb, LevelTable lt, bool vec_ok,
                                                 float* __restrict__ out, DevStatus* st) {
  __shared__ float s_lev[QGX_MAX_LEVELS];
  if (threadIdx.x < QGX_MAX_LEVELS) s_lev[threadIdx.x] = threadIdx.x < lt.nlev ? lt.lev[threadIdx.x] : 0.0f;
  __syncthreads();
  const size_t nquads = (d + kQuad - 1) / kQuad;
  const float Kf = (float)K;
  bool bad = false;
  for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < nquads; q += (size_t)gridDim.x * blockDim.x) {
    const size_t e = q * kQuad;
    const int nval = (int)min((size_t)kQuad, d - e);
    float acc[kQuad] = {0.f, 0.f, 0.f, 0.f};
    for (int k = 0; k < K; ++k) {
      uint32_t packed = 0;
      if (nval == kQuad && vec_ok) {
        packed = __ldcs(reinterpret_cast<const uint32_t*>(sym + (size_t)k * d + e));
      } else {
        for (int c = 0; c < nval; ++c) packed |= (uint32_t)sym[(size_t)k * d + e + c] << (8 * c);
      }
#pragma unroll
      for (int c = 0; c < kQuad; ++c) {
        if (c < nval) {
          const uint32_t s = (packed >> (8 * c)) & 0xffu;
          bad = bad || ((s & 31u) >= (uint32_t)lt.nlev);
          // a bucket never splits a quad when bucket % 4 == 0, but the tail of d may
          const float norm = norms[(size_t)k * nb + (e + c) / (size_t)bucket];
          acc[c] = __fadd_rn(acc[c], dequantize_symbol(s, norm, s_lev));
        }
      }
    }
    for (int c = 0; c < nval; ++c) out[e + c] = __fdiv_rn(acc[c], Kf);
  }
  if (bad) latch_error(st, QGX_ERR_CORRUPT);
}

static bool all_aligned16(std::initializer_list<const void*> ps) {
  for (const void* p : ps)
    if (p && (reinterpret_cast<uintptr_t>(p) & 15u)) return false;
  return true;
}

qgx_status launch_quantize(qgx_ctx* c, DualSource src, int K, size_t d, int bucket, const LevelTable& lt, int norm_type,
                           uint64_t seed, uint32_t xid, int norms_supplied, float* norms, uint8_t* sym) {
  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  const bool vec_ok = (d % kQuad == 0) && all_aligned16({src.v, src.a}) &&
                      ((reinterpret_cast<uintptr_t>(sym) & 3u) == 0);
  const PhiloxKey key = make_philox_key(seed);
  RoundTable qt;
  make_round_table(lt.lev, lt.nlev, &qt);
  const int v4 = bucket_v4(bucket);
  const dim3 grid((unsigned)nb, (unsigned)K);
  const int threads = bucket_threads(bucket, v4);
#define QGX_LAUNCH_Q(V)                                                                                      \
  k_quantize<V><<<grid, threads, 0, c->stream>>>(src, d, bucket, lt, key, qt, xid, norm_type, norms_supplied, \
                                                 vec_ok, norms, sym, c->dstatus)
  switch (v4) {
    case 1: QGX_LAUNCH_Q(1); break;
    case 2: QGX_LAUNCH_Q(2); break;
    case 4: QGX_LAUNCH_Q(4); break;
    default: QGX_LAUNCH_Q(8); break;
  }
#undef QGX_LAUNCH_Q
  count_launch(c);
  return cuda_status(cudaGetLastError());
}

}  // namespace qgx

using namespace qgx;

extern "C" {

qgx_status qgx_quantize(qgx_ctx* c, const float* v, int K, size_t d, int bucket, const float* levels, int nlev,
                        int norm_type, uint64_t seed, uint32_t exchange_id, int flags, float* norms, uint8_t* sym) {
  if (!c || !v || !norms || !sym || K < 1 || K > 65535 || d < 1 || bucket < kQuad || bucket > QGX_MAX_BUCKET ||
      bucket % kQuad != 0 || (norm_type != QGX_NORM_L2 && norm_type != QGX_NORM_LINF))
    return QGX_ERR_INVALID_ARG;
  if (check_levels_host(levels, nlev) != QGX_OK) return QGX_ERR_BAD_LEVELS;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  LevelTable lt;
  lt.nlev = nlev;
  for (int j = 0; j < QGX_MAX_LEVELS; ++j) lt.lev[j] = j < nlev ? levels[j] : 1.0f;
  DualSource src{v, nullptr, 0, 0};
  return launch_quantize(c, src, K, d, bucket, lt, norm_type, seed, exchange_id, (flags & QGX_NORMS_SUPPLIED) ? 1 : 0,
                         norms, sym);
}

qgx_status qgx_average(qgx_ctx* c, const float* norms, const uint8_t* sym, int K, size_t d, int bucket,
                       const float* levels, int nlev, float* out) {
  if (!c || !norms || !sym || !out || K < 1 || d < 1 || bucket < 1) return QGX_ERR_INVALID_ARG;
  if (check_levels_host(levels, nlev) != QGX_OK) return QGX_ERR_BAD_LEVELS;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  LevelTable lt;
  lt.nlev = nlev;
  for (int j = 0; j < QGX_MAX_LEVELS; ++j) lt.lev[j] = j < nlev ? levels[j] : 0.0f;
  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  const size_t nquads = (d + kQuad - 1) / kQuad;
  const bool vec_ok = (d % kQuad == 0) && ((reinterpret_cast<uintptr_t>(sym) & 3u) == 0);
  const int threads = 256;
  const unsigned blocks = (unsigned)std::min<size_t>((nquads + threads - 1) / threads, (size_t)c->num_sms * 16u);
  k_average<<<blocks, threads, 0, c->stream>>>(norms, sym, K, d, bucket, nb, lt, vec_ok, out, c->dstatus);
  count_launch(c);
  return cuda_status(cudaGetLastError());
}

}  // extern "C"
