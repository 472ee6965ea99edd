// Context, status and the host-side helpers of the qgx library: level-table checks, stream
// geometry, prefix-code builders (App. J), the level fit of Sec. 3.3 and the symbol weights of
// App. E.  Nothing here touches vector data; the kernels live in the other translation units.
#include "qgx_common.cuh"

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

namespace qgx {

qgx_status cuda_status(cudaError_t e) { return e == cudaSuccess ? QGX_OK : QGX_ERR_CUDA; }

qgx_status check_levels_host(const float* lev, int nlev) {
  if (lev == nullptr || nlev < 2 || nlev > QGX_MAX_LEVELS) return QGX_ERR_BAD_LEVELS;
  if (!(lev[0] == 0.0f) || !(lev[nlev - 1] == 1.0f)) return QGX_ERR_BAD_LEVELS;
  for (int j = 1; j < nlev; ++j)
    if (!(lev[j - 1] < lev[j])) return QGX_ERR_BAD_LEVELS;
  return QGX_OK;
}

// Validates a codebook (lengths in [1, 12], prefix-free) and lays it out for the kernels:
// stream order means the first transmitted bit sits at bit 0.
qgx_status make_code_table(const qgx_codebook* cb, int bucket, CodeTable* out) {
  if (cb == nullptr || cb->nlev < 2 || cb->nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  out->nlev = cb->nlev;
  int maxlen = 0;
  for (int j = 0; j < cb->nlev; ++j) {
    const int L = cb->len[j];
    if (L < 1 || L > QGX_MAX_CODE_LEN) return QGX_ERR_INVALID_ARG;
    if (cb->code[j] >> L) return QGX_ERR_INVALID_ARG;
    maxlen = std::max(maxlen, L);
    uint32_t r = 0;
    for (int b = 0; b < L; ++b) r |= ((cb->code[j] >> (L - 1 - b)) & 1u) << b;
    out->rev[j] = (uint16_t)r;
    out->len[j] = (uint8_t)L;
  }
  // no codeword may be a prefix of another
  for (int a = 0; a < cb->nlev; ++a)
    for (int b = 0; b < cb->nlev; ++b) {
      if (a == b || cb->len[a] > cb->len[b]) continue;
      if ((cb->code[b] >> (cb->len[b] - cb->len[a])) == cb->code[a]) return QGX_ERR_INVALID_ARG;
    }
  out->maxlen = maxlen;
  out->G = eff_subblock(bucket, cb->subblock);
  if (out->G % kQuad != 0) return QGX_ERR_INVALID_ARG;
  out->has_header = out->G < bucket ? 1 : 0;
  if ((uint64_t)out->G * (uint64_t)(maxlen + 1) > 0xFFFFull && out->has_header) return QGX_ERR_INVALID_ARG;
  return QGX_OK;
}

// Tables of round_fast.  The margin bounds, in units of 1 / S of an interval, everything by which the
// kernel's S (F - r) can differ from the exact routine's decision variable: u2 against the correctly
// rounded quotient and the rounding of b and of the knot (together under 2 * 2^-22 (l_{tau+1} + 2^-16) / width,
// with the narrower of the two intervals around a level), the rounding of a, three fused multiply-adds of
// results below 2^24, the slope-change term, and the exact routine's own roundings of xi plus the variate's
// dropped last bit (3.02 S / 2^24).
void make_round_table(const float* lev, int nlev, RoundTable* out) {
  std::memset(out, 0, sizeof(*out));
  out->nlev = nlev;
  const double S = nlev <= 17 ? 524288.0 : 262144.0;
  const double c0 = (double)kRoundShift;
  double b[QGX_MAX_LEVELS] = {0}, width[QGX_MAX_LEVELS] = {0};
  for (int t = 0; t <= nlev - 2; ++t) {
    width[t] = (double)(float)(lev[t + 1] - lev[t]);             // the fp32 difference the exact routine divides by
    b[t] = S / width[t];
    out->b[t] = (float)b[t];
    out->a[t] = (float)(S * t - b[t] * ((double)lev[t] + c0) + 1.5 * S);
  }
  for (int j = 0; j < QGX_MAX_LEVELS; ++j) {
    const bool interior = j >= 1 && j <= nlev - 2;
    out->knot[j] = interior ? (float)((double)lev[j] + c0) : 4.0f;
    out->db[j] = interior ? (float)(b[j] - b[j - 1]) : 0.0f;
  }
  double margin = 0.0;
  for (int t = 0; t <= nlev - 2; ++t) {
    const double wmin = std::min(width[t], t + 1 <= nlev - 2 ? width[t + 1] : width[t]);
    const double a_ulp = (double)std::nextafter(std::fabs(out->a[t]), INFINITY) - (double)std::fabs(out->a[t]);
    const double e = 2.0 * S * 0x1p-22 * ((double)lev[t + 1] + c0) / wmin + a_ulp + 1.5 + 1.0 + 3.02 * S / 16777216.0;
    margin = std::max(margin, e);
  }
  margin = (margin + 2.0) * 1.01;
  // the octet encoder's variant: only the leading 16 bits h of the variate are subtracted, as the float 2^23 + h
  // times -S 2^-16 (the 2^23 part is folded into a16); r lies within 2^-17 of the centre (h + 1/2) 2^-16
  double margin16 = 0.0;
  for (int t = 0; t <= nlev - 2; ++t) {
    out->a16[t] = (float)(S * t - b[t] * ((double)lev[t] + c0) + 0.5 * S - S / 131072.0 + 8388608.0 * (S / 65536.0));
    const double wmin = std::min(width[t], t + 1 <= nlev - 2 ? width[t + 1] : width[t]);
    const double a_ulp = (double)std::nextafter(std::fabs(out->a16[t]), INFINITY) - (double)std::fabs(out->a16[t]);
    const double e = 2.0 * S * 0x1p-22 * ((double)lev[t + 1] + c0) / wmin + a_ulp + 1.5 + 1.0 + 1.01 * S / 131072.0;
    margin16 = std::max(margin16, e);
  }
  margin16 = (margin16 + 2.0) * 1.01;
  bool usable = std::isfinite(margin) && margin < S / 4.0 && std::isfinite(margin16) && margin16 < S / 4.0;
  // the coarsest bins that still hold at most one level each (coarser bins are stored in more copies: see kKeyShiftMin)
  int shift = -1;
  for (int sh = kKeyShiftMax; sh >= kKeyShiftMin && usable && shift < 0; --sh) {
    const uint32_t nbins = ((kKeyTop - kKeyBase) >> sh) + 1u;
    bool ok = true;
    for (uint32_t i = 0; i < nbins && ok; ++i) {
      const uint32_t lo_bits = kKeyBase + (i << sh), hi_bits = kKeyBase + ((i + 1u) << sh) - 1u;
      float lo, hi;
      std::memcpy(&lo, &lo_bits, 4);
      std::memcpy(&hi, &hi_bits, 4);
      int inside = 0;
      for (int j = 1; j <= nlev - 2; ++j) inside += (out->knot[j] > lo && out->knot[j] <= hi) ? 1 : 0;
      if (inside > 1) ok = false;
    }
    if (ok) shift = sh;
  }
  if (shift < 0) usable = false;
  out->key_shift = shift < 0 ? kKeyShiftMin : shift;
  out->usable = usable ? 1 : 0;
  out->thr = usable ? (float)(S / 2.0 - margin) : -1.0f;
  out->neg_qscale = (float)(-S / 8388608.0);
  out->thr16 = usable ? (float)(S / 2.0 - margin16) : -1.0f;
  out->neg_qscale16 = (float)(-S / 65536.0);
  out->magic = (float)(1.5 * 8388608.0 * S);
}

void* ws_get(qgx_ctx* c, int which, size_t bytes) {
  if (bytes == 0) bytes = 16;
  if (c->ws_bytes[which] >= bytes) return c->ws[which];
  if (c->ws[which]) {
    cudaStreamSynchronize(c->stream);
    cudaFree(c->ws[which]);
    c->ws[which] = nullptr;
    c->ws_bytes[which] = 0;
  }
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  c->ws[which] = p;
  c->ws_bytes[which] = bytes;
  return p;
}

}  // namespace qgx

using namespace qgx;

static void timing_free(qgx_ctx* c) {
  for (int i = 0; i < 2 * c->timing_cap; ++i) cudaEventDestroy(c->timing_ev[i]);
  delete[] c->timing_ev;
  delete[] c->timing_kind;
  c->timing_ev = nullptr;
  c->timing_kind = nullptr;
  c->timing_cap = c->timing_used = c->timing_on = 0;
}

extern "C" {

qgx_status qgx_create(qgx_ctx** out, int device, void* cuda_stream) {
  if (out == nullptr) return QGX_ERR_INVALID_ARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) { cudaGetLastError(); return QGX_ERR_CUDA; }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return QGX_ERR_CUDA; }
  qgx_ctx* c = new (std::nothrow) qgx_ctx();
  if (!c) return QGX_ERR_CUDA;
  std::memset(c, 0, sizeof(*c));
  c->device = device;
  c->sym_slot = -1;
  c->wait_limit = kSpinLimit;
  c->num_sms = 1;
  if (cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || c->num_sms < 1) { cudaGetLastError(); c->num_sms = 1; }
  c->stream = (cudaStream_t)cuda_stream;
  if (cudaMalloc((void**)&c->dstatus, sizeof(DevStatus)) != cudaSuccess ||
      cudaMemsetAsync(c->dstatus, 0, sizeof(DevStatus), c->stream) != cudaSuccess ||
      cudaMallocHost((void**)&c->hstatus, sizeof(DevStatus)) != cudaSuccess) {
    cudaGetLastError();
    if (c->dstatus) cudaFree(c->dstatus);
    delete c;
    return QGX_ERR_CUDA;
  }
  *out = c;
  return QGX_OK;
}

void qgx_destroy(qgx_ctx* c) {
  if (!c) return;
  cudaSetDevice(c->device);
  cudaStreamSynchronize(c->stream);
  if (c->timing_ev) timing_free(c);
  free_seg_children(c);
  free_table_cache(c);
  for (int i = 0; i < 24; ++i)
    if (c->ws[i]) cudaFree(c->ws[i]);
  cudaFree(c->dstatus);
  cudaFreeHost(c->hstatus);
  delete c;
}

qgx_status qgx_sync_status(qgx_ctx* c) {
  if (!c) return QGX_ERR_INVALID_ARG;
  if (cudaMemcpyAsync(c->hstatus, c->dstatus, sizeof(DevStatus), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaMemsetAsync(c->dstatus, 0, sizeof(DevStatus), c->stream) != cudaSuccess ||
      cudaStreamSynchronize(c->stream) != cudaSuccess) {
    cudaGetLastError();
    return QGX_ERR_CUDA;
  }
  const unsigned int e = c->hstatus[0];
  return e <= (unsigned int)QGX_ERR_CUDA ? (qgx_status)e : QGX_ERR_CUDA;
}

const char* qgx_status_str(qgx_status s) {
  switch (s) {
    case QGX_OK: return "ok";
    case QGX_ERR_INVALID_ARG: return "invalid argument";
    case QGX_ERR_BAD_LEVELS: return "level table is not 0 = l_0 < ... < l_last = 1 with 2..32 entries";
    case QGX_ERR_CAPACITY: return "stream capacity too small";
    case QGX_ERR_CORRUPT: return "corrupt stream or symbol";
    case QGX_ERR_NONFINITE: return "non-finite bucket norm";
    case QGX_ERR_TIMEOUT: return "device-side wait ran out";
    case QGX_ERR_CUDA: return "CUDA runtime error";
    case QGX_ERR_TOO_LARGE: return "problem larger than the fixed scratch of the no-allocation entry point";
  }
  return "unknown status";
}

uint64_t qgx_launch_count(const qgx_ctx* c) { return c ? c->launches + seg_children_launches(c) : 0; }

qgx_status qgx_timing_enable(qgx_ctx* c, int max_records) {
  if (!c || max_records < 0 || max_records > (1 << 20)) return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  cudaStreamSynchronize(c->stream);
  if (c->timing_ev) timing_free(c);
  if (max_records == 0) return QGX_OK;
  c->timing_ev = new (std::nothrow) cudaEvent_t[2 * (size_t)max_records];
  c->timing_kind = new (std::nothrow) int[(size_t)max_records];
  if (!c->timing_ev || !c->timing_kind) return QGX_ERR_CUDA;
  for (int i = 0; i < 2 * max_records; ++i)
    if (cudaEventCreate(&c->timing_ev[i]) != cudaSuccess) { c->timing_cap = i / 2; timing_free(c); return QGX_ERR_CUDA; }
  c->timing_cap = max_records;
  c->timing_used = 0;
  c->timing_on = 1;
  return QGX_OK;
}

qgx_status qgx_timing_read(qgx_ctx* c, int kernel, int reset, int* launches, double* total_ms) {
  if (!c || !launches || !total_ms || kernel < 0 || kernel >= QGX_KERNEL_COUNT) return QGX_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return QGX_ERR_CUDA;
  int n = 0;
  double ms = 0.0;
  for (int i = 0; i < c->timing_used; ++i) {
    if (c->timing_kind[i] != kernel) continue;
    float t = 0.0f;
    if (cudaEventElapsedTime(&t, c->timing_ev[2 * i], c->timing_ev[2 * i + 1]) != cudaSuccess) return QGX_ERR_CUDA;
    ms += (double)t;
    ++n;
  }
  *launches = n;
  *total_ms = ms;
  if (reset) c->timing_used = 0;
  return QGX_OK;
}

qgx_status qgx_check_levels(const float* levels, int nlev) { return check_levels_host(levels, nlev); }

size_t qgx_stream_capacity_words(size_t d, int bucket, int subblock, int maxlen) {
  if (bucket < 1 || maxlen < 1) return 0;
  const uint64_t B = (uint64_t)bucket, G = (uint64_t)eff_subblock(bucket, subblock);
  const uint64_t nfull = d / B, tail = d % B;
  auto words = [&](uint64_t len) {
    const uint64_t nsub = (G < B) ? ceil_div_u64(len, G) : 0;
    return ceil_div_u64(kNormBits + 16 * nsub + len * (uint64_t)(maxlen + 1), 32);
  };
  return (size_t)(nfull * words(B) + (tail ? words(tail) : 0));
}

// canonical codewords from lengths: sorted by (length, index), each the previous plus one,
// shifted left when the length grows
static void assign_canonical(qgx_codebook* cb) {
  int idx[QGX_MAX_LEVELS];
  for (int j = 0; j < cb->nlev; ++j) idx[j] = j;
  std::stable_sort(idx, idx + cb->nlev, [&](int a, int b) { return cb->len[a] < cb->len[b]; });
  uint32_t next = 0;
  int curlen = cb->len[idx[0]];
  cb->maxlen = 0;
  for (int r = 0; r < cb->nlev; ++r) {
    const int j = idx[r];
    next <<= (cb->len[j] - curlen);
    curlen = cb->len[j];
    cb->code[j] = next++;
    cb->maxlen = std::max<int>(cb->maxlen, curlen);
  }
}

qgx_status qgx_build_codebook_fixed(int nlev, int subblock, qgx_codebook* cb) {
  if (cb == nullptr || nlev < 2 || nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  std::memset(cb, 0, sizeof(*cb));
  cb->nlev = nlev;
  cb->subblock = subblock;
  int bits = 1;
  while ((1 << bits) < nlev) ++bits;
  for (int j = 0; j < nlev; ++j) cb->len[j] = (uint8_t)bits;
  assign_canonical(cb);
  return QGX_OK;
}

// Elias' recursive code of j + 1 for level j.  The codeword is the closing 0 preceded by groups; walking
// backwards from the integer itself, each group is the binary form of the current value and the next value is
// that group's bit count minus one.  Groups are placed from the low end of the word upwards.
qgx_status qgx_build_codebook_elias(int nlev, int subblock, qgx_codebook* cb) {
  if (cb == nullptr || nlev < 2 || nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  std::memset(cb, 0, sizeof(*cb));
  cb->nlev = nlev;
  cb->subblock = subblock;
  for (int j = 0; j < nlev; ++j) {
    uint32_t word = 0;                    // the closing 0
    int used = 1;
    for (uint32_t value = (uint32_t)j + 1u; value > 1u;) {
      int width = 0;
      while ((value >> width) != 0u) ++width;
      word |= value << used;
      used += width;
      value = (uint32_t)width - 1u;
    }
    if (used > QGX_MAX_CODE_LEN) return QGX_ERR_INVALID_ARG;
    cb->len[j] = (uint8_t)used;
    cb->code[j] = word;
    cb->maxlen = std::max<int>(cb->maxlen, used);
  }
  return QGX_OK;
}

// Huffman lengths: a forest kept as parent links; each round joins the two lightest roots
// (among equal weights the root that has existed longest first) and every leaf below gains a bit.
static int huffman_depths(const double* w, int n, int* depth) {
  double weight[2 * QGX_MAX_LEVELS];
  int parent[2 * QGX_MAX_LEVELS];
  bool root[2 * QGX_MAX_LEVELS];
  int count = n;
  for (int j = 0; j < n; ++j) { weight[j] = w[j]; parent[j] = -1; root[j] = true; }
  for (int round = 0; round + 1 < n; ++round) {
    int first = -1, second = -1;
    for (int j = 0; j < count; ++j) {
      if (!root[j]) continue;
      if (first < 0 || weight[j] < weight[first]) first = j;
    }
    for (int j = 0; j < count; ++j) {
      if (!root[j] || j == first) continue;
      if (second < 0 || weight[j] < weight[second]) second = j;
    }
    weight[count] = weight[first] + weight[second];
    parent[count] = -1;
    root[count] = true;
    root[first] = root[second] = false;
    parent[first] = parent[second] = count;
    ++count;
  }
  int deepest = 0;
  for (int j = 0; j < n; ++j) {
    int dep = 0;
    for (int q = j; parent[q] >= 0; q = parent[q]) ++dep;
    depth[j] = dep < 1 ? 1 : dep;
    deepest = std::max(deepest, depth[j]);
  }
  return deepest;
}

qgx_status qgx_build_codebook_huffman(const double* p, int nlev, int subblock, qgx_codebook* cb) {
  if (cb == nullptr || p == nullptr || nlev < 2 || nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  for (int j = 0; j < nlev; ++j)
    if (!(p[j] >= 0.0) || !std::isfinite(p[j])) return QGX_ERR_INVALID_ARG;
  std::memset(cb, 0, sizeof(*cb));
  cb->nlev = nlev;
  cb->subblock = subblock;
  double w[QGX_MAX_LEVELS];
  int depth[QGX_MAX_LEVELS];
  for (int j = 0; j < nlev; ++j) w[j] = p[j];
  for (int m = 0; huffman_depths(w, nlev, depth) > QGX_MAX_CODE_LEN; ++m) {
    const double flat = std::ldexp(1.0, m - 16);
    for (int j = 0; j < nlev; ++j) w[j] = p[j] + flat;
  }
  for (int j = 0; j < nlev; ++j) cb->len[j] = (uint8_t)depth[j];
  assign_canonical(cb);
  return QGX_OK;
}

// ---- level fit ------------------------------------------------------------------------------
namespace {

// The histogram as a density that is constant inside each bin.  cum0 / cum1 are the mass and the
// first moment up to each bin edge.
struct BinnedCdf {
  int n;
  double width;
  std::vector<double> mass, cum0, cum1;
  BinnedCdf(const double* h, int nbins) : n(nbins), width(1.0 / nbins), mass(h, h + nbins), cum0(nbins + 1), cum1(nbins + 1) {
    cum0[0] = cum1[0] = 0.0;
    for (int j = 0; j < n; ++j) {
      const double mid = (j + 0.5) * width;              // centroid of a uniform bin
      cum0[j + 1] = cum0[j] + mass[j];
      cum1[j + 1] = cum1[j] + mass[j] * mid;
    }
  }
  int bin_of(double x) const { return std::min(n - 1, std::max(0, (int)(x * n))); }
  double m0(double x) const {                            // int_0^x dF
    if (x <= 0.0) return 0.0;
    if (x >= 1.0) return cum0[n];
    const int j = bin_of(x);
    return cum0[j] + mass[j] * (x - j * width) / width;
  }
  double m1(double x) const {                            // int_0^x u dF
    if (x <= 0.0) return 0.0;
    if (x >= 1.0) return cum1[n];
    const int j = bin_of(x);
    const double lo = j * width;
    return cum1[j] + mass[j] / width * 0.5 * (x - lo) * (x + lo);
  }
  // smallest x with m0(x) >= target
  double inverse(double target) const {
    if (target <= 0.0) return 0.0;
    if (target >= cum0[n]) {
      int j = n;
      while (j > 0 && cum0[j - 1] >= cum0[n]) --j;       // right edge of the last bin that holds mass
      return j * width;
    }
    const int j = (int)(std::lower_bound(cum0.begin() + 1, cum0.end(), target) - (cum0.begin() + 1));
    if (!(mass[j] > 0.0)) return j * width;
    return j * width + (target - cum0[j]) / mass[j] * width;
  }
};

}  // namespace

qgx_status qgx_code_bits(const uint64_t* counts, const qgx_codebook* cb, uint64_t* bits) {
  if (!counts || !cb || !bits || cb->nlev < 2 || cb->nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  uint64_t total = 0;
  for (int j = 0; j < cb->nlev; ++j) total += counts[j] * (uint64_t)(cb->len[j] + (j ? 1u : 0u));   // codeword, and a sign bit unless level 0
  *bits = total;
  return QGX_OK;
}

qgx_status qgx_choose_code_host(const uint64_t* counts, qgx_codebook* cb, int allow_rebuild, uint64_t* bits, int* winner) {
  if (!counts || !cb || !bits || !winner || cb->nlev < 2 || cb->nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  const int nlev = cb->nlev, sub = cb->subblock;
  qgx_codebook cand[4];
  bool have[4] = {true, false, false, false};
  cand[0] = *cb;
  uint64_t sent = 0;
  for (int j = 0; j < nlev; ++j) sent += counts[j];
  if (allow_rebuild && sent > 0) {                      // the code that the counts themselves call for
    double w[QGX_MAX_LEVELS];
    for (int j = 0; j < nlev; ++j) w[j] = (double)counts[j] / (double)sent;
    have[1] = qgx_build_codebook_huffman(w, nlev, sub, &cand[1]) == QGX_OK;
  }
  have[2] = qgx_build_codebook_elias(nlev, sub, &cand[2]) == QGX_OK;
  have[3] = qgx_build_codebook_fixed(nlev, sub, &cand[3]) == QGX_OK;
  int best = 0;
  for (int cnd = 0; cnd < 4; ++cnd) {
    bits[cnd] = ~(uint64_t)0;
    if (have[cnd]) qgx_code_bits(counts, &cand[cnd], &bits[cnd]);
    if (have[cnd] && bits[cnd] < bits[best]) best = cnd;   // ties keep the earlier candidate
  }
  *cb = cand[best];
  *winner = best;
  return QGX_OK;
}

qgx_status qgx_choose_code(qgx_ctx* c, qgx_quant_cfg* cfg, int allow_rebuild, uint64_t* counts_dev, uint64_t* bits, int* winner) {
  if (!c || !cfg || !counts_dev || !bits || !winner) return QGX_ERR_INVALID_ARG;
  if (cfg->cb.nlev != cfg->nlev || c->sym_nlev != cfg->nlev) return QGX_ERR_INVALID_ARG;
  qgx_status rc = qgx_level_counts(c, counts_dev);
  if (rc != QGX_OK) return rc;
  uint64_t host[QGX_MAX_LEVELS];
  if (cudaMemcpyAsync(host, counts_dev, sizeof(host), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaStreamSynchronize(c->stream) != cudaSuccess) {
    cudaGetLastError();
    return QGX_ERR_CUDA;
  }
  return qgx_choose_code_host(host, &cfg->cb, allow_rebuild, bits, winner);
}

qgx_status qgx_fit_levels(const double* hist, int nbins, float* levels, int nlev, int first_fit) {
  if (hist == nullptr || levels == nullptr || nbins < 1 || nlev < 2 || nlev > QGX_MAX_LEVELS) return QGX_ERR_INVALID_ARG;
  for (int j = 0; j < nbins; ++j)
    if (!(hist[j] >= 0.0) || !std::isfinite(hist[j])) return QGX_ERR_INVALID_ARG;
  BinnedCdf F(hist, nbins);
  const double total = F.cum0[nbins];
  const double min_gap = std::ldexp(1.0, -20);
  double l[QGX_MAX_LEVELS];
  if (first_fit) {
    for (int j = 0; j < nlev; ++j) l[j] = F.inverse(total * j / (double)(nlev - 1));
    l[0] = 0.0;
    l[nlev - 1] = 1.0;
  } else {
    if (check_levels_host(levels, nlev) != QGX_OK) return QGX_ERR_BAD_LEVELS;
    for (int j = 0; j < nlev; ++j) l[j] = levels[j];
  }
  for (int j = 1; j <= nlev - 2; ++j) l[j] = std::max(l[j], l[j - 1] + min_gap);
  for (int j = nlev - 2; j >= 1; --j) l[j] = std::min(l[j], l[j + 1] - min_gap);
  if (total > 0.0) {
    for (int sweep = 0; sweep < 32; ++sweep) {
      double moved = 0.0;
      for (int j = 1; j <= nlev - 2; ++j) {
        const double a = l[j - 1], c = l[j + 1];
        const double Fa = F.m0(a), Fc = F.m0(c);
        if (!(Fc - Fa > 0.0)) continue;
        // d/dl of the (QAda) objective is (c - a) F(l) - [c F(c) - a F(a) - (M1(c) - M1(a))]:
        // the coordinate minimiser is where the cdf reaches this value
        const double target = (c * Fc - a * Fa - (F.m1(c) - F.m1(a))) / (c - a);
        double x = F.inverse(target);
        x = std::min(std::max(x, a + min_gap), c - min_gap);
        moved = std::max(moved, std::fabs(x - l[j]));
        l[j] = x;
      }
      if (moved < 1e-7) break;
    }
  }
  levels[0] = 0.0f;
  levels[nlev - 1] = 1.0f;
  for (int j = 1; j <= nlev - 2; ++j) levels[j] = (float)l[j];
  return check_levels_host(levels, nlev);
}

qgx_status qgx_symbol_pmf(const double* hist, int nbins, const float* levels, int nlev, double* p) {
  if (hist == nullptr || p == nullptr || nbins < 1) return QGX_ERR_INVALID_ARG;
  if (check_levels_host(levels, nlev) != QGX_OK) return QGX_ERR_BAD_LEVELS;
  BinnedCdf F(hist, nbins);
  const double total = F.cum0[nbins];
  for (int j = 0; j < nlev; ++j) p[j] = 0.0;
  if (!(total > 0.0)) { p[0] = 1.0; return QGX_OK; }
  // a coordinate in [l_j, l_{j+1}] goes up with probability (u - l_j)/(l_{j+1} - l_j): walk the
  // intervals and split each one's mass between its two end levels
  for (int j = 0; j + 1 < nlev; ++j) {
    const double a = levels[j], c = levels[j + 1];
    const double mass = F.m0(c) - F.m0(a);
    const double up = ((F.m1(c) - F.m1(a)) - a * mass) / (c - a);
    p[j + 1] += up / total;
    p[j] += (mass - up) / total;
  }
  return QGX_OK;
}

}  // extern "C"
