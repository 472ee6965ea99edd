// Fused exchange: one pass over the dual vectors writes the compact streams (quantize + encode),
// one pass over the streams writes the mean (decode + average).  Same streams, bit for bit, and
// the same mean as qgx_quantize -> qgx_encode -> qgx_decode -> qgx_average.
#include "qgx_bucket.cuh"
#include "qgx_codec.cuh"

#include <cuda.h>

#include <algorithm>
#include <cstring>
#include <limits>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

namespace qgx {

// ---- chained scan of bucket lengths ("decoupled look-back") ----------------------------------
// status word of bucket (k, b): bits 62..63 state, bits 0..61 a word count.
constexpr unsigned long long kStEmpty = 0ull, kStAggregate = 1ull << 62, kStPrefix = 2ull << 62;
constexpr unsigned long long kStMask = 3ull << 62;

__device__ __forceinline__ unsigned long long ld_status(const unsigned long long* p) {
  return *reinterpret_cast<const volatile unsigned long long*>(p);
}
__device__ __forceinline__ void st_status(unsigned long long* p, unsigned long long v) {
  *reinterpret_cast<volatile unsigned long long*>(p) = v;
}

// Exclusive prefix (in words) of bucket b of one worker, by warp 0 of the CTA.  Buckets are handed
// out by a ticket counter in the order b-major, k-minor, so every predecessor (k, b') with b' < b
// belongs to a CTA that is already running or done: the wait below always ends; it is bounded all
// the same, and *timed_out reports a wait that ran out.
__device__ __forceinline__ unsigned long long lookback_prefix(unsigned long long* row /* status of worker k */, long long b,
                                                              int lane, int spin_limit, bool* timed_out) {
  unsigned long long prefix = 0;
  long long hi = b - 1;                                 // nearest predecessor not yet accounted for
  int spins = 0;
  bool fail = false;
  while (hi >= 0 && !fail) {
    const long long mine = hi - lane;
    unsigned long long s = kStPrefix;                   // positions before bucket 0 act as a zero prefix
    if (mine >= 0) s = ld_status(row + mine);
    const unsigned empty = __ballot_sync(0xffffffffu, (s & kStMask) == kStEmpty);
    const unsigned pref = __ballot_sync(0xffffffffu, (s & kStMask) == kStPrefix);
    // lanes are ordered from the nearest predecessor outwards
    const int first_pref = pref ? __ffs(pref) - 1 : 32;
    const int first_empty = empty ? __ffs(empty) - 1 : 32;
    if (first_empty < first_pref) {                     // a predecessor has not published yet
      if (++spins > spin_limit) fail = true;
      __nanosleep(64);
      continue;
    }
    const int take = first_pref < 32 ? first_pref + 1 : 32;
    unsigned long long part = lane < take ? (s & ~kStMask) : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    prefix += part;
    if (first_pref < 32) break;
    hi -= 32;
  }
  *timed_out = fail;
  return prefix;
}

struct EncodeArgs {
  DualSource src;
  size_t d;
  int bucket;
  int K;
  size_t nb;
  int norm_type;
  uint32_t xid;
  uint64_t quad_base;           // (index of the vector's first coordinate in the generator's counter space) / 4
  bool vec_ok;
  uint32_t* stream;
  size_t cap_words;
  uint32_t* bucket_bits;        // [K][nb]
  uint32_t* offsets;            // [K][nb] word offset of each bucket
  unsigned long long* total_bits;   // [K], zeroed before the launch
  float* norms;                 // [K][nb] (kept for the caller; the streams carry them too)
  unsigned long long* status;   // [K][nb], zeroed before the launch
  unsigned int* ticket;         // zeroed before the launch
  const struct EncodeTables* tables;   // the shared-memory tables of the configuration, built once (null: every CTA builds them)
  DevStatus* st;
  size_t nb_whole;              // buckets [0, nb_whole) of every worker belong to k_encode_staged ...
  size_t b_first;               // ... and buckets [b_first, nb) to k_exchange_encode
  int spin_limit;               // polls of a wait for another bucket's count before it gives up
};

// Norm of the bucket held by the CTA, one barrier: per-warp partials go to shared memory and every
// warp then reduces them in the same order (so all warps hold the same value).
template <int V4>
__device__ __forceinline__ float bucket_norm_all(const BucketRegs<V4>& r, int norm_type, double* red) {
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
    acc = __any_sync(0xffffffffu, bad) ? (double)__int_as_float(0x7fc00000) : (double)m;
  }
  if (lane == 0) red[warp] = acc;
  __syncthreads();
  double t = lane < nwarps ? red[lane] : 0.0;
  if (norm_type == QGX_NORM_L2) return (float)sqrt(warp_sum(t));
  const bool bad = __any_sync(0xffffffffu, t != t);
  const float m = warp_max((float)t);
  return bad ? __int_as_float(0x7fc00000) : m;
}

// Loads bucket [lo, lo + len) of worker k: warp w holds coordinates [w * 256 * P, (w + 1) * 256 * P), row j of
// them 32 octets (8 consecutive coordinates: two quads), lane l the l-th octet of the row.
template <int P>
__device__ __forceinline__ void load_bucket_octets(BucketRegs<2 * P>& r, const DualSource& s, size_t k, size_t d,
                                                   size_t lo, int len, bool vec_ok) {
  const size_t ld = s.ld ? s.ld : d;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (vec_ok && len == 256 * P * (int)(blockDim.x >> 5)) {
    // every lane holds full octets: the kind of source is decided once, not per quad
    const float4* pv = s.v ? reinterpret_cast<const float4*>(s.v + k * ld + lo) + ((warp * P * 32 + lane) << 1) : nullptr;
    const float4* pa = s.a ? reinterpret_cast<const float4*>(s.a + lo) + ((warp * P * 32 + lane) << 1) : nullptr;
    if (pa == nullptr) {
#pragma unroll
      for (int j = 0; j < 2 * P; ++j) r.x[j] = __ldcs(pv + (j >> 1) * 64 + (j & 1));
    } else if (pv == nullptr) {
#pragma unroll
      for (int j = 0; j < 2 * P; ++j) r.x[j] = __ldg(pa + (j >> 1) * 64 + (j & 1));
    } else if (s.mul) {
#pragma unroll
      for (int j = 0; j < 2 * P; ++j) r.x[j] = dual_combine(__ldg(pa + (j >> 1) * 64 + (j & 1)), __ldcs(pv + (j >> 1) * 64 + (j & 1)), 1);
    } else {
#pragma unroll
      for (int j = 0; j < 2 * P; ++j) r.x[j] = dual_combine(__ldg(pa + (j >> 1) * 64 + (j & 1)), __ldcs(pv + (j >> 1) * 64 + (j & 1)), 0);
    }
    return;
  }
#pragma unroll
  for (int j = 0; j < 2 * P; ++j) {
    const int e = ((((warp * P + (j >> 1)) * 32 + lane) << 1) + (j & 1)) * kQuad;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e + kQuad <= len && vec_ok) {
      if (s.a == nullptr) {
        x = __ldcs(reinterpret_cast<const float4*>(s.v + k * ld + lo + e));
      } else {
        const float4 av = __ldg(reinterpret_cast<const float4*>(s.a + lo + e));
        if (s.v) {
          const float4 u = __ldcs(reinterpret_cast<const float4*>(s.v + k * ld + lo + e));
          x = dual_combine(av, u, s.mul);
        } else {
          x = av;
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

// ---- rounding of one octet (eight consecutive coordinates of one lane) ---------------------------
// The rare way through an octet, out of line: every coordinate is tested again and the ones whose outcome the
// leading variate bits do not settle go through the exact routine.  Returns the eight signed level indices, one
// per byte.  w0, w1: the Philox blocks of the octet's two quads.
static __device__ __noinline__ uint64_t redo_octet(const float4 xa, const float4 xb, const uint4 w0, const uint4 w1, const RoundK rc,
                                                   float norm, const float* lev, int nlev) {
  const float x[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
  const uint32_t w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
  const float inv_S = -1.0f / (rc.nqs * 65536.0f);
  uint64_t out = 0;
  for (int i = 0; i < 8; ++i) {
    float worst = 0.0f;
    const float zi = round_signed(x[i], 0x4B000000u | (w[i] >> 16), rc, &worst);
    int idx = (int)fabsf(__fmul_rn(zi, inv_S));
    if (!(worst <= rc.thr)) idx = quantize_level_exact(fabsf(x[i]), norm, lev, nlev, w[i] >> 8);
    const int sidx = (__float_as_uint(x[i]) >> 31) ? -idx : idx;
    out |= (uint64_t)(uint8_t)(signed char)sidx << (8 * i);
  }
  return out;
}

// S * (signed level index) of the eight coordinates xa, xb of an octet, given the Philox blocks w0, w1 of its two
// quads.  S = the scale of the rounding table.
__device__ __forceinline__ void octet_levels_w(const float4 xa, const float4 xb, const uint4 w0, const uint4 w1, const RoundK& rc,
                                               float norm, float S, const float* lev, int nlev, float* z) {
  constexpr uint32_t kTwo23 = 0x4B000000u;              // pattern of 2^23: its low mantissa bytes are replaced by h
  const float x[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
  const uint32_t hb[8] = {prmt(w0.x, kTwo23, 0x7632u), prmt(w0.y, kTwo23, 0x7632u), prmt(w0.z, kTwo23, 0x7632u), prmt(w0.w, kTwo23, 0x7632u),
                          prmt(w1.x, kTwo23, 0x7632u), prmt(w1.y, kTwo23, 0x7632u), prmt(w1.z, kTwo23, 0x7632u), prmt(w1.w, kTwo23, 0x7632u)};
  float worst = 0.0f;
#pragma unroll
  for (int i = 0; i < 8; ++i) z[i] = round_signed(x[i], hb[i], rc, &worst);
  if (!(worst <= rc.thr)) {                             // some coordinate of the octet needs the exact routine
    const uint64_t fixed = redo_octet(xa, xb, w0, w1, rc, norm, lev, nlev);
#pragma unroll
    for (int i = 0; i < 8; ++i) z[i] = __fmul_rn((float)(int)(signed char)(uint8_t)(fixed >> (8 * i)), S);
  }
}

// the same for octet `oct` (its index in the generator's counter space) of worker k
__device__ __forceinline__ void octet_levels(const float4 xa, const float4 xb, uint64_t oct, uint32_t k, uint32_t xid,
                                             const PhiloxKey& key, const RoundK& rc, float norm, float S,
                                             const float* lev, int nlev, float* z) {
  uint4 w0, w1;
  philox4x32_10_x2(2ull * oct, 2ull * oct + 1ull, k, xid, key, &w0, &w1);
  octet_levels_w(xa, xb, w0, w1, rc, norm, S, lev, nlev, z);
}

// the pair table's entry for two consecutive coordinates, at byte 4 * ((first + 64 * second) mod 4096) of the
// table at shared address `pair`
__device__ __forceinline__ uint32_t pair_entry(uint32_t pair, float z_first, float z_second, float four_over_S) {
  const float t = fmaf(z_second, 64.0f * four_over_S, fmaf(z_first, four_over_S, 12582912.0f));   // 1.5 * 2^23 + 4 first + 256 second
  return lds_table32(pair + (__float_as_uint(t) & 0x3ffcu));
}

// The encoder's shared-memory tables as one block of global memory: built by one CTA when a configuration is first
// used and copied by every encode CTA after that (building them costs a CTA of a small bucket more than the bucket).
struct EncodeTables {
  float4 bin[kBinEntries];
  uint32_t pair[kPairLutSize];
  EncLut lut;
};
static_assert(sizeof(EncodeTables) % 16 == 0, "copied in 16-byte pieces");

__global__ void __launch_bounds__(512) k_build_encode_tables(const __grid_constant__ RoundTable rt, const __grid_constant__ CodeTable ct,
                                                             EncodeTables* out) {
  __shared__ __align__(128) float4 s_bin[kBinEntries];
  __shared__ __align__(16) uint32_t s_pair[kPairLutSize];
  __shared__ EncLut s_lut;
  fill_enc_lut(&s_lut, ct);
  fill_bin_table(s_bin, rt, true);
  __syncthreads();
  fill_pair_lut_signed(s_pair, &s_lut);
  __syncthreads();
  for (int i = threadIdx.x; i < kBinEntries; i += blockDim.x) out->bin[i] = s_bin[i];
  for (int i = threadIdx.x; i < kPairLutSize; i += blockDim.x) out->pair[i] = s_pair[i];
  for (int i = threadIdx.x; i < 2 * QGX_MAX_LEVELS; i += blockDim.x) out->lut.e[i] = s_lut.e[i];
}

// One persistent CTA per SM slot; each ticket is one bucket (k = ticket % K, b = ticket / K).
//   loads, zero the image | barrier | norm, Philox, rounding, packing, sub-block lengths, warp scans |
//   barrier | warp offsets, bit scatter, look-back (warp 0) | barrier | copy out
// The bucket image is double buffered, so the copy-out of one bucket needs no barrier before the next
// bucket starts.  A thread works on P octets; warp w owns the 256 * P coordinates [w * 256 * P, ...).
template <int P, int G>
__global__ void __launch_bounds__(P == 1 ? 256 : 512, P == 1 ? 4 : 2)
k_exchange_encode(const __grid_constant__ EncodeArgs a, const __grid_constant__ LevelTable lt,
                  const __grid_constant__ CodeTable ct, const __grid_constant__ PhiloxKey key,
                  const __grid_constant__ RoundTable rt) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ __align__(128) float4 s_bin[kBinEntries];
  __shared__ EncLut s_lut;
  __shared__ __align__(16) uint32_t s_pair[kPairLutSize];
  __shared__ float s_lev[QGX_MAX_LEVELS];
  __shared__ double s_red[2][32];
  __shared__ uint32_t s_wtot[2][32];
  __shared__ unsigned int s_ticket[2];
  __shared__ unsigned long long s_prefix[2];
  __shared__ int s_skip[2];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  // words of one image, a multiple of 4 so that both images are 16-byte aligned
  const int img_words = (int)((((((uint32_t)a.bucket * (uint32_t)(ct.maxlen + 1) + 16u * (uint32_t)(a.bucket / G + 1) + kNormBits + 31u) >> 5) + 4) + 3u) & ~3u);
  const unsigned long long total = (unsigned long long)(a.nb - a.b_first) * (unsigned long long)a.K;
  constexpr int kOctet = 2 * kQuad;
  constexpr int kSegLanes = G / kOctet;                 // lanes per sub-block within a row of 256 coordinates
  constexpr int kSegs = 32 / kSegLanes;                 // sub-blocks per row

  if (a.tables) {
    const uint4* gb = reinterpret_cast<const uint4*>(a.tables->bin);
    const uint4* gp = reinterpret_cast<const uint4*>(a.tables->pair);
    uint4* sb = reinterpret_cast<uint4*>(s_bin);
    uint4* sp = reinterpret_cast<uint4*>(s_pair);
    for (int i = threadIdx.x; i < kBinEntries; i += blockDim.x) sb[i] = __ldg(gb + i);
    for (int i = threadIdx.x; i < kPairLutSize / 4; i += blockDim.x) sp[i] = __ldg(gp + i);
    for (int i = threadIdx.x; i < 2 * QGX_MAX_LEVELS; i += blockDim.x) s_lut.e[i] = __ldg(a.tables->lut.e + i);
  } else {
    fill_enc_lut(&s_lut, ct);
    fill_bin_table(s_bin, rt, true);
  }
  if (threadIdx.x < QGX_MAX_LEVELS) s_lev[threadIdx.x] = threadIdx.x < lt.nlev ? lt.lev[threadIdx.x] : 1.0f;
  if (threadIdx.x == 0) s_ticket[0] = atomicAdd(a.ticket, 1u);
  for (int i = threadIdx.x; i < 2 * img_words; i += blockDim.x) s_dyn[i] = 0;
  __syncthreads();
  if (!a.tables) fill_pair_lut_signed(s_pair, &s_lut);
  __syncthreads();
  const int nlev = lt.nlev;
  const uint32_t pair_sa = smem_addr(s_pair);
  const float S = -rt.neg_qscale16 * 65536.0f, four_over_S = 4.0f / S;
  uint32_t used_words[2] = {0u, 0u};                    // words of each image that the last bucket in it dirtied

  for (int par = 0;; par ^= 1) {
    const unsigned long long t = s_ticket[par];
    if (t >= total) break;
    const size_t b = a.b_first + (size_t)(t / (unsigned long long)a.K), k = (size_t)(t % (unsigned long long)a.K);
    const size_t lo = b * (size_t)a.bucket;
    const int len = (int)min((size_t)a.bucket, a.d - lo);
    uint32_t* s_img = s_dyn + par * img_words;

    BucketRegs<2 * P> r;
    load_bucket_octets<P>(r, a.src, k, a.d, lo, len, a.vec_ok);
    {
      // this image was last read by the copy-out two buckets ago; two barriers have passed since
      uint4* z = reinterpret_cast<uint4*>(s_img);
      const int n4 = (int)((used_words[par] + 3u + 3u) >> 2);
      for (int i = threadIdx.x; i < n4; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    const float norm = bucket_norm_all<2 * P>(r, a.norm_type, s_red[par]);   // barrier inside: the image is zero
    const bool finite = (norm - norm) == 0.0f;
    const RoundK rc = round_k(rt, norm, s_bin);
    if (threadIdx.x == 0) {
      a.norms[k * a.nb + b] = norm;
      if (!finite) latch_error(a.st, QGX_ERR_NONFINITE);
      s_img[0] = __float_as_uint(norm);
    }
    const uint32_t nsub = (uint32_t)((len + G - 1) / G);
    const uint32_t hdr_bits = kNormBits + 16u * nsub;
    // every lane holds full octets that are octets of the generator's counter space too: no checks
    const bool whole = (len == a.bucket) && a.vec_ok && (a.bucket % (32 * kOctet * P) == 0) && (((a.quad_base + (uint64_t)(lo >> 2)) & 1ull) == 0);
    const bool live = finite && norm != 0.0f;             // otherwise every coordinate is level 0
    const uint64_t oct0 = (a.quad_base + (uint64_t)(lo >> 2)) >> 1;   // the bucket's first octet in the counter space (when `whole`)

    uint64_t qbits[2 * P];
    uint32_t qn[P], qoff[P];                              // qn: bits of the first quad | bits of the second << 8
    if (whole && live) {                                  // the common case, without per-coordinate decisions
#pragma unroll
      for (int j = 0; j < P; ++j) {
        const int o = (warp * P + j) * 32 + lane;
        float z[8];
        octet_levels(r.x[2 * j], r.x[2 * j + 1], oct0 + (uint64_t)o, (uint32_t)k, a.xid, key, rc, norm, S, s_lev, nlev, z);
        const uint32_t e01 = pair_entry(pair_sa, z[0], z[1], four_over_S), e23 = pair_entry(pair_sa, z[2], z[3], four_over_S);
        const uint32_t e45 = pair_entry(pair_sa, z[4], z[5], four_over_S), e67 = pair_entry(pair_sa, z[6], z[7], four_over_S);
        uint32_t n0, n1;
        pack_pair_entries(e01, e23, &qbits[2 * j], &n0);
        pack_pair_entries(e45, e67, &qbits[2 * j + 1], &n1);
        qn[j] = n0 | (n1 << 8);
      }
    } else {
#pragma unroll
      for (int j = 0; j < P; ++j) {
        const int o = (warp * P + j) * 32 + lane;           // octet of the bucket
        const int nv = whole ? kOctet : max(0, min(kOctet, len - o * kOctet));
        uint32_t sy[2] = {0u, 0u};                          // symbol bytes (level | sign << 7) of the two quads
        if (live && nv > 0) {
          const uint64_t e0 = 4ull * (a.quad_base + (uint64_t)(lo >> 2)) + (uint64_t)o * kOctet;   // first coordinate in the counter space
          const float x[8] = {r.x[2 * j].x, r.x[2 * j].y, r.x[2 * j].z, r.x[2 * j].w,
                              r.x[2 * j + 1].x, r.x[2 * j + 1].y, r.x[2 * j + 1].z, r.x[2 * j + 1].w};
          for (int i = 0; i < nv; ++i) {                    // ragged ends and odd offsets: the exact routine throughout
            const uint32_t rb = variate_bits(e0 + (uint64_t)i, (uint32_t)k, a.xid, key);
            const int idx = quantize_level_exact(fabsf(x[i]), norm, s_lev, nlev, rb);
            sy[i >> 2] |= symbol_of(x[i], idx) << (8 * (i & 3));
          }
        }
        uint32_t n0, n1;
        pack_quad(sy[0], min(nv, kQuad), &s_lut, &qbits[2 * j], &n0);
        pack_quad(sy[1], max(nv - kQuad, 0), &s_lut, &qbits[2 * j + 1], &n1);
        qn[j] = n0 | (n1 << 8);
      }
    }
    // warp scans of the bit counts, two rows per 32-bit word (a row holds at most 32 * 104 bits);
    // qoff[j] becomes the octet's bit offset inside the warp's part of the payload
    uint32_t warp_bits = 0;
#pragma unroll
    for (int j = 0; j < P; j += 2) {
      const uint32_t cnt0 = (qn[j] & 0xffu) + (qn[j] >> 8);
      const uint32_t cnt1 = j + 1 < P ? (qn[j + 1 < P ? j + 1 : j] & 0xffu) + (qn[j + 1 < P ? j + 1 : j] >> 8) : 0u;
      const uint32_t both = cnt0 | (cnt1 << 16);
      const uint32_t incl = warp_incl_scan(both, lane);
      const uint32_t before = __shfl_up_sync(0xffffffffu, incl, kSegLanes);
      const uint32_t seg = incl - (lane >= kSegLanes ? before : 0u);   // per field: no borrow, the scans are monotone
      const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (j + h < P) {
          const uint32_t mine = (incl >> (16 * h)) & 0xffffu;
          qoff[j + h < P ? j + h : j] = warp_bits + mine - (h == 0 ? cnt0 : cnt1);
          warp_bits += (tot >> (16 * h)) & 0xffffu;
          // sub-block lengths: the last lane of each sub-block knows its total; the 16-bit fields are
          // halfword aligned, a plain store
          if ((lane + 1) % kSegLanes == 0) {
            const int sb = (warp * P + j + h) * kSegs + lane / kSegLanes;
            if (whole || sb * G < len) reinterpret_cast<uint16_t*>(s_img)[2 + sb] = (uint16_t)((seg >> (16 * h)) & 0xffffu);
          }
        }
      }
    }
    if (lane == 0) s_wtot[par][warp] = warp_bits;
    __syncthreads();
    // where this warp's part starts: exclusive prefix of the warps' totals
    const uint32_t wt = lane < nwarps ? s_wtot[par][lane] : 0u;
    const uint32_t wincl = warp_incl_scan(wt, lane);
    const uint32_t wbase = __shfl_sync(0xffffffffu, wincl - wt, warp);
    const uint32_t payload = __shfl_sync(0xffffffffu, wincl, 31);
    const uint32_t nbits = hdr_bits + payload;
    const uint32_t nwords = (nbits + 31) >> 5;
    used_words[par] = nwords;
    unsigned long long* row = a.status + k * a.nb;
    if (threadIdx.x == 0) {
      st_status(row + b, kStAggregate | (unsigned long long)nwords);
      a.bucket_bits[k * a.nb + b] = nbits;
      atomicAdd(a.total_bits + k, (unsigned long long)nbits);
    }
    const uint32_t base = hdr_bits + wbase;
#pragma unroll
    for (int j = 0; j < P; ++j) put_bits2(s_img, base + qoff[j], qbits[2 * j], qn[j] & 0xffu, qbits[2 * j + 1], qn[j] >> 8);
    if (warp == 0) {
      bool timed_out = false;
      const unsigned long long excl = lookback_prefix(row, (long long)b, lane, a.spin_limit, &timed_out);
      if (lane == 0) {
        st_status(row + b, kStPrefix | (excl + (unsigned long long)nwords));
        int skip = 0;
        if (timed_out) { latch_error(a.st, QGX_ERR_TIMEOUT); skip = 1; }
        if (excl + nwords > (unsigned long long)a.cap_words) { latch_error(a.st, QGX_ERR_CAPACITY); skip = 1; }
        a.offsets[k * a.nb + b] = (uint32_t)min(excl, (unsigned long long)0xffffffffu);
        s_prefix[par] = excl;
        s_skip[par] = skip;
        s_ticket[par ^ 1] = atomicAdd(a.ticket, 1u);
      }
    }
    __syncthreads();
    if (!s_skip[par]) {
      uint32_t* dst = a.stream + k * a.cap_words + s_prefix[par];
      for (uint32_t i = threadIdx.x; i < nwords; i += blockDim.x) dst[i] = s_img[i];
    }
    // no barrier here: the next bucket works in the other image, and this one is next written after
    // two more barriers
  }
}

}  // namespace qgx

#include "qgx_encode_staged.cuh"

namespace qgx {

// ---- decode + average ------------------------------------------------------------------------
// Decoder table of the fused path: index = the next maxlen + 1 stream bits (codeword, then the sign
// bit of a nonzero level); entry = the signed level value and, in `len`, the bits consumed (bits 0..4) and the
// symbol byte (bits 8..15).  Where no codeword starts like the index the value is NaN -- it stays in the running
// sum of its coordinate, where the kernel looks for it -- and one bit is consumed so that the walk goes on.
struct DecEntry {
  float val;
  uint32_t len;
};

struct DecodeArgs {
  const uint32_t* stream;       // [K][cap_words]
  size_t cap_words;
  const uint32_t* bucket_bits;  // [K][nb]
  const uint32_t* offsets;      // [K][nb]
  size_t d;
  int bucket;
  int K;
  size_t nb;
  const DecEntry* lut;          // decoder table in global memory, 1 << (maxlen + 1) entries
  float* mean;                  // [d]
  // optional fused state update (the two axpy of Eq. Q-GenX)
  int update;                   // 0 none, 1: xout = xin - gamma * mean, 2: xout = xin - mean
  const float* xin;
  float* xout;
  const double* scalars;        // scalars[1] = gamma_t
  bool vec_out;                 // d % 4 == 0 and mean, xin, xout 16-byte aligned: 128-bit stores
  // small vectors: a thread decodes its sub-block of ONE worker and stores the values to values[K][d]; the
  // ordered sum over the workers, the division and the state update follow in k_sum_workers
  float* values;                // [K][d] or null
  // large vectors: the walk alone (one worker per thread, VAL = false) writes every worker's symbol bytes to sym_out
  // and the norms it read from the streams to norms_out; k_symbols_mean forms the ordered sums from them
  float* norms_out;             // [K][nb] or null
  // optional: keep the decoded symbols (1 byte per coordinate and worker) ...
  // Symbol bytes are kept transposed, so that a warp's accesses coalesce: worker k, sub-block gs, coordinate i of the
  // sub-block -> byte k * sym_ld + (gs / 32) * 32 * G + (i / 4) * 128 + (gs % 32) * 4 + i % 4.
  uint8_t* sym_out;             // [K][sym_ld] or null
  // ... or compare with the symbols and norms kept by the other exchange of the iteration:
  // *sum_sq += sum_k ||vhat_k of that exchange - vhat_k of this one||^2 (fp32 differences, fp64 sum)
  const uint8_t* sym_prev;      // [K][sym_ld] or null
  size_t sym_ld;
  const float* norms_prev;      // [K][nb]
  double* sum_sq;
  DevStatus* st;
};

constexpr int kDecThreads = 128;
constexpr bool kTwoPassByDefault = false;   // large vectors decode in two passes (walk, then sums) unless told otherwise
constexpr uint32_t kBadSymbol = 0x40u;      // symbol byte of an index that no codeword starts like (no level has bit 6)

// Bits not yet consumed of one sub-block: a 64-bit window refilled 32 bits at a time.  The streams
// of the fused path lie in the context's workspace, which extends past every bucket, so a read a
// few words beyond a (corrupt) sub-block stays inside allocated memory.  SH: the words are read from the warp's
// staged row by shared-memory loads (the address is a 32-bit shared address); otherwise from wherever p points.
template <bool SH>
struct Window {
  using Addr = typename std::conditional<SH, uint32_t, const uint32_t*>::type;
  Addr next;              // address of `ahead`
  Addr first;             // address of the word that held the first bit
  uint32_t lo, hi;
  uint32_t ahead;         // the word after the window, fetched one refill early
  int avail;
  uint32_t sh0;
  static __device__ __forceinline__ uint32_t word(uint32_t a) { return lds32(a); }
  static __device__ __forceinline__ uint32_t word(const uint32_t* a) { return *a; }
  static __device__ __forceinline__ Addr at(const uint32_t* p, std::true_type) { return smem_addr(p); }
  static __device__ __forceinline__ Addr at(const uint32_t* p, std::false_type) { return p; }
  static __device__ __forceinline__ uint32_t step(uint32_t a, int words) { return a + 4u * (uint32_t)words; }
  static __device__ __forceinline__ const uint32_t* step(const uint32_t* a, int words) { return a + words; }
  // p = address of the word that holds the first bit, sh = first bit within it
  __device__ __forceinline__ void open(const uint32_t* p, uint32_t sh) {
    first = at(p, std::integral_constant<bool, SH>());
    const uint32_t w0 = word(first), w1 = word(step(first, 1)), w2 = word(step(first, 2));
    lo = __funnelshift_r(w0, w1, sh);
    hi = w1 >> sh;
    avail = 64 - (int)sh;                               // the window ends on a word boundary
    sh0 = sh;
    ahead = w2;
    next = step(first, 2);
  }
  __device__ __forceinline__ void refill() {            // needs avail <= 32
    const uint32_t w = ahead;
    next = step(next, 1);
    ahead = word(next);                                 // not needed before the next refill
    lo |= __funnelshift_lc(0u, w, (uint32_t)avail);     // w << avail, nothing when avail == 32
    hi |= __funnelshift_lc(w, 0u, (uint32_t)avail);     // the bits of w that do not fit the low word
    avail += 32;
  }
  __device__ __forceinline__ void skip(uint32_t n) {    // n < 32
    lo = __funnelshift_r(lo, hi, n);
    hi >>= n;
    avail -= (int)n;
  }
  static __device__ __forceinline__ uint32_t words_from(uint32_t a, uint32_t b) { return (a - b) >> 2; }
  static __device__ __forceinline__ uint32_t words_from(const uint32_t* a, const uint32_t* b) { return (uint32_t)(a - b); }
  // bits consumed since open(): the words taken in so far, less what is still in the window
  __device__ __forceinline__ uint32_t used() const { return 32u * words_from(next, first) - sh0 - (uint32_t)avail; }
};

// start of sub-block `s` (bits after the header) = sum of the 16-bit lengths before it; all lanes of
// the warp share the bucket and hold consecutive sub-blocks
__device__ __forceinline__ uint32_t header_sum_before_warp(const uint32_t* w, uint32_t warp_first, int lane) {
  uint32_t before = 0;
  for (uint32_t i = (uint32_t)lane; i < warp_first; i += 32) {
    const uint32_t bit = kNormBits + 16u * i;
    before += (w[bit >> 5] >> (bit & 31u)) & 0xffffu;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
  return before;
}

// where sub-block s of bucket (k, b) starts and how long it is; false if the bucket's numbers disagree
__device__ __forceinline__ bool locate_subblock(const uint32_t* stream, size_t cap_words, const uint32_t* bucket_bits,
                                                const uint32_t* offsets, size_t kb, uint32_t hdr_bits, uint32_t s,
                                                bool exists, bool uniform, int lane, const uint32_t** words, float* norm,
                                                uint32_t* start, uint32_t* want, uint32_t* row_before, uint32_t* row_bits) {
  const uint32_t nbits = bucket_bits[kb];
  const uint32_t off = offsets[kb];
  const uint32_t* w = stream + off;
  *words = w;
  const bool ok = nbits >= hdr_bits && (size_t)off + ((nbits + 31) >> 5) <= cap_words;
  uint32_t st = 0, len = 0;
  float nm = 0.0f;
  *row_before = 0;
  *row_bits = 0;
  if (ok) {
    nm = __uint_as_float(w[0]);
    if (uniform) {
      const uint32_t bit = kNormBits + 16u * s;
      len = exists ? ((w[bit >> 5] >> (bit & 31u)) & 0xffffu) : 0u;
      const uint32_t incl = warp_incl_scan(len, lane);
      const uint32_t before = header_sum_before_warp(w, s - (uint32_t)lane, lane);
      st = before + incl - len;
      *row_before = before;
      *row_bits = __shfl_sync(0xffffffffu, incl, 31);
    } else if (exists) {
      for (uint32_t i = 0; i <= s; ++i) {
        const uint32_t bit = kNormBits + 16u * i;
        const uint32_t L = (w[bit >> 5] >> (bit & 31u)) & 0xffffu;
        if (i < s) st += L; else len = L;
      }
    }
  }
  *norm = nm;
  *start = hdr_bits + st;
  *want = len;
  return ok && (!exists || (hdr_bits + st + len <= nbits && nbits < (1u << 18) && len < (1u << 14)));
}

// One thread per sub-block, workers in the outer loop: the thread keeps all G running sums of its
// sub-block in registers (fixed k order, so the mean is bit-identical to a sequential sum) and reads each
// worker's sub-block once, front to back, so that every fetched sector is used up at once.  The next
// worker's sub-block is located while the current one is decoded.
struct SubBlockAt {
  const uint32_t* p;      // word that holds the first bit: in the warp's staged row (shared memory) or in the stream
  uint32_t sh;            // first bit within that word
  uint32_t want;          // bits of the sub-block
  float norm;
  float norm_prev;        // norm of the same bucket in the other exchange (when comparing)
  bool ok;
  bool staged;            // p points into the warp's staged row
};

// Words that a thread may read past the first word of its sub-block: G symbols of at most 13 bits, the
// partial first word and the two words fetched ahead.
template <int G>
struct DecodeReach { static constexpr int kWords = (G * 13) / 32 + 4; };

// Locates sub-block s of bucket (k, b) and starts the asynchronous copy of the warp's row -- the stream words
// of its 32 consecutive sub-blocks plus what a thread may read past them -- into `row` (shared memory, row_words
// words).  A thread whose reads would leave the staged words reads the stream itself.  The copies belong to the
// caller's next commit group.
template <int G>
__device__ __forceinline__ SubBlockAt find_subblock(const DecodeArgs& a, int k, size_t b, uint32_t hdr_bits, uint32_t s,
                                                    bool exists, bool uniform, int lane, uint32_t* row, int row_words) {
  SubBlockAt r;
  const uint32_t* w;
  uint32_t st, row_before, row_bits;
  r.ok = locate_subblock(a.stream + (size_t)k * a.cap_words, a.cap_words, a.bucket_bits, a.offsets, (size_t)k * a.nb + b,
                         hdr_bits, s, exists, uniform, lane, &w, &r.norm, &st, &r.want, &row_before, &row_bits);
  // a bucket whose numbers disagree is reported, and its walk reads the start of the worker's stream instead
  // (in range whatever the offsets say)
  if (!r.ok) { st = 0; r.want = 0; r.norm = 0.0f; w = a.stream + (size_t)k * a.cap_words; }
  r.p = w + (st >> 5);
  r.sh = st & 31u;
  // bucket-level validity is the same for all lanes; the lengths are bounded, so the row is at most 2^19 bits
  const bool stage = uniform && __all_sync(0xffffffffu, r.ok) && row_bits < (1u << 19);
  r.staged = false;
  if (stage) {
    const size_t first = (size_t)(w - a.stream) + ((hdr_bits + row_before) >> 5);       // word index in the whole buffer
    const size_t first_al = first & ~(size_t)3;                                          // 16-byte aligned
    const size_t last = (size_t)(w - a.stream) + ((hdr_bits + row_before + row_bits + 31u) >> 5) + DecodeReach<G>::kWords;
    const int nwords = (int)min((size_t)row_words, ((last - first_al) + 3) & ~(size_t)3);   // the buffer ends 64 words after the streams
    for (int c = lane; c < nwords / 4; c += 32) {
      const unsigned sa = (unsigned)__cvta_generic_to_shared(row + 4 * c);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(a.stream + first_al + 4 * (size_t)c) : "memory");
    }
    const size_t mine = (size_t)(r.p - a.stream) - first_al;
    if (mine + DecodeReach<G>::kWords <= (size_t)nwords) { r.p = row + mine; r.staged = true; }
  }
  r.norm_prev = a.norms_prev ? a.norms_prev[(size_t)k * a.nb + b] : 0.0f;
  return r;
}

// Copies one row of kept symbol words (kWords words, contiguous, 16-byte aligned) into shared memory without
// waiting; the copies belong to the caller's next commit group.
template <int kWords>
__device__ __forceinline__ void stage_symbol_row(uint32_t* dst, const uint8_t* src, int lane) {
#pragma unroll
  for (int c = lane; c < kWords / 4; c += 32) {
    const unsigned sa = (unsigned)__cvta_generic_to_shared(dst + 4 * c);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(src + 16 * (size_t)c) : "memory");
  }
}

// shared memory of the decode kernel after its table: per warp two stream rows and (when comparing) two symbol rows --
// one of each when a thread walks a single worker and nothing is fetched a worker ahead (VAL = false)
template <int G, int SYM, bool VAL>
struct DecodeSmem {
  static constexpr int kStreamRow = 9 * G + 64;         // words, a multiple of 4
  static constexpr int kBufs = VAL ? 2 : 1;
  static constexpr size_t kBytes = sizeof(uint32_t) * kBufs * (128 / 32) * (size_t)(kStreamRow + ((SYM & 2) ? G * 8 : 0));
};

// SYM, a set of bits: 1 keeps the decoded symbols; 2 adds the squared differences between the vectors kept by an
// earlier exchange (whose level table is `lt`) and the ones decoded now to *sum_sq; 4 adds the squared decoded values
// themselves (an earlier vector of zero).  1 | 2 compares first and then overwrites the kept symbols in place.
// VAL = false: the walk alone, one worker per thread -- no running sums, so half the registers and twice the warps;
// symbols always go to a.sym_out, the norms read from the streams to a.norms_out.
template <int G, int SYM, bool VAL>
__global__ void __launch_bounds__(kDecThreads, VAL ? (G == 128 ? 3 : (G == 64 ? 4 : 6)) : 10) k_exchange_decode(const __grid_constant__ DecodeArgs a,
                                                                      const __grid_constant__ CodeTable ct,
                                                                      const __grid_constant__ LevelTable lt) {
  constexpr bool kStore = (SYM & 1) != 0 || !VAL, kCompare = VAL && (SYM & 2) != 0, kSquare = VAL && (SYM & 4) != 0;
  constexpr int kBufs = DecodeSmem<G, SYM, VAL>::kBufs;
  extern __shared__ __align__(16) unsigned char s_raw[];
  __shared__ float s_lev[QGX_MAX_LEVELS];            // the table of the kept symbols (comparing)
  // comparing: the kept symbol words of the warp's 32 sub-blocks, one worker ahead (asynchronous copies)
  constexpr int kRowWords = G * 8;                      // 32 sub-blocks x G bytes
  // the stream words of the warp's 32 sub-blocks, one worker ahead (asynchronous copies): room for 8 bits per
  // symbol and sign on average; longer rows are partly read from the stream itself
  constexpr int kStreamRow = DecodeSmem<G, SYM, VAL>::kStreamRow;
  const int lut_n = 2 << ct.maxlen;
  // dynamic shared memory: table, stream rows, symbol rows.  The walk alone needs only the entries' second word
  // (bits consumed, symbol byte).
  DecEntry* s_lut = reinterpret_cast<DecEntry*>(s_raw);
  uint32_t* s_len = reinterpret_cast<uint32_t*>(s_raw);
  uint32_t* s_rows = reinterpret_cast<uint32_t*>(s_raw + (VAL ? sizeof(DecEntry) : sizeof(uint32_t)) * (size_t)lut_n);
  uint32_t* s_prev = s_rows + kBufs * (kDecThreads / 32) * kStreamRow;
  {
    const uint2* src = reinterpret_cast<const uint2*>(a.lut);
    uint2* dst = reinterpret_cast<uint2*>(s_lut);
    for (int i = threadIdx.x; i < lut_n; i += blockDim.x) {
      if constexpr (VAL) dst[i] = src[i];
      else s_len[i] = src[i].y;
    }
  }
  if (threadIdx.x < QGX_MAX_LEVELS) s_lev[threadIdx.x] = threadIdx.x < lt.nlev ? lt.lev[threadIdx.x] : 0.0f;
  __syncthreads();
  const uint32_t mask = (uint32_t)lut_n - 1u;
  const int lane = threadIdx.x & 31, tid = threadIdx.x;
  const size_t spb = (size_t)a.bucket / G;
  const size_t total_sub = a.nb * spb;
  const bool uniform = (spb % 32 == 0);
  const float Kf = (float)a.K;
  // the mean is sum / K, one fp32 division; for K a power of two the product with 1 / K is the same number
  const bool k_pow2 = (a.K & (a.K - 1)) == 0;
  const float Kinv = 1.0f / Kf;
  bool bad = false;
  double sq = 0.0;

  const bool wide = !VAL || a.values != nullptr;
  const size_t sub_pad = (total_sub + 31) & ~(size_t)31;                // whole warps per worker
  const size_t items = wide ? sub_pad * (size_t)a.K : total_sub;
  for (size_t item = (size_t)blockIdx.x * blockDim.x + tid; item - lane < items; item += (size_t)gridDim.x * blockDim.x) {
    const size_t gs = wide ? item % sub_pad : item;                      // the sub-block
    const int kbeg = wide ? (int)(item / sub_pad) : 0, kend = wide ? kbeg + 1 : a.K;
    const bool live = gs < total_sub;
    const size_t b = live ? gs / spb : a.nb - 1;
    const uint32_t s = live ? (uint32_t)(gs % spb) : 0u;
    const size_t lo = b * (size_t)a.bucket;
    const int len = (int)min((size_t)a.bucket, a.d - lo);
    const int first = (int)s * G;
    const int count = live ? max(0, min(G, len - first)) : 0;
    const uint32_t nsub = (uint32_t)((len + G - 1) / G);
    const uint32_t hdr_bits = kNormBits + 16u * nsub;
    if (!__any_sync(0xffffffffu, count > 0)) continue;   // beyond the end of a short last bucket
    const size_t e0 = lo + (size_t)first;
    const size_t sbase = (gs >> 5) * (size_t)(32 * G) + (size_t)(gs & 31) * 4;   // see DecodeArgs::sym_out

    float acc[VAL ? G : 1];
#pragma unroll
    for (int i = 0; i < (VAL ? G : 1); ++i) acc[i] = 0.0f;
    uint32_t* my_rows = s_prev + (kCompare ? (tid >> 5) * kBufs * kRowWords : 0);
    uint32_t* my_stream = s_rows + (tid >> 5) * kBufs * kStreamRow;
    __syncwarp();                                         // the previous sub-block's rows are no longer read
    SubBlockAt nxt = find_subblock<G>(a, kbeg, b, hdr_bits, s, count > 0, uniform, lane, my_stream + (kbeg & (kBufs - 1)) * kStreamRow, kStreamRow);
    if (kCompare)
      stage_symbol_row<kRowWords>(my_rows + (kbeg & (kBufs - 1)) * kRowWords, a.sym_prev + (size_t)kbeg * a.sym_ld + (gs >> 5) * (size_t)(32 * G), lane);
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int k = kbeg; k < kend; ++k) {
      const SubBlockAt cur = nxt;
      const uint32_t* prev_row = my_rows + (k & (kBufs - 1)) * kRowWords + lane;
      __syncwarp();                                       // every lane is done with the rows that are overwritten next
      if (k + 1 < kend) {
        nxt = find_subblock<G>(a, k + 1, b, hdr_bits, s, count > 0, uniform, lane, my_stream + ((k + 1) & (kBufs - 1)) * kStreamRow, kStreamRow);
        if (kCompare)
          stage_symbol_row<kRowWords>(my_rows + ((k + 1) & (kBufs - 1)) * kRowWords,
                                      a.sym_prev + (size_t)(k + 1) * a.sym_ld + (gs >> 5) * (size_t)(32 * G), lane);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");       // one group per worker, empty after the last
      asm volatile("cp.async.wait_group 1;" ::: "memory");       // worker k's rows have landed
      __syncwarp();
      bad = bad || !cur.ok;
      uint32_t used = 0;
      // the walk over the sub-block's symbols, with the window's words read from the staged row (every lane's
      // words are there) or from wherever they are
      auto walk = [&](auto shared_tag) {
        Window<decltype(shared_tag)::value> win;
        win.open(cur.p, cur.sh);
        if (count == G) {
          uint32_t pack = 0, prev4 = 0;
#pragma unroll
          for (int i = 0; i < G; ++i) {
            if ((i & 1) == 0) {                              // two symbols use at most 26 bits
              if (win.avail <= 32) win.refill();
            }
            if (kCompare && (i & 3) == 0) prev4 = prev_row[(i >> 2) * 32];
            DecEntry e;
            if constexpr (VAL) e = s_lut[win.lo & mask];
            else { e.len = s_len[win.lo & mask]; e.val = 0.0f; }
            win.skip(e.len & 31u);
            const float val = __fmul_rn(cur.norm, e.val);
            if constexpr (VAL) acc[i] = __fadd_rn(acc[i], val);
            if (kCompare) {
              const float dlt = __fsub_rn(dequantize_symbol((prev4 >> (8 * (i & 3))) & 0xffu, cur.norm_prev, s_lev), val);
              sq = fma((double)dlt, (double)dlt, sq);
            }
            if (kSquare) sq = fma((double)val, (double)val, sq);
            if (kStore) {
              // byte 1 of e.len, the symbol byte, becomes byte i % 4 of the word
              pack = prmt(pack, e.len, (i & 3) == 0 ? 0x3215u : ((i & 3) == 1 ? 0x3250u : ((i & 3) == 2 ? 0x3510u : 0x5210u)));
              if ((i & 3) == 3) *reinterpret_cast<uint32_t*>(a.sym_out + (size_t)k * a.sym_ld + sbase + (i >> 2) * 128) = pack;
            }
          }
        } else {
#pragma unroll
          for (int i = 0; i < G; ++i) {
            if ((i & 1) == 0) {
              if (win.avail <= 32) win.refill();
            }
            if (i < count) {
              DecEntry e;
              if constexpr (VAL) e = s_lut[win.lo & mask];
              else { e.len = s_len[win.lo & mask]; e.val = 0.0f; }
              win.skip(e.len & 31u);
              const float val = __fmul_rn(cur.norm, e.val);
              if constexpr (VAL) acc[i] = __fadd_rn(acc[i], val);
              if (kCompare) {
                const float dlt = __fsub_rn(dequantize_symbol(a.sym_prev[(size_t)k * a.sym_ld + sbase + (i >> 2) * 128 + (i & 3)], cur.norm_prev, s_lev), val);
                sq = fma((double)dlt, (double)dlt, sq);
              }
              if (kSquare) sq = fma((double)val, (double)val, sq);
              if (kStore) a.sym_out[(size_t)k * a.sym_ld + sbase + (i >> 2) * 128 + (i & 3)] = (uint8_t)((e.len >> 8) & 0xffu);
            }
          }
        }
        used = win.used();
      };
      if (__all_sync(0xffffffffu, cur.staged)) walk(std::true_type());
      else walk(std::false_type());
      bad = bad || (count > 0 && used != cur.want);          // every sub-block uses exactly its length
    }
    if (count <= 0) continue;
    if constexpr (!VAL) {
      if (s == 0) a.norms_out[(size_t)kbeg * a.nb + b] = nxt.norm;       // the bucket's norm as the stream gives it
    } else {
    {
      // an index that no codeword starts like left a NaN in its coordinate's sum (as a norm that is not finite does)
      bool marked = false;
#pragma unroll
      for (int i = 0; i < G; ++i) marked = marked || (acc[i] != acc[i]);
      bad = bad || marked;
    }
    if (wide) {                                         // the worker's values; summed by k_sum_workers
      float* out = a.values + (size_t)kbeg * a.d + e0;
      if (count == G && a.vec_out) {
#pragma unroll
        for (int i = 0; i < G; i += 4) *reinterpret_cast<float4*>(out + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < G; ++i)
          if (i < count) out[i] = acc[i];
      }
      continue;
    }

    float gam = 1.0f;
    if (a.update == 1) gam = (float)a.scalars[1];
    if (count == G && a.vec_out) {
      auto emit = [&](auto pow2_tag) {
        auto mean_of = [&](float sum) { return decltype(pow2_tag)::value ? __fmul_rn(sum, Kinv) : __fdiv_rn(sum, Kf); };
#pragma unroll
        for (int i = 0; i < G; i += 4) {
          const float4 m = make_float4(mean_of(acc[i]), mean_of(acc[i + 1]), mean_of(acc[i + 2]), mean_of(acc[i + 3]));
          *reinterpret_cast<float4*>(a.mean + e0 + i) = m;
          if (a.update != 0) {
            const float4 x = *reinterpret_cast<const float4*>(a.xin + e0 + i);
            const float g = a.update == 1 ? gam : 1.0f;      // update 2 subtracts the mean itself (1 * m is exact)
            *reinterpret_cast<float4*>(a.xout + e0 + i) =
                make_float4(__fsub_rn(x.x, __fmul_rn(g, m.x)), __fsub_rn(x.y, __fmul_rn(g, m.y)),
                            __fsub_rn(x.z, __fmul_rn(g, m.z)), __fsub_rn(x.w, __fmul_rn(g, m.w)));
          }
        }
      };
      if (k_pow2) emit(std::true_type());
      else emit(std::false_type());
    } else {
#pragma unroll
      for (int i = 0; i < G; ++i) {
        if (i < count) {
          const float m = __fdiv_rn(acc[i], Kf);
          a.mean[e0 + i] = m;
          if (a.update == 1) a.xout[e0 + i] = __fsub_rn(a.xin[e0 + i], __fmul_rn(gam, m));
          if (a.update == 2) a.xout[e0 + i] = __fsub_rn(a.xin[e0 + i], m);
        }
      }
    }
    }   // VAL
  }
  if (kCompare || kSquare) {
    sq = warp_sum(sq);
    if (lane == 0 && sq != 0.0) atomicAdd(a.sum_sq, sq);
  }
  if (bad) latch_error(a.st, QGX_ERR_CORRUPT);
}

// The ordered sums of the two-pass decode: worker k's quantized coordinate is norm_k * (signed level of its symbol
// byte), added in the order k = 0..K-1, divided by K, and the state update applied -- the same operations in the same
// order as the one-pass kernel's.  A thread takes 16 consecutive coordinates of one sub-block (four symbol words per
// worker; the transposed layout makes a warp's loads of one word index contiguous).  The signed level values sit in
// shared memory once per lane (bank = lane), NaN for bytes that are no symbol: a NaN mean reports the stream.
// SYM & 2: also adds sum_k ||vhat_k kept by the other exchange - vhat_k of this one||^2 to *sum_sq (fp32 differences,
// fp64 sum; the kept symbols dequantized with their own table and norms); SYM & 4: sum_k ||vhat_k||^2 instead.
struct MeanArgs {
  const uint8_t* sym;           // [K][sym_ld], this exchange's symbol bytes (transposed layout of DecodeArgs::sym_out)
  size_t sym_ld;
  const float* norms;           // [K][nb], as the walk read them from the streams
  const uint8_t* sym_prev;      // [K][sym_ld] or null
  const float* norms_prev;      // [K][nb]
  double* sum_sq;
  int K;
  size_t d;
  int bucket;
  size_t nb;
  float* mean;
  int update;
  const float* xin;
  float* xout;
  const double* scalars;
  bool vec_out;
  DevStatus* st;
};

template <int G, int SYM>
__global__ void __launch_bounds__(256) k_symbols_mean(const __grid_constant__ MeanArgs a, const __grid_constant__ LevelTable lt,
                                                      const __grid_constant__ LevelTable lt_kept) {
  constexpr bool kCompare = (SYM & 2) != 0, kSquare = (SYM & 4) != 0;
  extern __shared__ __align__(16) float s_val[];                       // [256][32], then (comparing) the kept table [256]
  for (int t = threadIdx.x; t < 256 * 32; t += blockDim.x) {
    const int byte = t >> 5, idx = byte & 31;
    const bool symbol = (byte & 0x60) == 0 && idx < lt.nlev && byte != 0x80;
    s_val[t] = symbol ? ((byte & 0x80) ? -lt.lev[idx] : lt.lev[idx]) : __int_as_float(0x7fc00000);
  }
  if (kCompare) {
    for (int t = threadIdx.x; t < 256; t += blockDim.x) {
      const int idx = t & 31;
      s_val[256 * 32 + t] = idx < lt_kept.nlev ? ((t & 0x80) ? -lt_kept.lev[idx] : lt_kept.lev[idx]) : 0.0f;
    }
  }
  __syncthreads();
  constexpr int kParts = G / 16;                                       // threads per sub-block
  const uint32_t val_sa = smem_addr(s_val) + 4u * (threadIdx.x & 31u);
  const uint32_t kept_sa = smem_addr(s_val + 256 * 32);
  const size_t spb = (size_t)a.bucket / G, total_sub = a.nb * spb, rows = (total_sub + 31) / 32;
  const int K = a.K;
  const float Kf = (float)K, Kinv = 1.0f / Kf;
  const bool k_pow2 = (K & (K - 1)) == 0;
  const int lane = threadIdx.x & 31;
  float gam = 1.0f;
  if (a.update == 1) gam = (float)a.scalars[1];
  bool bad = false;
  double sq = 0.0;
  const size_t ldw = a.sym_ld / 4;
  const size_t items = rows * kParts * 32;
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < items; t += (size_t)gridDim.x * blockDim.x) {
    const size_t rest = t >> 5, row = rest / kParts;
    const int part = (int)(rest % kParts);
    const size_t gs = row * 32 + (size_t)lane;
    if (gs >= total_sub) continue;
    const size_t b = gs / spb, lo = b * (size_t)a.bucket;
    const int len = (int)min((size_t)a.bucket, a.d - lo);
    const int first = (int)(gs % spb) * G + 16 * part;                 // of this thread's coordinates, within the bucket
    const int count = max(0, min(16, len - first));
    if (count == 0) continue;
    const size_t word0 = row * (size_t)(8 * G) + (size_t)(4 * part) * 32 + lane;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(a.sym) + word0;
    const uint32_t* kept = kCompare ? reinterpret_cast<const uint32_t*>(a.sym_prev) + word0 : nullptr;
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.0f;
    auto add = [&](const uint32_t (&w)[4], const uint32_t (&p)[4], float norm, float norm_kept) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t byte = prmt(w[j], 0u, 0x4440u + (uint32_t)q);                 // byte q of the word
          const float val = __fmul_rn(norm, __uint_as_float(lds_table32(val_sa + (byte << 7))));
          acc[4 * j + q] = __fadd_rn(acc[4 * j + q], val);
          if (kCompare) {
            const uint32_t pbyte = prmt(p[j], 0u, 0x4440u + (uint32_t)q);
            const float was = __fmul_rn(norm_kept, __uint_as_float(lds_table32(kept_sa + (pbyte << 2))));
            const float dlt = __fsub_rn(was, val);
            if (4 * j + q < count) sq = fma((double)dlt, (double)dlt, sq);
          }
          if (kSquare) { if (4 * j + q < count) sq = fma((double)val, (double)val, sq); }
        }
      }
    };
    // one worker's words and norms are asked for while the one before is added (k = K asks for nothing)
    uint32_t w[4] = {0u, 0u, 0u, 0u}, p[4] = {0u, 0u, 0u, 0u};
    float nrm = 0.0f, nrm_kept = 0.0f;
    auto fetch = [&](int k, uint32_t (&fw)[4], uint32_t (&fp)[4], float* fn, float* fk) {
      if (k >= K) return;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        fw[j] = __ldcs(words + (size_t)k * ldw + j * 32);
        if (kCompare) fp[j] = __ldcs(kept + (size_t)k * ldw + j * 32);
      }
      *fn = a.norms[(size_t)k * a.nb + b];
      if (kCompare) *fk = a.norms_prev[(size_t)k * a.nb + b];
    };
    fetch(0, w, p, &nrm, &nrm_kept);
    for (int k = 0; k < K; k += 2) {
      uint32_t w1[4] = {0u, 0u, 0u, 0u}, p1[4] = {0u, 0u, 0u, 0u};
      float n1 = 0.0f, m1 = 0.0f;
      fetch(k + 1, w1, p1, &n1, &m1);
      add(w, p, nrm, nrm_kept);
      fetch(k + 2, w, p, &nrm, &nrm_kept);
      if (k + 1 < K) add(w1, p1, n1, m1);
    }
    const size_t e0 = lo + (size_t)first;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float m[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        m[q] = k_pow2 ? __fmul_rn(acc[4 * j + q], Kinv) : __fdiv_rn(acc[4 * j + q], Kf);
        bad = bad || (4 * j + q < count && m[q] != m[q]);
      }
      if (4 * j + 4 <= count && a.vec_out) {
        *reinterpret_cast<float4*>(a.mean + e0 + 4 * j) = make_float4(m[0], m[1], m[2], m[3]);
        if (a.update != 0) {
          const float4 x = *reinterpret_cast<const float4*>(a.xin + e0 + 4 * j);
          const float g = a.update == 1 ? gam : 1.0f;      // update 2 subtracts the mean itself (1 * m is exact)
          *reinterpret_cast<float4*>(a.xout + e0 + 4 * j) =
              make_float4(__fsub_rn(x.x, __fmul_rn(g, m[0])), __fsub_rn(x.y, __fmul_rn(g, m[1])),
                          __fsub_rn(x.z, __fmul_rn(g, m[2])), __fsub_rn(x.w, __fmul_rn(g, m[3])));
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (4 * j + q < count) {
            a.mean[e0 + 4 * j + q] = m[q];
            if (a.update == 1) a.xout[e0 + 4 * j + q] = __fsub_rn(a.xin[e0 + 4 * j + q], __fmul_rn(gam, m[q]));
            if (a.update == 2) a.xout[e0 + 4 * j + q] = __fsub_rn(a.xin[e0 + 4 * j + q], m[q]);
          }
        }
      }
    }
  }
  if (kCompare || kSquare) {
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0 && sq != 0.0) atomicAdd(a.sum_sq, sq);
  }
  if (bad) latch_error(a.st, QGX_ERR_CORRUPT);
}

}  // namespace qgx

// ---- host side ---------------------------------------------------------------------------------
namespace qgx {

// workspace slots of a context
enum { WS_OFF64 = 0, WS_FLAGS = 1, WS_LUT = 2, WS_SLOT0 = 3 /* stream, bits, offsets, total: 3..6 and 7..10 */,
       WS_NORMS = 12, WS_SYM = 13, WS_NORMS2 = 14, WS_OPVAL = 15, WS_MEAN = 16, WS_DLUT = 18, WS_SEGBITS = 19, WS_VALUES = 20, WS_SYMTMP = 21, WS_NORMSDEC = 22 };

// Small vectors, second part: mean_i = (((0 + v_{0,i}) + v_{1,i}) + ...) / K in worker order (the same sequential
// sum as in the fused decode pass), then the optional state update.
__global__ void __launch_bounds__(256) k_sum_workers(const float* __restrict__ values, int K, size_t d, float* __restrict__ mean,
                                                     int update, const float* xin, float* xout, const double* scalars) {
  const float Kf = (float)K;
  const float gam = update == 1 ? (float)scalars[1] : 1.0f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (size_t)gridDim.x * blockDim.x) {
    float acc = 0.0f;
    for (int k = 0; k < K; ++k) acc = __fadd_rn(acc, values[(size_t)k * d + i]);
    const float m = __fdiv_rn(acc, Kf);
    mean[i] = m;
    if (update == 1) xout[i] = __fsub_rn(xin[i], __fmul_rn(gam, m));
    if (update == 2) xout[i] = __fsub_rn(xin[i], m);
  }
}

qgx_status launch_decode_average(qgx_ctx* c, const DecodeArgs& args, const CodeTable& ct, const LevelTable& lt, int sym_mode,
                                 bool walk_only = false);

// ---- what a call derives from a quantizer configuration, kept between calls --------------------
// Building the rounding table, the code table and the decoder table and copying the latter to the device costs
// more host time than a small exchange; iterations reuse a handful of configurations, so the results are kept,
// keyed by the configuration's contents (compared in full on a hit).
struct CachedTables {
  bool valid;
  int nlev, bucket;
  float levels[QGX_MAX_LEVELS];
  qgx_codebook cb;
  CodeTable ct;
  RoundTable rt;
  DecEntry* lut_dev;                    // 2 * kDecLutMax entries, owned
  EncodeTables* enc_dev;                // owned; built by k_build_encode_tables
};
constexpr int kTableCacheSlots = 32;
struct LaunchShape { size_t smem; int per_sm; };      // smem == 0: not asked yet
struct TableCache {
  CachedTables e[kTableCacheSlots];
  LaunchShape enc[3][3];                // [octets per thread 1, 2, 4][sub-block 32, 64, 128]
  LaunchShape enc_staged[3];            // [sub-block]
  LaunchShape dec[3][6];                // [sub-block][symbol mode]
  LaunchShape dec_walk[3][6];           // the walk alone
};

// Lets a kernel use all the dynamic shared memory that the device allows, once per kernel and device.  (The
// attribute belongs to the function, not to a context: a per-context "largest size asked so far" would be undone
// by another context asking for less.)
template <typename Kernel>
static void allow_max_dynamic_smem(Kernel kernel, int device) {
  struct Seen { const void* fn; int device; };
  static Seen seen[256];                                // all template instances of a kernel share this function
  static int nseen = 0;
  static std::mutex guard;                              // contexts may be driven from different host threads
  std::lock_guard<std::mutex> lock(guard);
  const void* fn = reinterpret_cast<const void*>(kernel);
  for (int i = 0; i < nseen; ++i)
    if (seen[i].fn == fn && seen[i].device == device) return;
  int optin = 0;
  cudaFuncAttributes fa;
  if (cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) == cudaSuccess &&
      cudaFuncGetAttributes(&fa, kernel) == cudaSuccess && optin > (int)fa.sharedSizeBytes)
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);
  else
    cudaGetLastError();
  if (nseen < 256) { seen[nseen].fn = fn; seen[nseen].device = device; ++nseen; }
}

void free_table_cache(qgx_ctx* c) {
  TableCache* tc = (TableCache*)c->table_cache;
  if (!tc) return;
  for (int i = 0; i < kTableCacheSlots; ++i) {
    if (tc->e[i].lut_dev) cudaFree(tc->e[i].lut_dev);
    if (tc->e[i].enc_dev) cudaFree(tc->e[i].enc_dev);
  }
  delete tc;
  c->table_cache = nullptr;
}

static TableCache* table_cache(qgx_ctx* c) {
  if (!c->table_cache) c->table_cache = new (std::nothrow) TableCache();   // value-initialized: all zero
  return (TableCache*)c->table_cache;
}

// tables of cfg (built, and the decoder table copied to the device, on a miss)
static qgx_status cached_tables(qgx_ctx* c, const qgx_quant_cfg* cfg, const CachedTables** out) {
  TableCache* tc = table_cache(c);
  if (!tc) return QGX_ERR_CUDA;
  uint64_t h = 1469598103934665603ull;
  auto mix = [&](const void* p, size_t n) {
    const unsigned char* b = (const unsigned char*)p;
    for (size_t i = 0; i < n; ++i) { h ^= b[i]; h *= 1099511628211ull; }
  };
  mix(&cfg->nlev, sizeof(int)); mix(&cfg->bucket, sizeof(int)); mix(cfg->levels, sizeof(float) * (size_t)cfg->nlev);
  mix(&cfg->cb.subblock, sizeof(int)); mix(cfg->cb.len, (size_t)cfg->nlev); mix(cfg->cb.code, sizeof(uint32_t) * (size_t)cfg->nlev);
  CachedTables* e = &tc->e[h % kTableCacheSlots];
  const bool hit = e->valid && e->nlev == cfg->nlev && e->bucket == cfg->bucket && e->cb.nlev == cfg->cb.nlev &&
                   e->cb.subblock == cfg->cb.subblock &&
                   std::memcmp(e->levels, cfg->levels, sizeof(float) * (size_t)cfg->nlev) == 0 &&
                   std::memcmp(e->cb.len, cfg->cb.len, (size_t)cfg->nlev) == 0 &&
                   std::memcmp(e->cb.code, cfg->cb.code, sizeof(uint32_t) * (size_t)cfg->nlev) == 0;
  if (!hit) {
    e->valid = false;
    qgx_status rc = make_code_table(&cfg->cb, cfg->bucket, &e->ct);
    if (rc != QGX_OK) return rc;
    make_round_table(cfg->levels, cfg->nlev, &e->rt);
    if (!e->lut_dev && cudaMalloc((void**)&e->lut_dev, sizeof(DecEntry) * (size_t)(2 * kDecLutMax)) != cudaSuccess) {
      cudaGetLastError();
      e->lut_dev = nullptr;
      return QGX_ERR_CUDA;
    }
    // decoder table: the next maxlen + 1 bits -> signed level value and bits consumed
    const CodeTable& ct = e->ct;
    std::vector<uint16_t> by_code((size_t)1 << ct.maxlen);
    build_dec_lut_host(ct, by_code.data());
    std::vector<DecEntry> h_lut((size_t)2 << ct.maxlen);
    for (size_t i = 0; i < h_lut.size(); ++i) {
      const uint16_t w = by_code[i & (((size_t)1 << ct.maxlen) - 1)];
      const uint32_t L = w >> 8, idx = w & 0xffu;
      if (L == 0) { h_lut[i].val = std::numeric_limits<float>::quiet_NaN(); h_lut[i].len = 1u | (kBadSymbol << 8); continue; }   // no codeword starts like this
      if (idx == 0) { h_lut[i].val = 0.0f; h_lut[i].len = L; continue; }       // symbol byte 0
      const bool neg = (i >> L) & 1u;
      h_lut[i].val = neg ? -cfg->levels[idx] : cfg->levels[idx];
      h_lut[i].len = (L + 1u) | ((idx | (neg ? 0x80u : 0u)) << 8);       // bits 8..15: the symbol byte
    }
    // stream-ordered after the kernels that still read this slot's previous table; the source is pageable, so
    // the call returns once it has been staged
    if (cudaMemcpyAsync(e->lut_dev, h_lut.data(), h_lut.size() * sizeof(DecEntry), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
      return QGX_ERR_CUDA;
    // the encoder's tables, built on the device by the routines that the kernels would run themselves
    if (!e->enc_dev && cudaMalloc((void**)&e->enc_dev, sizeof(EncodeTables)) != cudaSuccess) {
      cudaGetLastError();
      e->enc_dev = nullptr;
      return QGX_ERR_CUDA;
    }
    k_build_encode_tables<<<1, 512, 0, c->stream>>>(e->rt, e->ct, e->enc_dev);
    count_launch(c);
    if (cudaGetLastError() != cudaSuccess) return QGX_ERR_CUDA;
    e->nlev = cfg->nlev;
    e->bucket = cfg->bucket;
    std::memcpy(e->levels, cfg->levels, sizeof(e->levels));
    e->cb = cfg->cb;
    e->valid = true;
  }
  *out = e;
  return QGX_OK;
}

// Tensor map of `rows` rows of 32 floats (128 bytes) starting at base, copied `box_rows` rows at a time with the
// 128-byte swizzle: what k_encode_staged's bulk copies read.  The encoder of the map is a driver entry point,
// looked up once (the library does not link the driver).
static bool make_rows_map(const float* base, unsigned long long rows, unsigned box_rows, CUtensorMap* out) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_fn encode = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      encode = reinterpret_cast<encode_fn>(fn);
    else
      cudaGetLastError();
  });
  if (!encode || rows == 0) return false;
  const cuuint64_t gdim[2] = {(cuuint64_t)kLaneCoords, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)(kLaneCoords * sizeof(float))};
  const cuuint32_t box[2] = {(cuuint32_t)kLaneCoords, (cuuint32_t)box_rows};
  const cuuint32_t estride[2] = {1u, 1u};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), gdim, gstride, box, estride,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The whole exchange.  sym_mode 1 keeps the decoded symbols (and the norms) in the workspace; sym_mode 2
// adds sum_k ||vhat_k kept by the other slot - vhat_k decoded in this exchange||^2 to *sum_sq.
qgx_status exchange_impl(qgx_ctx* c, DualSource src, int K, size_t d, const qgx_quant_cfg* cfg, uint32_t xid, int slot,
                         float* mean_out, uint64_t* total_bits_out, const ExchangeUpdate* upd, int sym_mode, double* sum_sq,
                         uint64_t coord_base) {
  if (coord_base % kQuad != 0) return QGX_ERR_INVALID_ARG;
  if (!c || !cfg || !mean_out || K < 1 || K > 65535 || d < 1 || slot < 0 || slot > 1) return QGX_ERR_INVALID_ARG;
  const int bucket = cfg->bucket;
  if (bucket < kQuad || bucket > QGX_MAX_BUCKET || bucket % kQuad != 0) return QGX_ERR_INVALID_ARG;
  if (cfg->norm_type != QGX_NORM_L2 && cfg->norm_type != QGX_NORM_LINF) return QGX_ERR_INVALID_ARG;
  if (check_levels_host(cfg->levels, cfg->nlev) != QGX_OK) return QGX_ERR_BAD_LEVELS;
  if (cfg->cb.nlev != cfg->nlev) return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  const CachedTables* tables = nullptr;
  qgx_status rc = cached_tables(c, cfg, &tables);
  if (rc != QGX_OK) return rc;
  const CodeTable& ct = tables->ct;
  LevelTable lt;
  lt.nlev = cfg->nlev;
  for (int j = 0; j < QGX_MAX_LEVELS; ++j) lt.lev[j] = j < cfg->nlev ? cfg->levels[j] : 1.0f;

  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  const size_t cap = qgx_stream_capacity_words(d, bucket, cfg->cb.subblock, QGX_MAX_CODE_LEN);   // fits any codebook
  const int base = WS_SLOT0 + 4 * slot;
  uint32_t* stream = (uint32_t*)ws_get(c, base + 0, sizeof(uint32_t) * ((size_t)K * cap + 64));   // slack: see Window
  uint32_t* bbits = (uint32_t*)ws_get(c, base + 1, sizeof(uint32_t) * (size_t)K * nb);
  uint32_t* offs = (uint32_t*)ws_get(c, base + 2, sizeof(uint32_t) * (size_t)K * nb);
  // one block per slot, zeroed by one memset: the per-worker bit totals, the ticket counter, the status words of the scan
  unsigned long long* tot = (unsigned long long*)ws_get(c, base + 3, sizeof(uint64_t) * ((size_t)K + 2 + (size_t)K * nb));
  unsigned long long* status = tot ? tot + K + 2 : nullptr;
  float* norms = (float*)ws_get(c, slot == 0 ? WS_NORMS : WS_NORMS2, sizeof(float) * (size_t)K * nb);
  const DecEntry* lut = tables->lut_dev;
  if (!stream || !bbits || !offs || !tot || !status || !norms || !lut) return QGX_ERR_CUDA;
  c->slot_cap_words[slot] = cap;
  c->slot_K[slot] = K;
  c->slot_nb[slot] = nb;

  const bool do_encode = !c->decode_only;               // the decode-only entry point works on the streams that are there
  if (do_encode && cudaMemsetAsync(tot, 0, sizeof(uint64_t) * ((size_t)K + 2 + (size_t)K * nb), c->stream) != cudaSuccess) return QGX_ERR_CUDA;

  EncodeArgs ea;
  ea.src = src; ea.d = d; ea.bucket = bucket; ea.K = K; ea.nb = nb; ea.norm_type = cfg->norm_type; ea.xid = xid; ea.quad_base = coord_base / kQuad;
  ea.vec_ok = (d % kQuad == 0) && (src.ld % kQuad == 0) && ((reinterpret_cast<uintptr_t>(src.v) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(src.a) & 15u) == 0);
  ea.stream = stream; ea.cap_words = cap; ea.bucket_bits = bbits; ea.offsets = offs; ea.total_bits = tot; ea.norms = norms;
  ea.status = status; ea.ticket = reinterpret_cast<unsigned int*>(tot + K); ea.st = c->dstatus; ea.tables = tables->enc_dev;
  uint8_t* sym_out = nullptr;
  const uint8_t* sym_prev = nullptr;
  const size_t sym_ld = ((nb * (size_t)(bucket / ct.G) + 31) / 32) * 32 * (size_t)ct.G;   // see DecodeArgs::sym_out
  const float* norms_prev = nullptr;
  if (sym_mode < 0 || sym_mode > 5) return QGX_ERR_INVALID_ARG;
  if ((sym_mode & 6) && !sum_sq) return QGX_ERR_INVALID_ARG;
  LevelTable lt_kept = lt;                                  // the table of the symbols compared with
  if (sym_mode & 2) {
    if (c->sym_slot != 1 - slot || c->sym_K != K || c->sym_d != d || c->sym_ld != sym_ld || c->slot_nb[1 - slot] != nb) return QGX_ERR_INVALID_ARG;
    sym_prev = (const uint8_t*)c->ws[WS_SYM];
    norms_prev = (const float*)c->ws[slot == 0 ? WS_NORMS2 : WS_NORMS];
    lt_kept.nlev = c->sym_nlev;
    for (int j = 0; j < QGX_MAX_LEVELS; ++j) lt_kept.lev[j] = j < c->sym_nlev ? c->sym_levels[j] : 1.0f;
  }
  if (sym_mode & 1) {
    sym_out = (uint8_t*)ws_get(c, WS_SYM, (size_t)K * sym_ld + 16);
    if (!sym_out) return QGX_ERR_CUDA;
    c->sym_slot = slot; c->sym_K = K; c->sym_d = d; c->sym_ld = sym_ld; c->sym_bucket = bucket; c->sym_G = ct.G;
    c->sym_nlev = cfg->nlev;
    for (int j = 0; j < cfg->nlev; ++j) c->sym_levels[j] = cfg->levels[j];
  }
  const PhiloxKey key = make_philox_key(cfg->seed);
  const RoundTable& qt = tables->rt;
  if (!ct.has_header || bucket % ct.G != 0 || (ct.G != 32 && ct.G != 64 && ct.G != 128)) return QGX_ERR_INVALID_ARG;
  // octets per thread chosen so that CTAs have at most 256 / 512 / 512 threads
  const int pp = bucket <= 2048 ? 1 : (bucket <= 8192 ? 2 : 4);
  const int threads = bucket_threads(bucket, 2 * pp);
  const size_t img_words = (((((size_t)bucket * (ct.maxlen + 1) + 16u * (bucket / ct.G + 1) + kNormBits + 31u) >> 5) + 4) + 3) & ~(size_t)3;
  const size_t smem = sizeof(uint32_t) * 2 * img_words;   // two images: see k_exchange_encode
  int per_sm = 1;
#define QGX_LAUNCH_E(V, GG)                                                                                    \
  do {                                                                                                         \
    allow_max_dynamic_smem(k_exchange_encode<V, GG>, c->device);                                               \
    LaunchShape& shape = table_cache(c)->enc[V == 1 ? 0 : (V == 2 ? 1 : 2)][GG == 32 ? 0 : (GG == 64 ? 1 : 2)];  \
    if (shape.smem != smem + 1 + (size_t)threads * 0x100000) {   /* occupancy asked once per shape */          \
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_exchange_encode<V, GG>, threads, smem);         \
      shape.smem = smem + 1 + (size_t)threads * 0x100000;                                                      \
      shape.per_sm = per_sm < 1 ? 1 : per_sm;                                                                  \
    }                                                                                                          \
    per_sm = shape.per_sm;                                                                                     \
    const unsigned long long want = (unsigned long long)(nb - ea.b_first) * (unsigned long long)K;             \
    const unsigned grid = (unsigned)std::min<unsigned long long>(want, (unsigned long long)c->num_sms * (unsigned long long)per_sm);   \
    k_exchange_encode<V, GG><<<grid, threads, smem, c->stream>>>(ea, lt, ct, key, qt);                         \
  } while (0)
#define QGX_LAUNCH_EG(V)                                   \
  do {                                                     \
    if (ct.G == 32) QGX_LAUNCH_E(V, 32);                   \
    else if (ct.G == 64) QGX_LAUNCH_E(V, 64);              \
    else QGX_LAUNCH_E(V, 128);                             \
  } while (0)
  // Whole buckets of a multiple of 1024 coordinates that divides 16384 go through the staged kernel; what is left
  // (a short last bucket, other bucket sizes, unaligned vectors) through the bucket-in-registers kernel.
  bool staged_ok = ea.vec_ok && bucket % kWarpCoords == 0 && kStageCoords % bucket == 0 && coord_base % 8 == 0 &&
                   c->encode_path == QGX_ENCODE_STAGED && d / (size_t)bucket > 0 && c->skip_buckets == 0;
  CUtensorMap tmap;
  std::memset(&tmap, 0, sizeof(tmap));
  if (staged_ok) {
    // the staged source: the workers' rows (worker k at k * ld) or, without them, the shared vector a
    const size_t ldv = src.ld ? src.ld : d;
    const size_t whole = (d / (size_t)bucket) * (size_t)bucket;
    const float* base = src.v ? src.v : src.a;
    const unsigned long long floats = src.v ? (unsigned long long)(K - 1) * ldv + whole : whole;
    staged_ok = (!src.v || ldv % kLaneCoords == 0) &&
                make_rows_map(base, floats / kLaneCoords, (unsigned)std::min(256, bucket / kLaneCoords), &tmap);
  }
  ea.nb_whole = staged_ok ? d / (size_t)bucket : 0;
  ea.b_first = staged_ok ? ea.nb_whole : std::min(c->skip_buckets, nb);
  c->skip_buckets = 0;
  ea.spin_limit = c->wait_limit;
  if (do_encode) {
    ScopedKernelTimer timer(c, QGX_KERNEL_ENCODE);
    if (ea.nb_whole > 0) {
      const size_t smem_st = sizeof(float) * kStageCoords * kStageBuffers;
      const unsigned long long per_group = (unsigned long long)(kStageCoords / bucket);
      const unsigned long long groups = ((unsigned long long)ea.nb_whole * (unsigned long long)K + per_group - 1ull) / per_group;
#define QGX_LAUNCH_SG(GG)                                                                                            \
  do {                                                                                                               \
    allow_max_dynamic_smem(k_encode_staged<GG>, c->device);                                                          \
    LaunchShape& shape = table_cache(c)->enc_staged[GG == 32 ? 0 : (GG == 64 ? 1 : 2)];                              \
    if (shape.smem == 0) {                                                                                           \
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_encode_staged<GG>, kStagedThreads, smem_st);          \
      shape.smem = 1;                                                                                                \
      shape.per_sm = per_sm < 1 ? 1 : per_sm;                                                                        \
    }                                                                                                                \
    const unsigned grid = (unsigned)std::min<unsigned long long>((groups + 1ull) / 2ull, (unsigned long long)c->num_sms * (unsigned long long)shape.per_sm); \
    /* a cooperative launch: the static assignment of groups needs every CTA of the grid resident at once, */       \
    /* also when other kernels (another exchange on a helper stream) share the device                      */       \
    void* kargs[] = {(void*)&ea, (void*)&lt, (void*)&ct, (void*)&key, (void*)&qt, (void*)&tmap};                     \
    cudaLaunchCooperativeKernel((const void*)k_encode_staged<GG>, dim3(grid), dim3(kStagedThreads), kargs, smem_st, c->stream); \
  } while (0)
      if (ct.G == 32) QGX_LAUNCH_SG(32);
      else if (ct.G == 64) QGX_LAUNCH_SG(64);
      else QGX_LAUNCH_SG(128);
#undef QGX_LAUNCH_SG
      count_launch(c);
    }
    if (ea.b_first < nb) {
      switch (pp) {
        case 1: QGX_LAUNCH_EG(1); break;
        case 2: QGX_LAUNCH_EG(2); break;
        default: QGX_LAUNCH_EG(4); break;
      }
      count_launch(c);
    }
  }
#undef QGX_LAUNCH_EG
#undef QGX_LAUNCH_E
  if (cudaGetLastError() != cudaSuccess) return QGX_ERR_CUDA;
  if (total_bits_out &&
      cudaMemcpyAsync(total_bits_out, tot, sizeof(uint64_t) * (size_t)K, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
    return QGX_ERR_CUDA;

  DecodeArgs da;
  da.stream = stream; da.cap_words = cap; da.bucket_bits = bbits; da.offsets = offs;
  da.sym_out = sym_out; da.sym_prev = sym_prev; da.sym_ld = sym_ld; da.norms_prev = norms_prev; da.sum_sq = sum_sq;
  da.d = d; da.bucket = bucket; da.K = K; da.nb = nb; da.lut = lut; da.mean = mean_out;
  da.update = upd ? upd->mode : 0; da.xin = upd ? upd->xin : nullptr; da.xout = upd ? upd->xout : nullptr;
  da.scalars = upd ? upd->scalars : nullptr; da.st = c->dstatus;
  da.vec_out = (d % kQuad == 0) && ((reinterpret_cast<uintptr_t>(mean_out) & 15u) == 0) &&
               ((reinterpret_cast<uintptr_t>(da.xin) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(da.xout) & 15u) == 0);
  // Small vectors leave most of the GPU idle and make every thread walk all K workers one after the other: there
  // the decode pass runs one worker per thread and a second kernel forms the ordered sums.
  const size_t total_sub = nb * (size_t)(bucket / ct.G);
  da.values = nullptr;
  const bool fits = (size_t)K * d * sizeof(float) <= ((size_t)256 << 20);
  const bool small = total_sub * 2 < (size_t)c->num_sms * kDecThreads * 4;
  if (K > 1 && fits && c->decode_split != QGX_SPLIT_NEVER && c->decode_split != QGX_SPLIT_SYMBOLS && (small || c->decode_split == QGX_SPLIT_ALWAYS)) {
    da.values = (float*)ws_get(c, WS_VALUES, sizeof(float) * (size_t)K * d);
    if (!da.values) return QGX_ERR_CUDA;
  }
  // Large vectors: the walk alone with one worker per thread (twice the warps of the one-pass kernel, whose 64 running
  // sums per thread fill the register file), every worker's symbol bytes kept, and the ordered sums from those.
  da.norms_out = nullptr;
  const bool in_place = (sym_mode & 3) == 3;             // compares with the kept symbols and overwrites them: one pass
  const bool two_pass = K > 1 && !da.values && !in_place &&
                        (c->decode_split == QGX_SPLIT_SYMBOLS || (c->decode_split == QGX_SPLIT_AUTO && !small && kTwoPassByDefault));
  if (two_pass) {
    if (!da.sym_out) da.sym_out = (uint8_t*)ws_get(c, WS_SYMTMP, (size_t)K * sym_ld);
    da.norms_out = (float*)ws_get(c, WS_NORMSDEC, sizeof(float) * (size_t)K * nb);
    if (!da.sym_out || !da.norms_out) return QGX_ERR_CUDA;
    rc = launch_decode_average(c, da, ct, lt_kept, 0, true);
    if (rc != QGX_OK) return rc;
    MeanArgs ma;
    ma.sym = da.sym_out; ma.sym_ld = sym_ld; ma.norms = da.norms_out; ma.sym_prev = da.sym_prev; ma.norms_prev = da.norms_prev;
    ma.sum_sq = da.sum_sq; ma.K = K; ma.d = d; ma.bucket = bucket; ma.nb = nb; ma.mean = mean_out; ma.update = da.update;
    ma.xin = da.xin; ma.xout = da.xout; ma.scalars = da.scalars; ma.vec_out = da.vec_out; ma.st = c->dstatus;
    {
      ScopedKernelTimer timer(c, QGX_KERNEL_DECODE);
      const size_t rows = (total_sub + 31) / 32;
      const size_t threads = rows * (size_t)(ct.G / 16) * 32;
      const unsigned grid = (unsigned)std::max<size_t>(1, std::min<size_t>((threads + 255) / 256, (size_t)c->num_sms * 6));
      const size_t smem = sizeof(float) * (256 * 32 + 256);
#define QGX_LAUNCH_M(GG, SS) k_symbols_mean<GG, SS><<<grid, 256, smem, c->stream>>>(ma, lt, lt_kept)
#define QGX_LAUNCH_MG(GG)                                  \
  do {                                                     \
    if (sym_mode & 2) QGX_LAUNCH_M(GG, 2);                 \
    else if (sym_mode & 4) QGX_LAUNCH_M(GG, 4);            \
    else QGX_LAUNCH_M(GG, 0);                              \
  } while (0)
      if (ct.G == 32) QGX_LAUNCH_MG(32);
      else if (ct.G == 64) QGX_LAUNCH_MG(64);
      else QGX_LAUNCH_MG(128);
#undef QGX_LAUNCH_MG
#undef QGX_LAUNCH_M
    }
    count_launch(c);
    return cuda_status(cudaGetLastError());
  }
  rc = launch_decode_average(c, da, ct, lt_kept, sym_mode);
  if (rc != QGX_OK || !da.values) return rc;
  {
    ScopedKernelTimer timer(c, QGX_KERNEL_DECODE);
    const unsigned grid = (unsigned)std::max<size_t>(1, std::min<size_t>((d + 255) / 256, (size_t)c->num_sms * 8));
    k_sum_workers<<<grid, 256, 0, c->stream>>>(da.values, K, d, mean_out, da.update, da.xin, da.xout, da.scalars);
  }
  count_launch(c);
  return cuda_status(cudaGetLastError());
}

template <int G, int SYM, bool VAL>
static qgx_status launch_decode_gs(qgx_ctx* c, const DecodeArgs& da, const CodeTable& ct, const LevelTable& lt) {
  const size_t subs = da.nb * ((size_t)da.bucket / G);
  const size_t total_sub = (!VAL || da.values) ? ((subs + 31) & ~(size_t)31) * (size_t)da.K : subs;   // threads wanted
  const size_t lut_bytes = (VAL ? sizeof(DecEntry) : sizeof(uint32_t)) * ((size_t)2 << ct.maxlen) + DecodeSmem<G, SYM, VAL>::kBytes;   // table, then the rows
  const size_t want = (total_sub + kDecThreads - 1) / kDecThreads;
  int per_sm = 1;
  {
    ScopedKernelTimer timer(c, QGX_KERNEL_DECODE);
    allow_max_dynamic_smem(k_exchange_decode<G, SYM, VAL>, c->device);
    TableCache* tc = table_cache(c);
    LaunchShape& shape = (VAL ? tc->dec : tc->dec_walk)[G == 32 ? 0 : (G == 64 ? 1 : 2)][SYM];
    if (shape.smem != lut_bytes + 1) {                       // occupancy asked once per shape, not per call
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_exchange_decode<G, SYM, VAL>, kDecThreads, lut_bytes);
      shape.smem = lut_bytes + 1;
      shape.per_sm = per_sm < 1 ? 1 : per_sm;
    }
    per_sm = shape.per_sm;
    const unsigned grid = (unsigned)std::max<size_t>(1, std::min<size_t>(want, (size_t)c->num_sms * per_sm));
    k_exchange_decode<G, SYM, VAL><<<grid, kDecThreads, lut_bytes, c->stream>>>(da, ct, lt);
  }
  count_launch(c);
  return cuda_status(cudaGetLastError());
}

template <int G, bool VAL>
static qgx_status launch_decode_g(qgx_ctx* c, const DecodeArgs& da, const CodeTable& ct, const LevelTable& lt, int sym_mode) {
  switch (sym_mode) {
    case 1: return launch_decode_gs<G, 1, VAL>(c, da, ct, lt);
    case 2: return launch_decode_gs<G, 2, VAL>(c, da, ct, lt);
    case 3: return launch_decode_gs<G, 3, VAL>(c, da, ct, lt);
    case 4: return launch_decode_gs<G, 4, VAL>(c, da, ct, lt);
    case 5: return launch_decode_gs<G, 5, VAL>(c, da, ct, lt);
    default: return launch_decode_gs<G, 0, VAL>(c, da, ct, lt);
  }
}

qgx_status launch_decode_average(qgx_ctx* c, const DecodeArgs& da, const CodeTable& ct, const LevelTable& lt, int sym_mode,
                                 bool walk_only) {
  if (!ct.has_header || da.bucket % ct.G != 0) return QGX_ERR_INVALID_ARG;
  if (walk_only) {
    switch (ct.G) {
      case 32: return launch_decode_g<32, false>(c, da, ct, lt, sym_mode);
      case 64: return launch_decode_g<64, false>(c, da, ct, lt, sym_mode);
      case 128: return launch_decode_g<128, false>(c, da, ct, lt, sym_mode);
      default: return QGX_ERR_INVALID_ARG;
    }
  }
  switch (ct.G) {
    case 32: return launch_decode_g<32, true>(c, da, ct, lt, sym_mode);
    case 64: return launch_decode_g<64, true>(c, da, ct, lt, sym_mode);
    case 128: return launch_decode_g<128, true>(c, da, ct, lt, sym_mode);
    default: return QGX_ERR_INVALID_ARG;
  }
}

// ---- helper contexts of the layer-wise exchange -------------------------------------------------
// The tensors of a layer-wise vector are independent; most are small, so one after the other they leave the GPU
// mostly idle.  They are spread over a few helper contexts, each with its own stream and workspace; the caller's
// stream forks into them and joins them again (events), so the call stays asynchronous and ordered on that stream.
constexpr int kSegStreams = 4;
struct SegChildren {
  qgx_ctx* ctx[kSegStreams];
  cudaEvent_t fork, join[kSegStreams];
};

void free_seg_children(qgx_ctx* c) {
  SegChildren* sc = (SegChildren*)c->seg_children;
  if (!sc) return;
  for (int i = 0; i < kSegStreams; ++i) {
    qgx_ctx* h = sc->ctx[i];
    if (!h) continue;
    cudaStreamSynchronize(h->stream);
    free_table_cache(h);
    for (int w = 0; w < 24; ++w)
      if (h->ws[w]) cudaFree(h->ws[w]);
    cudaStreamDestroy(h->stream);
    cudaEventDestroy(sc->join[i]);
    delete h;                                           // the status block belongs to the parent
  }
  cudaEventDestroy(sc->fork);
  delete sc;
  c->seg_children = nullptr;
}

uint64_t seg_children_launches(const qgx_ctx* c) {
  const SegChildren* sc = (const SegChildren*)c->seg_children;
  uint64_t n = 0;
  if (sc)
    for (int i = 0; i < kSegStreams; ++i) n += sc->ctx[i] ? sc->ctx[i]->launches : 0;
  return n;
}

static SegChildren* seg_children(qgx_ctx* c) {
  if (c->seg_children) return (SegChildren*)c->seg_children;
  SegChildren* sc = new (std::nothrow) SegChildren();
  if (!sc) return nullptr;
  bool ok = cudaEventCreateWithFlags(&sc->fork, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < kSegStreams && ok; ++i) {
    qgx_ctx* h = new (std::nothrow) qgx_ctx();
    if (!h) { ok = false; break; }
    std::memset(h, 0, sizeof(*h));
    h->device = c->device;
    h->sym_slot = -1;
    h->wait_limit = c->wait_limit;
    h->decode_split = c->decode_split;
    h->encode_path = c->encode_path;
    h->num_sms = c->num_sms;
    h->dstatus = c->dstatus;                            // errors latch into the parent's status block
    if (cudaStreamCreateWithFlags(&h->stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&sc->join[i], cudaEventDisableTiming) != cudaSuccess) {
      delete h;
      ok = false;
      break;
    }
    sc->ctx[i] = h;
  }
  c->seg_children = sc;
  if (!ok) { cudaGetLastError(); free_seg_children(c); return nullptr; }
  return sc;
}

// counts[j] += coordinates of the kept symbols (layout: DecodeArgs::sym_out) that carry level j
__global__ void __launch_bounds__(256) k_level_counts(const uint8_t* __restrict__ sym, int K, size_t d, size_t sym_ld, int bucket, int G,
                                                      unsigned long long* counts) {
  __shared__ unsigned int s_cnt[8][QGX_MAX_LEVELS];                  // one set per warp
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) < QGX_MAX_LEVELS) s_cnt[warp][threadIdx.x & 31] = 0u;
  __syncwarp();
  const size_t wpw = sym_ld / 4;                                      // words per worker
  const size_t spb = (size_t)(bucket / G);
  const size_t total_sub = ((d + (size_t)bucket - 1) / (size_t)bucket) * spb;
  for (size_t w = (size_t)blockIdx.x * blockDim.x + threadIdx.x; w < (size_t)K * wpw; w += (size_t)gridDim.x * blockDim.x) {
    const size_t at = (w % wpw) * 4;                                  // byte inside the worker's symbols
    const size_t gs = (at / (size_t)(32 * G)) * 32 + (at % 128) / 4;  // the sub-block
    const size_t i0 = ((at % (size_t)(32 * G)) / 128) * 4;            // first of the word's four coordinates in it
    if (gs >= total_sub) continue;
    const size_t e0 = (gs / spb) * (size_t)bucket + (gs % spb) * (size_t)G + i0;
    const uint32_t four = *reinterpret_cast<const uint32_t*>(sym + w * 4);
    for (int cc = 0; cc < 4; ++cc)
      if (e0 + cc < d && e0 + cc < (gs / spb + 1) * (size_t)bucket) atomicAdd(&s_cnt[warp][(four >> (8 * cc)) & 31u], 1u);
  }
  __syncwarp();
  const unsigned int mine = (threadIdx.x & 31) < QGX_MAX_LEVELS ? s_cnt[warp][threadIdx.x & 31] : 0u;
  if (mine) atomicAdd(counts + (threadIdx.x & 31), (unsigned long long)mine);
}

// acc[i] += x[i]; several streams may add into the same totals
__global__ void k_add_u64_atomic(unsigned long long* acc, const unsigned long long* x, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) atomicAdd(acc + i, x[i]);
}

}  // namespace qgx

using namespace qgx;

extern "C" {

qgx_status qgx_set_decode_split(qgx_ctx* c, int mode) {
  if (!c || mode < QGX_SPLIT_AUTO || mode > QGX_SPLIT_SYMBOLS) return QGX_ERR_INVALID_ARG;
  c->decode_split = mode;
  return QGX_OK;
}

qgx_status qgx_set_encode_path(qgx_ctx* c, int mode) {
  if (!c || (mode != QGX_ENCODE_AUTO && mode != QGX_ENCODE_REGISTERS && mode != QGX_ENCODE_STAGED)) return QGX_ERR_INVALID_ARG;
  c->encode_path = mode;
  return QGX_OK;
}

qgx_status qgx_exchange(qgx_ctx* c, const float* v, int K, size_t d, const qgx_quant_cfg* cfg, uint32_t exchange_id,
                        int slot, float* mean_out, uint64_t* total_bits) {
  if (!v) return QGX_ERR_INVALID_ARG;
  DualSource src{v, nullptr, 0, 0};
  return exchange_impl(c, src, K, d, cfg, exchange_id, slot, mean_out, total_bits, nullptr, (c && c->keep_symbols) ? 1 : 0, nullptr, 0);
}

qgx_status qgx_exchange_segments(qgx_ctx* c, const float* v, int K, size_t d, const qgx_segment* segs, int nseg,
                                 uint32_t exchange_id, float* mean_out, uint64_t* total_bits) {
  if (!c || !v || !segs || nseg < 1 || !mean_out || K < 1) return QGX_ERR_INVALID_ARG;
  // the segments must tile [0, d) in order, each starting on a multiple of 4 coordinates
  size_t at = 0;
  for (int s = 0; s < nseg; ++s) {
    if (segs[s].offset != at || segs[s].length < 1 || segs[s].offset % kQuad != 0 || !segs[s].cfg) return QGX_ERR_INVALID_ARG;
    at += segs[s].length;
  }
  if (at != d) return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  if (total_bits && cudaMemsetAsync(total_bits, 0, sizeof(uint64_t) * (size_t)K, c->stream) != cudaSuccess) return QGX_ERR_CUDA;
  SegChildren* sc = nseg > 1 ? seg_children(c) : nullptr;
  if (nseg > 1 && !sc) return QGX_ERR_CUDA;
  const int lanes = sc ? std::min(nseg, kSegStreams) : 0;
  if (sc) {                                             // fork: the helpers start after everything queued so far
    if (cudaEventRecord(sc->fork, c->stream) != cudaSuccess) return QGX_ERR_CUDA;
    for (int i = 0; i < lanes; ++i) {
      sc->ctx[i]->decode_split = c->decode_split;
      sc->ctx[i]->encode_path = c->encode_path;
      if (cudaStreamWaitEvent(sc->ctx[i]->stream, sc->fork, 0) != cudaSuccess) return QGX_ERR_CUDA;
    }
  }
  qgx_status rc = QGX_OK;
  for (int s = 0; s < nseg && rc == QGX_OK; ++s) {
    qgx_ctx* h = sc ? sc->ctx[s % lanes] : c;
    uint64_t* seg_bits = nullptr;
    if (total_bits) {
      seg_bits = (uint64_t*)ws_get(h, WS_SEGBITS, sizeof(uint64_t) * (size_t)K);
      if (!seg_bits) { rc = QGX_ERR_CUDA; break; }
    }
    DualSource src{v + segs[s].offset, nullptr, d, 0};
    rc = exchange_impl(h, src, K, segs[s].length, segs[s].cfg, exchange_id, 0, mean_out + segs[s].offset, seg_bits,
                       nullptr, 0, nullptr, segs[s].offset);
    if (rc == QGX_OK && total_bits) {
      k_add_u64_atomic<<<(K + 255) / 256, 256, 0, h->stream>>>(reinterpret_cast<unsigned long long*>(total_bits),
                                                               reinterpret_cast<const unsigned long long*>(seg_bits), K);
      count_launch(h);
    }
  }
  if (sc) {                                             // join, also after an error: the caller's stream waits for the helpers
    for (int i = 0; i < lanes; ++i)
      if (cudaEventRecord(sc->join[i], sc->ctx[i]->stream) != cudaSuccess ||
          cudaStreamWaitEvent(c->stream, sc->join[i], 0) != cudaSuccess)
        rc = rc == QGX_OK ? QGX_ERR_CUDA : rc;
  }
  if (rc != QGX_OK) return rc;
  return cuda_status(cudaGetLastError());
}

qgx_status qgx_exchange_decode(qgx_ctx* c, int K, size_t d, const qgx_quant_cfg* cfg, int slot, float* mean_out) {
  if (!c || slot < 0 || slot > 1 || !cfg || c->slot_K[slot] != K || K < 1 || d < 1 || cfg->bucket < kQuad ||
      c->slot_nb[slot] != (d + (size_t)cfg->bucket - 1) / (size_t)cfg->bucket)
    return QGX_ERR_INVALID_ARG;
  DualSource none{nullptr, nullptr, 0, 0};
  c->decode_only = 1;
  const qgx_status rc = exchange_impl(c, none, K, d, cfg, 0, slot, mean_out, nullptr, nullptr, 0, nullptr, 0);
  c->decode_only = 0;
  return rc;
}

qgx_status qgx_set_wait_limit(qgx_ctx* c, int polls) {
  if (!c || polls < 1) return QGX_ERR_INVALID_ARG;
  c->wait_limit = polls;
  return QGX_OK;
}

qgx_status qgx_debug_skip_buckets(qgx_ctx* c, size_t buckets) {
  if (!c) return QGX_ERR_INVALID_ARG;
  c->skip_buckets = buckets;
  return QGX_OK;
}

qgx_status qgx_set_keep_symbols(qgx_ctx* c, int on) {
  if (!c) return QGX_ERR_INVALID_ARG;
  c->keep_symbols = on ? 1 : 0;
  return QGX_OK;
}

qgx_status qgx_level_counts(qgx_ctx* c, uint64_t* counts) {
  if (!c || !counts || c->sym_slot < 0 || !c->ws[WS_SYM] || c->sym_G <= 0) return QGX_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  if (cudaMemsetAsync(counts, 0, sizeof(uint64_t) * QGX_MAX_LEVELS, c->stream) != cudaSuccess) return QGX_ERR_CUDA;
  const size_t words = (size_t)c->sym_K * (c->sym_ld / 4);
  const unsigned grid = (unsigned)std::max<size_t>(1, std::min<size_t>((words + 255) / 256, (size_t)c->num_sms * 8));
  k_level_counts<<<grid, 256, 0, c->stream>>>((const uint8_t*)c->ws[WS_SYM], c->sym_K, c->sym_d, c->sym_ld, c->sym_bucket, c->sym_G,
                                               reinterpret_cast<unsigned long long*>(counts));
  count_launch(c);
  return cuda_status(cudaGetLastError());
}

qgx_status qgx_exchange_streams(qgx_ctx* c, int slot, const uint32_t** stream, size_t* cap_words,
                                const uint32_t** bucket_bits, const uint64_t** total_bits) {
  if (!c || slot < 0 || slot > 1 || c->slot_K[slot] == 0) return QGX_ERR_INVALID_ARG;
  const int base = WS_SLOT0 + 4 * slot;
  if (stream) *stream = (const uint32_t*)c->ws[base + 0];
  if (cap_words) *cap_words = c->slot_cap_words[slot];
  if (bucket_bits) *bucket_bits = (const uint32_t*)c->ws[base + 1];
  if (total_bits) *total_bits = (const uint64_t*)c->ws[base + 3];
  return QGX_OK;
}

}  // extern "C"
