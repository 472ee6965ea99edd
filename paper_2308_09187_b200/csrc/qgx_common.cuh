// Shared device/host helpers of the qgx CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/qgx.h"

namespace qgx {

constexpr int kWarp = 32;
constexpr int kNormBits = 32;            // C_b of App. E: the norm travels as an IEEE fp32 pattern
constexpr int kQuad = 4;                 // coordinates per 128-bit load and per Philox block
constexpr int kSpinLimit = 1 << 22;      // polls before a device-side wait gives up

// device-resident status block of a context
struct DevStatus {
  unsigned int error;                    // first latched qgx_status, 0 if none
  unsigned int pad;
};

}  // namespace qgx

struct qgx_ctx {
  int device;
  cudaStream_t stream;
  unsigned int* hstatus;                 // pinned host mirror
  uint64_t launches;
  // workspace of the fused calls, grown on demand
  qgx::DevStatus* dstatus;               // [dev]
  void* ws[24];
  size_t ws_bytes[24];
  // bookkeeping of the exchange slots
  size_t slot_cap_words[2];
  int slot_K[2];
  size_t slot_nb[2];
  // which exchange slot last kept its symbols in the workspace (-1: none), and for what shape
  int sym_slot;
  int sym_K;
  size_t sym_d;
  size_t sym_ld;                         // bytes per worker in the kept-symbol layout
  int sym_bucket, sym_G;                 // bucket and sub-block sizes of that layout
  int keep_symbols;                      // qgx_exchange keeps its decoded symbols too (qgx_set_keep_symbols)
  int wait_limit;                        // polls of a device-side wait before it gives up (qgx_set_wait_limit)
  size_t skip_buckets;                   // diagnostic: the next exchange leaves these first buckets unencoded
  int decode_only;                       // set around the decode-only entry point
  int sym_nlev;                          // the level table those symbols were quantized with
  float sym_levels[QGX_MAX_LEVELS];
  int decode_split;                      // QGX_SPLIT_AUTO / NEVER / ALWAYS: see qgx_set_decode_split
  int encode_path;                       // QGX_ENCODE_AUTO / REGISTERS: see qgx_set_encode_path
  int num_sms;                           // multiprocessors of the device
  // host-side cache of the fused calls: tables derived from a quantizer configuration (with their device copies)
  // and launch shapes; owned by qgx_exchange.cu
  void* table_cache;
  // helper contexts (own streams and workspaces) that run the tensors of a layer-wise exchange side by side;
  // owned by qgx_exchange.cu
  void* seg_children;
  // optional per-kernel timing: pairs of events recorded around instrumented launches
  int timing_on;
  int timing_cap;                        // pairs allocated
  int timing_used;
  cudaEvent_t* timing_ev;                // 2 * timing_cap events
  int* timing_kind;                      // kernel id of each pair
};

namespace qgx {

// ---- level table and code tables handed to kernels by value ---------------------------------
struct LevelTable {
  int nlev;
  float lev[QGX_MAX_LEVELS];
};

// Bins of the rounding table over the float pattern of the normalized coordinate (see round_fast).  A bin covers
// 2^key_shift consecutive patterns (2^(23 - key_shift) bins per octave of u: 64 at key_shift 17, 8 at 20); patterns
// below 2^-16 share bin 0 and the table ends at u = 1.  Every bin is stored 2^(key_shift - 17) times, once per
// residue of the lane number, so that the lanes of a quarter warp read different bank groups whatever bins they
// hit: the coarser the bins the levels allow (at most one level per bin), the fewer bank conflicts.  All layouts
// take the same 16.1 KB.
constexpr int kKeyShiftMin = 17, kKeyShiftMax = 20;
constexpr uint32_t kKeyBase = 0x37800000u;          // pattern of 2^-16
constexpr uint32_t kKeyTop = 0x3F800000u;           // pattern of 1.0
constexpr int kBinEntries = ((kKeyTop - kKeyBase) >> kKeyShiftMin) + (1 << (kKeyShiftMax - kKeyShiftMin));   // float4 entries, any layout
constexpr int kBinAddrShift = kKeyShiftMin - 4;     // pattern >> 13 = byte offset of the bin's first copy (+ a constant)
constexpr uint32_t kBinAddrBase = kKeyBase >> kBinAddrShift;
struct CodeTable {
  int nlev;
  int maxlen;
  int G;                                 // coordinates per sub-block (== bucket: no header)
  int has_header;
  // per level index: stream-order bits (first sent bit at bit 0) and length, without sign
  uint16_t rev[QGX_MAX_LEVELS];
  uint8_t len[QGX_MAX_LEVELS];
};

__host__ __device__ inline uint64_t ceil_div_u64(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

inline int eff_subblock(int bucket, int subblock) {
  return (subblock <= 0 || subblock >= bucket) ? bucket : subblock;
}

// latch the first error
__device__ __forceinline__ void latch_error(DevStatus* st, unsigned int code) {
  atomicCAS(&st->error, 0u, code);
}

// ---- Philox4x32-10 (Salmon et al., SC'11): counter-based, ten rounds ------------------------
struct PhiloxKey {                       // the ten round keys, the same for every thread
  uint32_t k0[10];
  uint32_t k1[10];
};

inline PhiloxKey make_philox_key(uint64_t seed) {
  PhiloxKey k;
  uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    k.k0[r] = a;
    k.k1[r] = b;
    a += 0x9E3779B9u;                    // Weyl sequence of the golden ratio
    b += 0xBB67AE85u;                    // Weyl sequence of sqrt(3) - 1
  }
  return k;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKey& key) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;      // one wide multiply gives both halves
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ key.k0[r];
    const uint32_t n2 = hi0 ^ c3 ^ key.k1[r];
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// two blocks that share the last two counter words, round by round (the round keys are fetched once)
__device__ __forceinline__ void philox4x32_10_x2(uint64_t ctr_a, uint64_t ctr_b, uint32_t c2, uint32_t c3, const PhiloxKey& key,
                                                 uint4* out_a, uint4* out_b) {
  uint32_t a0 = (uint32_t)ctr_a, a1 = (uint32_t)(ctr_a >> 32), a2 = c2, a3 = c3;
  uint32_t b0 = (uint32_t)ctr_b, b1 = (uint32_t)(ctr_b >> 32), b2 = c2, b3 = c3;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t k0 = key.k0[r], k1 = key.k1[r];
    const uint64_t pa0 = (uint64_t)0xD2511F53u * (uint64_t)a0, pa1 = (uint64_t)0xCD9E8D57u * (uint64_t)a2;
    const uint64_t pb0 = (uint64_t)0xD2511F53u * (uint64_t)b0, pb1 = (uint64_t)0xCD9E8D57u * (uint64_t)b2;
    const uint32_t na0 = (uint32_t)(pa1 >> 32) ^ a1 ^ k0, na2 = (uint32_t)(pa0 >> 32) ^ a3 ^ k1;
    const uint32_t nb0 = (uint32_t)(pb1 >> 32) ^ b1 ^ k0, nb2 = (uint32_t)(pb0 >> 32) ^ b3 ^ k1;
    a0 = na0; a1 = (uint32_t)pa1; a2 = na2; a3 = (uint32_t)pa0;
    b0 = nb0; b1 = (uint32_t)pb1; b2 = nb2; b3 = (uint32_t)pb0;
  }
  *out_a = make_uint4(a0, a1, a2, a3);
  *out_b = make_uint4(b0, b1, b2, b3);
}

// four blocks with consecutive counters ctr, ctr + 1, ctr + 2, ctr + 3 (same last two counter words), round by round
__device__ __forceinline__ void philox4x32_10_x4(uint64_t ctr, uint32_t c2, uint32_t c3, const PhiloxKey& key, uint4* out) {
  uint32_t s0[4], s1[4], s2[4], s3[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint64_t c = ctr + (uint64_t)j;
    s0[j] = (uint32_t)c; s1[j] = (uint32_t)(c >> 32); s2[j] = c2; s3[j] = c3;
  }
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t k0 = key.k0[r], k1 = key.k1[r];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)s0[j], p1 = (uint64_t)0xCD9E8D57u * (uint64_t)s2[j];
      const uint32_t n0 = (uint32_t)(p1 >> 32) ^ s1[j] ^ k0, n2 = (uint32_t)(p0 >> 32) ^ s3[j] ^ k1;
      s0[j] = n0; s1[j] = (uint32_t)p1; s2[j] = n2; s3[j] = (uint32_t)p0;
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) out[j] = make_uint4(s0[j], s1[j], s2[j], s3[j]);
}

// ---- Definition 1 for one normalized coordinate, every operation one IEEE rounding ----------
// returns the level index; lev points to the table in shared memory
__device__ __forceinline__ int quantize_level(float absv, float norm, const float* lev, int nlev, uint32_t word) {
  float u = (norm > 0.0f) ? __fdiv_rn(absv, norm) : 0.0f;
  u = fminf(u, 1.0f);
  int tau = 0;
  for (int j = 1; j <= nlev - 2; ++j) tau = (lev[j] <= u) ? j : tau;
  const float num = __fsub_rn(u, lev[tau]);
  const float den = __fsub_rn(lev[tau + 1], lev[tau]);
  const float xi = __fdiv_rn(num, den);
  const float r = __fmul_rn(__uint2float_rn(word >> 8), 5.9604644775390625e-8f);   // exact
  return tau + ((r < xi) ? 1 : 0);
}

// The exact routine as one out-of-line copy (it runs for about 1e-5 of the coordinates).
static __device__ __noinline__ int quantize_level_slow(float absv, float norm, const float* lev, int nlev, uint32_t word) {
  return quantize_level(absv, norm, lev, nlev, word);
}

// ---- rounding through the level map -----------------------------------------------------------
// F(u) = tau + (u - l_tau) / (l_{tau+1} - l_tau) is continuous and piecewise linear, and Definition 1
// rounds u to level floor(F(u) - r) + 1 (r the uniform variate) unless F(u) - r is an integer.  The
// kernels evaluate S F(u) with S = 2^19 (2^18 above 17 levels) from a table over the float pattern
// of u2 = |v| RN(1 / norm) + 2^-16 (64 bins per octave, every bin holding at most one level: the lower
// piece plus a slope change past that level), subtract S r, and read the level index off the mantissa
// after adding 1.5 * 2^23 * S.  Whenever S (F - r) comes closer than `margin` to a multiple of S the
// exact routine decides instead; the margin (see make_round_table) covers the difference between u2 and
// the exact quotient, the table's roundings and the three fused multiply-adds.
constexpr float kRoundShift = 1.52587890625e-05f;       // 2^-16: keeps u2 inside the table
struct RoundTable {
  int nlev;
  int usable;                            // 0: some bin holds two levels, or the margin is too wide
  int key_shift;                         // layout of the bin table: kKeyShiftMin..kKeyShiftMax
  float thr;                             // S / 2 - margin
  float neg_qscale;                      // -S / 2^23
  float magic;                           // 1.5 * 2^23 * S
  float a[QGX_MAX_LEVELS];               // per interval: S tau - b (l_tau + 2^-16) + 1.5 S
  float b[QGX_MAX_LEVELS];               //               S / (l_{tau+1} - l_tau)
  float knot[QGX_MAX_LEVELS];            // l_j + 2^-16 for interior levels j, else a value never reached
  float db[QGX_MAX_LEVELS];              // b[j] - b[j - 1]
  // the same map for the octet encoder, which subtracts only the leading 16 bits h of the variate (as the float
  // 2^23 + h) and leaves the rest to the exact routine:
  float a16[QGX_MAX_LEVELS];             // S tau - b (l_tau + 2^-16) + S / 2 - S 2^-17 + 2^23 S 2^-16
  float thr16;                           // S / 2 - (margin + what the dropped variate bits can move)
  float neg_qscale16;                    // -S / 2^16
};

// one entry per bin and copy: {a (or a16), b, knot, db} of the interval of the bin's lowest value
__device__ __forceinline__ void fill_bin_table(float4* bin, const RoundTable& rt, bool octet_encoder = false) {
  const int rep_log = rt.key_shift - kKeyShiftMin;
  const int nbins = (int)((kKeyTop - kKeyBase) >> rt.key_shift) + 1;
  for (int i = threadIdx.x; i < (nbins << rep_log); i += blockDim.x) {
    const uint32_t b = (uint32_t)(i >> rep_log);
    const float lo = __uint_as_float(kKeyBase + (b << rt.key_shift));
    const float hi = __uint_as_float(kKeyBase + ((b + 1u) << rt.key_shift) - 1u);
    int t0 = 0;
    for (int j = 1; j <= rt.nlev - 2; ++j) t0 = (rt.knot[j] <= lo) ? j : t0;
    const bool straddle = (t0 + 1 <= rt.nlev - 2) && (rt.knot[t0 + 1] <= hi);
    bin[i] = make_float4(octet_encoder ? rt.a16[t0] : rt.a[t0], rt.b[t0], straddle ? rt.knot[t0 + 1] : 4.0f, straddle ? rt.db[t0 + 1] : 0.0f);
  }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

struct RoundConsts {
  float rn;                              // RN(1 / norm)
  float thr;                             // negative: every coordinate goes to the exact routine
  float neg_qscale, magic;
  uint32_t bin_mask;                     // keeps the bin part of pattern >> kBinAddrShift
  uint32_t bin_lane;                     // byte offset of this lane's copy inside a bin
};

__device__ __forceinline__ RoundConsts round_consts(const RoundTable& rt, float norm) {
  const bool ok = rt.usable && norm > 7.9e-31f && norm < 1.2e30f;
  RoundConsts c;
  c.rn = ok ? __frcp_rn(norm) : 0.0f;
  c.thr = ok ? rt.thr : -1.0f;
  c.neg_qscale = rt.neg_qscale;
  c.magic = rt.magic;
  const uint32_t copy_bytes = 16u << (rt.key_shift - kKeyShiftMin);
  c.bin_mask = ~(copy_bytes - 1u);
  c.bin_lane = ((threadIdx.x & 31u) << 4) & (copy_bytes - 1u);
  return c;
}

// pattern of the float whose low mantissa bits are the level index; *unsafe: ask the exact routine
__device__ __forceinline__ uint32_t round_fast(float absv, const RoundConsts& c, const float4* bin, uint32_t word, bool* unsafe) {
  const float u2 = fminf(fmaf(absv, c.rn, kRoundShift), 1.0f + kRoundShift);   // a supplied norm may be smaller than |v|
  const uint32_t off = ((__float_as_uint(u2) >> kBinAddrShift) & c.bin_mask) | c.bin_lane;
  const float4 e = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(bin) + off - kBinAddrBase);
  float X = fmaf(u2, e.y, e.x);
  X = fmaf(__saturatef(__fsub_rn(u2, e.z)), e.w, X);
  const float mb = __uint_as_float(0x4B000000u | (word >> 9));                    // 2^23 + (m >> 1), exact
  const float D = fmaf(mb, c.neg_qscale, X);                                       // S (F - r) + S / 2
  const float Z = __fadd_rn(D, c.magic);
  const float rho = __fsub_rn(D, __fsub_rn(Z, c.magic));                            // D minus the nearest multiple of S
  *unsafe = fabsf(rho) > c.thr;
  return __float_as_uint(Z);
}

// The four coordinates of a quad as 6-bit codes, one per byte: level index, bit 5 the sign of a
// nonzero level.
__device__ __forceinline__ uint32_t quantize_quad_codes(const float4 x, const uint4 w, const RoundConsts& c, float norm,
                                                        const float4* bin, const float* lev, int nlev) {
  bool u0, u1, u2, u3;
  const uint32_t z0 = round_fast(fabsf(x.x), c, bin, w.x, &u0);
  const uint32_t z1 = round_fast(fabsf(x.y), c, bin, w.y, &u1);
  const uint32_t z2 = round_fast(fabsf(x.z), c, bin, w.z, &u2);
  const uint32_t z3 = round_fast(fabsf(x.w), c, bin, w.w, &u3);
  uint32_t idx4 = prmt(prmt(z0, z1, 0x0040u), prmt(z2, z3, 0x0040u), 0x5410u);    // the low bytes
  if (u0 | u1 | u2 | u3) {
    uint32_t i0 = idx4 & 0xffu, i1 = (idx4 >> 8) & 0xffu, i2 = (idx4 >> 16) & 0xffu, i3 = idx4 >> 24;
    if (u0) i0 = (uint32_t)quantize_level_slow(fabsf(x.x), norm, lev, nlev, w.x);
    if (u1) i1 = (uint32_t)quantize_level_slow(fabsf(x.y), norm, lev, nlev, w.y);
    if (u2) i2 = (uint32_t)quantize_level_slow(fabsf(x.z), norm, lev, nlev, w.z);
    if (u3) i3 = (uint32_t)quantize_level_slow(fabsf(x.w), norm, lev, nlev, w.w);
    idx4 = i0 | (i1 << 8) | (i2 << 16) | (i3 << 24);
  }
  // sign bytes (0x00 / 0xff) of the four floats, kept at bit 5 where the level is not zero
  const uint32_t s4 = prmt(prmt(__float_as_uint(x.x), __float_as_uint(x.y), 0x00fbu),
                           prmt(__float_as_uint(x.z), __float_as_uint(x.w), 0x00fbu), 0x5410u);
  const uint32_t nz = (idx4 + 0x1f1f1f1fu) & 0x20202020u;                          // level indices are < 0x20
  return idx4 | (s4 & nz);
}

// ---- the octet encoder's rounding ---------------------------------------------------------------
// The variate of coordinate i is r = (w >> 8) 2^-24, w = word (i & 3) of the Philox block with counter
// (i >> 2, worker, exchange).  The fast path uses only the leading 16 bits h of r (the centre of the interval of r
// they leave) and sends a coordinate to the exact routine when the outcome could depend on the remaining bits.
// Shared memory by 32-bit address (what ld.shared takes): the hot loops compute table addresses themselves.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// read-only tables: the address depends on the data just loaded, so the compiler cannot move these too early
__device__ __forceinline__ float4 lds_table128(uint32_t addr) {
  float4 v;
  asm("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_table32(uint32_t addr) {
  uint32_t v;
  asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
// data that other threads or copies write: ordered with the barriers around them
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }

struct RoundK {
  float rn;                              // RN(1 / norm)
  float thr;                             // negative: every coordinate goes to the exact routine
  float nqs, magic;
  uint32_t bin_mask;                     // clears the bits of pattern >> kBinAddrShift below a bin's copies
  uint32_t bin_base;                     // shared address of the bin table (128-byte aligned) minus kBinAddrBase
  uint32_t bin_lane;                     // byte offset of this lane's copy inside a bin
};

// bin = the bin table (entries with a16) in shared memory, aligned to 128 bytes
__device__ __forceinline__ RoundK round_k(const RoundTable& rt, float norm, const float4* bin) {
  const bool ok = rt.usable && norm > 7.9e-31f && norm < 1.2e30f;
  RoundK c;
  c.rn = ok ? __frcp_rn(norm) : 0.0f;
  c.thr = ok ? rt.thr16 : -1.0f;
  c.nqs = rt.neg_qscale16;
  c.magic = rt.magic;
  const uint32_t copy_bytes = 16u << (rt.key_shift - kKeyShiftMin);
  c.bin_mask = ~(copy_bytes - 1u);
  c.bin_base = smem_addr(bin) - kBinAddrBase;           // a multiple of 128, like a bin's copies together
  c.bin_lane = ((threadIdx.x & 31u) << 4) & (copy_bytes - 1u);
  return c;
}

// One coordinate: returns S * (signed level index) as a float (the level of x, negative for negative x) and raises
// *worst to the distance of S (F - r~) + S / 2 from that multiple of S: above c.thr the exact routine has to decide.
// hbits = pattern of the float 2^23 + h.
__device__ __forceinline__ float round_signed(float x, uint32_t hbits, const RoundK& c, float* worst) {
  const float u2 = fmaf(fabsf(x), c.rn, kRoundShift);
  // pattern >> 13 as the high word of pattern * 2^19, the table's address added in the same multiply-add
  const float4 e = lds_table128(((__umulhi(__float_as_uint(u2), 1u << (32 - kBinAddrShift)) + c.bin_base) & c.bin_mask) | c.bin_lane);
  const float t1 = fmaf(__uint_as_float(hbits), c.nqs, e.x);                       // exact: both are multiples of S 2^-16
  float X = fmaf(u2, e.y, t1);
  X = fmaf(__saturatef(__fsub_rn(u2, e.z)), e.w, X);                               // S (F - r~) + S / 2
  const float sg = __uint_as_float((__float_as_uint(x) & 0x80000000u) | 0x3f800000u);
  const float Z = fmaf(X, sg, c.magic);
  const float zi = __fsub_rn(Z, c.magic);                                          // the nearest multiple of S, signed
  const float rho = fmaf(X, sg, -zi);
  *worst = fmaxf(*worst, fabsf(rho));
  return zi;
}

// The 24 variate bits of coordinate e (its index in the generator's counter space) on their own: a whole block
// per call, for ragged ends only.
static __device__ __noinline__ uint32_t variate_bits(uint64_t e, uint32_t k, uint32_t xid, const PhiloxKey& key) {
  const uint64_t q = e >> 2;
  const uint4 w = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), k, xid, key);
  const int c = (int)(e & 3u);
  return (c == 0 ? w.x : (c == 1 ? w.y : (c == 2 ? w.z : w.w))) >> 8;
}

// Definition 1 for one coordinate, every operation one IEEE rounding; r24 = the 24-bit variate.  Out of line: it
// runs for about 1e-4 of the coordinates.
static __device__ __noinline__ int quantize_level_exact(float absv, float norm, const float* lev, int nlev, uint32_t r24) {
  float u = (norm > 0.0f) ? __fdiv_rn(absv, norm) : 0.0f;
  u = fminf(u, 1.0f);
  int tau = 0;
  for (int j = 1; j <= nlev - 2; ++j) tau = (lev[j] <= u) ? j : tau;
  const float num = __fsub_rn(u, lev[tau]);
  const float den = __fsub_rn(lev[tau + 1], lev[tau]);
  const float xi = __fdiv_rn(num, den);
  const float r = __fmul_rn(__uint2float_rn(r24), 5.9604644775390625e-8f);        // exact
  return tau + ((r < xi) ? 1 : 0);
}

__device__ __forceinline__ uint32_t symbol_of(float v, int idx) {
  const uint32_t neg = (__float_as_uint(v) >> 31) & (idx != 0 ? 1u : 0u);
  return (uint32_t)idx | (neg << 7);
}

__device__ __forceinline__ float dequantize_symbol(uint32_t sym, float norm, const float* lev) {
  const float val = __fmul_rn(norm, lev[sym & 31u]);
  return __uint_as_float(__float_as_uint(val) ^ ((sym & 0x80u) << 24));
}

// ---- reductions ------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t x, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  return x;
}

// optional state update fused into the decode epilogue of an exchange
struct ExchangeUpdate {
  int mode;                      // 0 none, 1: xout = xin - gamma * mean, 2: xout = xin - mean
  const float* xin;
  float* xout;
  const double* scalars;         // scalars[1] = gamma_t
};

// host side
qgx_status check_levels_host(const float* lev, int nlev);
qgx_status make_code_table(const qgx_codebook* cb, int bucket, CodeTable* out);
void make_round_table(const float* lev, int nlev, RoundTable* out);
void* ws_get(qgx_ctx* c, int which, size_t bytes);          // nullptr on failure
void free_table_cache(qgx_ctx* c);
void free_seg_children(qgx_ctx* c);
uint64_t seg_children_launches(const qgx_ctx* c);
qgx_status cuda_status(cudaError_t e);
inline void count_launch(qgx_ctx* c, int n = 1) { c->launches += (uint64_t)n; }

// Brackets an instrumented kernel launch with two events when timing is on (qgx_timing_enable).
struct ScopedKernelTimer {
  qgx_ctx* c;
  int slot;
  ScopedKernelTimer(qgx_ctx* ctx, int kind) : c(ctx), slot(-1) {
    if (c->timing_on && c->timing_used < c->timing_cap) {
      slot = c->timing_used++;
      c->timing_kind[slot] = kind;
      cudaEventRecord(c->timing_ev[2 * slot], c->stream);
    }
  }
  ~ScopedKernelTimer() {
    if (slot >= 0) cudaEventRecord(c->timing_ev[2 * slot + 1], c->stream);
  }
};

}  // namespace qgx
