// The fused quantize + encode pass for whole buckets of a multiple of 1024 coordinates (the layout of every large
// configuration).  One CTA per SM, two teams of 16 warps, three stage buffers of 16384 coordinates in shared
// memory: while each team works on the bucket (or group of smaller buckets) in its buffer, bulk tensor copies
// (TMA) fill the third buffer with the group that the team finishing first takes next, so the dual vectors stream
// in throughout and no registers are tied up while they are in flight.  A lane owns 32 consecutive coordinates
// (one 128-byte line of the stage), a warp 1024, a bucket bucket / 1024 warps of a team.  Every warp packs its
// bits into a region of its own -- inside the part of the stage that only this warp reads, once it has read it --
// so a team synchronises three times per group: the norm, "all regions complete", and "copied out".  The
// copy-out shifts each region to its place in the bucket's stream, which is where the warps' bit counts first meet.
//
// Included by qgx_exchange.cu (uses its status words, look-back and EncodeArgs).
#pragma once

namespace qgx {

constexpr int kTeamThreads = 512;
constexpr int kStagedWarps = kTeamThreads / 32;          // warps of a team
constexpr int kStagedThreads = 2 * kTeamThreads;         // two teams
constexpr int kStageBuffers = 3;
constexpr int kLaneCoords = 32;                          // coordinates per lane: one 128-byte line
constexpr int kWarpCoords = 32 * kLaneCoords;
constexpr int kStageCoords = kStagedWarps * kWarpCoords; // 16384

// float index, inside a bucket's stage, of 16-byte chunk c (0..7) of line `line`: the chunks of a line are permuted
// by the line number (the 128-byte swizzle of the bulk tensor copies that fill the stage), so that lanes reading
// the same chunk of 8 consecutive lines hit different bank groups
__device__ __forceinline__ int stage_at(int line, int c) { return line * kLaneCoords + ((c ^ (line & 7)) << 2); }

// the four pair-table entries of an octet -> its stream bits m[0..3] (at most 104) and their count
__device__ __forceinline__ void merge_octet(uint32_t e0, uint32_t e1, uint32_t e2, uint32_t e3, uint32_t* m, uint32_t* n) {
  const uint32_t b0 = e0 & 0x3ffffffu, n0 = e0 >> 26, b1 = e1 & 0x3ffffffu, n1 = e1 >> 26;
  const uint32_t b2 = e2 & 0x3ffffffu, n2 = e2 >> 26, b3 = e3 & 0x3ffffffu, n3 = e3 >> 26;
  const uint64_t A = (uint64_t)b0 | ((uint64_t)b1 << n0);            // at most 52 bits
  const uint64_t B = (uint64_t)b2 | ((uint64_t)b3 << n2);
  const uint32_t nA = n0 + n1;
  const uint64_t lo = A | (B << nA);
  const uint64_t hi = (B >> 1) >> (63u - nA);                        // the bits of B past bit 63 (none when nA == 0)
  m[0] = (uint32_t)lo; m[1] = (uint32_t)(lo >> 32); m[2] = (uint32_t)hi; m[3] = (uint32_t)(hi >> 32);
  *n = nA + n2 + n3;
}

// Appends the n (8..104) bits m[0..3] to a lane's run of bits in the region at shared address R: full words are
// stored, the partial word stays in carry (nc < 32 bits of it valid).  wa = shared address of the word that carry
// will become.
__device__ __forceinline__ void append_bits(uint32_t& wa, uint32_t& nc, uint32_t& carry, const uint32_t* m, uint32_t n) {
  const uint32_t s0 = carry | (m[0] << nc);
  const uint32_t s1 = __funnelshift_l(m[0], m[1], nc);
  const uint32_t s2 = __funnelshift_l(m[1], m[2], nc);
  const uint32_t s3 = __funnelshift_l(m[2], m[3], nc);
  const uint32_t s4 = __funnelshift_l(m[3], 0u, nc);
  const uint32_t tot = nc + n;
  const uint32_t nfull = tot >> 5;                                   // 0..4
  const bool p0 = nfull > 0u, p1 = nfull > 1u, p2 = nfull > 2u, p3 = nfull > 3u;
  if (p0) sts32(wa, s0);
  if (p1) sts32(wa + 4u, s1);
  if (p2) sts32(wa + 8u, s2);
  if (p3) sts32(wa + 12u, s3);
  carry = p3 ? s4 : (p2 ? s3 : (p1 ? s2 : (p0 ? s1 : s0)));
  wa += nfull << 2;
  nc = tot & 31u;
}

// ---- the pieces of the ring: a barrier per buffer that completes when its copies have landed, a barrier per team ----
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(count) : "memory");
}
// one arrival that also announces `bytes` of bulk copies, which complete the phase when they have landed
__device__ __forceinline__ void mbar_arrive_expect(unsigned long long* bar, unsigned bytes) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }"
               ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(bytes) : "memory");
}
// Bulk tensor copy (TMA) of one box of the map -- 128-byte rows, the 16-byte chunks of row r stored permuted by
// r & 7 (the 128-byte swizzle) -- from row `row` on, into shared memory at dst (1024-byte aligned).
__device__ __forceinline__ void tma_load_rows(void* dst, const CUtensorMap* map, int row, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(reinterpret_cast<unsigned long long>(map)), "r"(0), "r"(row),
                 "r"((unsigned)__cvta_generic_to_shared(bar)) : "memory");
}
// orders this thread's earlier accesses to shared memory before later bulk copies into it
__device__ __forceinline__ void fence_before_bulk_copy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Waits (one lane polls for its warp, backing off) for the phase of the given parity to complete; false if the
// bounded wait ran out.  Called by whole warps.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity) {
  const unsigned addr = (unsigned)__cvta_generic_to_shared(bar);
  unsigned done = 0;
  if ((threadIdx.x & 31u) == 0) {
    for (int spin = 0; spin < kSpinLimit && !done; ++spin) {
      asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                   : "=r"(done) : "r"(addr), "r"(parity) : "memory");
      if (!done && spin > 4) __nanosleep(100);
    }
  }
  done = __shfl_sync(0xffffffffu, done, 0);
  if (done) {                                           // every lane observes the completed phase itself (and its data)
    unsigned again;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(again) : "r"(addr), "r"(parity) : "memory");
    done = again;
  }
  return __all_sync(0xffffffffu, done != 0);
}
__device__ __forceinline__ void team_sync(int team) {
  asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(kTeamThreads) : "memory");
}

// where a warp keeps the 16-bit lengths of its sub-blocks: inside its part of the stage, past its region
constexpr int kWarpHdrWord = 420;                        // a region has at most 1024 * 13 / 32 + 1 = 417 words

// One segment of a bucket's stream for the copy-out: a region (shared address R) of T valid bits that starts at
// bit s of the bucket.
struct Segment {
  uint32_t R;
  uint32_t s, T;
};

// Stores the words of the bucket's stream whose first bit lies in `seg` (the last of them, when it runs past the
// segment's end, takes its remaining bits from the first word of the following region, at shared address next_R
// or 0 for none; every following segment has >= 32 bits).
__device__ __forceinline__ void copy_segment(const Segment seg, uint32_t next_R, uint32_t* dst, int lane) {
  const uint32_t m_lo = (seg.s + 31u) >> 5, m_hi = (seg.s + seg.T + 31u) >> 5;
  const uint32_t q0 = (m_lo << 5) - seg.s;                           // the region's bit that the first word starts at: 0..31
  const uint32_t nw = (seg.T + 31u) >> 5;
  const uint32_t count = m_hi - m_lo;
  const uint32_t tail = (seg.T - q0) & 31u;                          // valid bits of the last word (0: all 32)
  for (uint32_t j = (uint32_t)lane; j < count; j += 32u) {
    const uint32_t lo = lds32(seg.R + 4u * j);
    const uint32_t hi = (j + 1u < nw) ? lds32(seg.R + 4u * j + 4u) : 0u;
    uint32_t v = __funnelshift_r(lo, hi, q0);
    if (j + 1u == count && tail != 0u) {
      v &= (1u << tail) - 1u;
      if (next_R != 0u) v |= lds32(next_R) << tail;
    }
    dst[m_lo + j] = v;
  }
}

// Buckets [0, a.nb_whole) of every worker; G coordinates per sub-block; a.bucket a multiple of 1024 that divides
// 16384; all sources 16-byte aligned, the workers' rows a multiple of 32 floats apart, and the vector's first
// coordinate a multiple of 8 in the generator's counter space (the host checks).  tmap: the staged source as rows
// of 32 floats.  Buckets are taken in the order b-major, k-minor, 16384 / bucket at a time; group g belongs to CTA
// g mod gridDim.x, which works on its groups in increasing order (its n-th group by team n & 1 in buffer n % 3).
// The launch is cooperative, so all CTAs are resident whatever else runs on the device, and they advance at the
// same pace: the buckets a bucket looks back at (the same worker's earlier buckets, which lie in groups before
// its own) have usually been counted when it asks.  A bucket waits
// only for buckets of smaller groups, and a group that is staged but not started waits only for its own team's
// current group, which is smaller: the smallest unfinished group is always being worked on and waits for
// nothing, so every wait ends.
template <int G>
__global__ void __launch_bounds__(kStagedThreads, 1)
k_encode_staged(const __grid_constant__ EncodeArgs a, const __grid_constant__ LevelTable lt, const __grid_constant__ CodeTable ct,
                const __grid_constant__ PhiloxKey key, const __grid_constant__ RoundTable rt, const __grid_constant__ CUtensorMap tmap) {
  extern __shared__ __align__(1024) float s_stage[];                 // kStageBuffers * kStageCoords floats
  __shared__ __align__(128) float4 s_bin[kBinEntries];
  __shared__ uint32_t s_pair[kPairLutSize];
  __shared__ EncLut s_lut;
  __shared__ float s_lev[QGX_MAX_LEVELS];
  __shared__ double s_red[2 * kStagedWarps];
  __shared__ uint32_t s_tot[2 * kStagedWarps];
  __shared__ uint32_t s_pre[2 * kStagedWarps];                        // bits of the bucket's warps before this one
  __shared__ unsigned long long s_bk[kStageBuffers][kStagedWarps];   // bucket of a buffer's slot: b | k << 48, or ~0
  __shared__ unsigned int s_cnt[2 * kStagedWarps];                    // warps of a bucket that have their bit count
  __shared__ unsigned long long s_base[2 * kStagedWarps];             // word offset of the bucket in its worker's stream
  __shared__ int s_skip[2 * kStagedWarps];
  __shared__ unsigned int s_group[kStageBuffers];                     // the group whose data a buffer holds
  __shared__ unsigned int s_next[2];                                  // the group a team has drawn for the buffer it frees
  __shared__ __align__(8) unsigned long long s_full[kStageBuffers];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int team = warp / kStagedWarps, tw = warp - team * kStagedWarps;
  const int wpb = a.bucket / kWarpCoords;                             // warps per bucket: 1, 2, 4, 8 or 16
  const int M = kStagedWarps / wpb;                                   // buckets per group
  const int slot = tw / wpb, wis = tw - slot * wpb;                   // this warp's bucket of the group, its place in it
  const int gslot = team * kStagedWarps + slot;                       // index of the bucket's shared variables
  const int line = wis * 32 + lane;                                   // this lane's line of the bucket
  const int bthreads = 32 * wpb;
  const int spb = a.bucket / G;                                       // sub-blocks per bucket
  constexpr int kSubPerWarp = kWarpCoords / G;                        // 32, 16 or 8
  const uint32_t hdr_bits = kNormBits + 16u * (uint32_t)spb;          // a whole number of words: spb is even
  const uint32_t hdr_words = hdr_bits >> 5;

  fill_enc_lut(&s_lut, ct);
  fill_bin_table(s_bin, rt, true);
  if (tid < QGX_MAX_LEVELS) s_lev[tid] = tid < lt.nlev ? lt.lev[tid] : 1.0f;
  if (tid < 2 * kStagedWarps) s_cnt[tid] = 0u;
  if (tid == 0) {
    for (int i = 0; i < kStageBuffers; ++i) {
      mbar_init(&s_full[i], 1);
      s_group[i] = blockIdx.x + (unsigned)i * gridDim.x;              // the CTA's first three groups
    }
  }
  __syncthreads();
  fill_pair_lut_signed(s_pair, &s_lut);
  __syncthreads();
  const int nlev = lt.nlev;
  const uint32_t pair_sa = smem_addr(s_pair), stage_sa = smem_addr(s_stage);
  const float S = -rt.neg_qscale16 * 65536.0f, four_over_S = 4.0f / S;
  const size_t ld = a.src.ld ? a.src.ld : a.d;
  const unsigned long long total = (unsigned long long)a.nb_whole * (unsigned long long)a.K;
  const unsigned long long ngroups = (total + (unsigned long long)M - 1ull) / (unsigned long long)M;
  const bool two = a.src.v && a.src.a;

  // Starts the bulk copies of group g into buffer `buf` (one thread for the team) and arrives on the buffer's
  // barrier, whose phase completes when the bytes have landed; records which group the buffer holds.
  const int box_rows = min(256, a.bucket / kLaneCoords);
  auto issue_load = [&](int buf, unsigned long long g) {
    s_group[buf] = (unsigned int)min(g, (unsigned long long)0xffffffffu);
    const unsigned long long t0 = g * (unsigned long long)M;
    const int nslots = g < ngroups ? (int)min((unsigned long long)M, total - t0) : 0;
    for (int sl = 0; sl < M; ++sl) {
      const unsigned long long t = t0 + (unsigned long long)sl;
      s_bk[buf][sl] = sl < nslots ? ((t / (unsigned long long)a.K) | ((t % (unsigned long long)a.K) << 48)) : ~0ull;
    }
    mbar_arrive_expect(&s_full[buf], (unsigned)nslots * (unsigned)a.bucket * 4u);
    for (int sl = 0; sl < nslots; ++sl) {
      const unsigned long long bk = s_bk[buf][sl];
      const size_t bb = (size_t)(bk & 0xffffffffffffull), kk = (size_t)(bk >> 48);
      const size_t first = (a.src.v ? kk * ld : 0) + bb * (size_t)a.bucket;         // in floats from the map's base
      for (int r0 = 0; r0 < a.bucket / kLaneCoords; r0 += box_rows)
        tma_load_rows(s_stage + buf * kStageCoords + sl * a.bucket + r0 * kLaneCoords, &tmap, (int)(first / kLaneCoords) + r0, &s_full[buf]);
    }
  };
  const bool loader = (tid & (kTeamThreads - 1)) == 0;                // the thread of a team that starts its copies
  if ((reinterpret_cast<uintptr_t>(s_stage) & 1023u) != 0) {          // the swizzle assumes this alignment
    if (tid == 0) latch_error(a.st, QGX_ERR_CUDA);
    return;
  }
  // team 0 starts with the CTA's groups 0 and 2, team 1 with group 1
  if (loader) {
    issue_load(team, s_group[team]);
    if (team == 0) issue_load(2, s_group[2]);
  }

  for (unsigned n = (unsigned)team;; n += 2u) {
    const int buf = (int)(n % kStageBuffers);
    if (!mbar_wait(&s_full[buf], (n / kStageBuffers) & 1u) && lane == 0) latch_error(a.st, QGX_ERR_TIMEOUT);
    __syncwarp();
    const unsigned long long g = s_group[buf];
    if (g >= ngroups) {
      // out of groups: the other team, whose later buffer may still hold a group drawn earlier than this one,
      // finds the end marker in this buffer too when it comes round
      team_sync(team);                                                // every thread of the team has seen this phase complete
      if (loader) issue_load(buf, ngroups);
      break;
    }
    const unsigned long long bk = s_bk[buf][slot];
    const bool active = bk != ~0ull;
    const size_t b = active ? (size_t)(bk & 0xffffffffffffull) : 0, k = active ? (size_t)(bk >> 48) : 0;
    const size_t lo = b * (size_t)a.bucket;
    const uint32_t slot_sa = stage_sa + 4u * (uint32_t)(buf * kStageCoords + slot * a.bucket);    // the bucket's stage
    const uint32_t region = stage_sa + 4u * (uint32_t)(buf * kStageCoords + tw * kWarpCoords);    // the warp's part of it
    const uint32_t line_sa = slot_sa + 4u * (uint32_t)(line * kLaneCoords);

    // ---- partial norm over this thread's chunks (chunk line, line + bthreads, ...: a warp reads contiguous
    //      memory of the second source); with two sources the stage receives their combination ----
    double acc = 0.0;
    float mx = 0.0f;
    bool nan = false;
    if (active) {
      float4 av[8];
      if (two) {
#pragma unroll
        for (int r = 0; r < 8; ++r) av[r] = __ldg(reinterpret_cast<const float4*>(a.src.a + lo) + r * bthreads + line);
      }
      const uint32_t l3 = (uint32_t)line >> 3, l7 = (uint32_t)line & 7u, step = (uint32_t)bthreads >> 3;
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const uint32_t li = (uint32_t)r * step + l3;                  // chunk r * bthreads + line: chunk l7 of line li
        const uint32_t pa = slot_sa + (li << 7) + ((l7 ^ (li & 7u)) << 4);
        float4 x = lds128(pa);
        if (two) {
          x = dual_combine(av[r], x, a.src.mul);
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(pa), "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w) : "memory");
        }
        if (a.norm_type == QGX_NORM_L2) {
          const double x0 = x.x, x1 = x.y, x2 = x.z, x3 = x.w;
          acc = fma(x0, x0, acc); acc = fma(x1, x1, acc); acc = fma(x2, x2, acc); acc = fma(x3, x3, acc);
        } else {
          nan = nan || (x.x != x.x) || (x.y != x.y) || (x.z != x.z) || (x.w != x.w);
          mx = fmaxf(mx, fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w))));
        }
      }
    }
    if (a.norm_type == QGX_NORM_L2) {
      acc = warp_sum(acc);
    } else {
      mx = warp_max(mx);
      acc = __any_sync(0xffffffffu, nan) ? (double)__int_as_float(0x7fc00000) : (double)mx;
    }
    if (lane == 0) s_red[warp] = acc;
    team_sync(team);                                                  // the partial norms (and the combined vectors) are in
    float norm;
    {
      double v = lane < wpb ? s_red[team * kStagedWarps + slot * wpb + lane] : 0.0;
      if (a.norm_type == QGX_NORM_L2) {
        norm = (float)sqrt(warp_sum(v));
      } else {
        const bool bad = __any_sync(0xffffffffu, v != v);
        const float m2 = warp_max((float)v);
        norm = bad ? __int_as_float(0x7fc00000) : m2;
      }
    }
    const bool finite = (norm - norm) == 0.0f;
    const bool live = finite && norm != 0.0f;                         // otherwise every coordinate is level 0
    const RoundK rc = round_k(rt, norm, s_bin);

    // ---- rounding, pair codes and stream bits of this lane's 32 coordinates: four octets ----
    uint32_t mb[16];                                                  // the bits of the four octets, four words each
    uint32_t npack = 0, nbits_lane = 0;                               // their bit counts, a byte each, and the sum
    if (active) {
      const uint64_t oct0 = ((a.quad_base + (uint64_t)(lo >> 2)) >> 1) + 4ull * (uint64_t)line;
      const uint32_t l7 = (uint32_t)line & 7u;
      uint4 W[4];                                                     // the Philox blocks of two octets (four quads)
#pragma unroll
      for (int o = 0; o < 4; ++o) {
        float z[8];
        if (live) {
          if ((o & 1) == 0) philox4x32_10_x4(2ull * (oct0 + (uint64_t)o), (uint32_t)k, a.xid, key, W);
          const float4 xa = lds128(line_sa + (((uint32_t)(2 * o) ^ l7) << 4));
          const float4 xb = lds128(line_sa + (((uint32_t)(2 * o + 1) ^ l7) << 4));
          octet_levels_w(xa, xb, W[2 * (o & 1)], W[2 * (o & 1) + 1], rc, norm, S, s_lev, nlev, z);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) z[i] = 0.0f;
        }
        uint32_t n2;
        merge_octet(pair_entry(pair_sa, z[0], z[1], four_over_S), pair_entry(pair_sa, z[2], z[3], four_over_S),
                    pair_entry(pair_sa, z[4], z[5], four_over_S), pair_entry(pair_sa, z[6], z[7], four_over_S), &mb[4 * o], &n2);
        npack |= n2 << (8 * o);
        nbits_lane += n2;
      }
    }
    // bit offsets inside the warp's region, the warp's total; the warp that completes the bucket's bit count
    // publishes it straight away, for the buckets that will look back at this one
    const uint32_t incl = warp_incl_scan(nbits_lane, lane);
    const uint32_t warp_bits = __shfl_sync(0xffffffffu, incl, 31);
    bool last_of_bucket = false;
    if (lane == 0 && active) {
      s_tot[warp] = warp_bits;
      __threadfence_block();
      last_of_bucket = atomicAdd(&s_cnt[gslot], 1u) == (unsigned)(wpb - 1);
    }
    last_of_bucket = __shfl_sync(0xffffffffu, last_of_bucket ? 1 : 0, 0) != 0;
    unsigned long long* row = a.status + k * a.nb;
    uint32_t nbits = 0, nwords = 0;
    if (last_of_bucket) {
      const uint32_t mine = lane < wpb ? s_tot[team * kStagedWarps + slot * wpb + lane] : 0u;
      const uint32_t upto = warp_incl_scan(mine, lane);
      if (lane < wpb) s_pre[team * kStagedWarps + slot * wpb + lane] = upto - mine;
      nbits = hdr_bits + __shfl_sync(0xffffffffu, upto, 31);
      nwords = (nbits + 31u) >> 5;
      if (lane == 0) {
        st_status(row + b, kStAggregate | (unsigned long long)nwords);
        a.bucket_bits[k * a.nb + b] = nbits;
        atomicAdd(a.total_bits + k, (unsigned long long)nbits);
        a.norms[k * a.nb + b] = norm;
        if (!finite) latch_error(a.st, QGX_ERR_NONFINITE);
      }
    }
    __syncwarp();                                                     // every lane has read its line: the region may overwrite it

    // ---- the sub-block lengths, then this lane's bits, into the warp's part of the stage ----
    if (active) {
      constexpr int kSubLanes = G / kLaneCoords;                      // lanes per sub-block: 1, 2 or 4
      const uint32_t before = __shfl_up_sync(0xffffffffu, incl, kSubLanes);
      const uint32_t sub = incl - (lane >= kSubLanes ? before : 0u);
      if ((lane + 1) % kSubLanes == 0)
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(region + 4u * kWarpHdrWord + 2u * (uint32_t)(lane / kSubLanes)), "h"((uint16_t)sub) : "memory");
    }
    uint32_t wa = region + (((incl - nbits_lane) >> 5) << 2), nc = (incl - nbits_lane) & 31u, carry = 0u;
    const uint32_t wa0 = wa, nc0 = nc;
    if (active) {
#pragma unroll
      for (int o = 0; o < 4; ++o) append_bits(wa, nc, carry, &mb[4 * o], (npack >> (8 * o)) & 0xffu);
    }
    {
      // the first word of a lane's run also holds the last bits of the lane before it
      const uint32_t prev = __shfl_up_sync(0xffffffffu, carry, 1);
      if (active && lane > 0 && nc0 != 0u) sts32(wa0, lds32(wa0) | prev);
      if (active && lane == 31 && nc != 0u) sts32(wa, carry);
    }

    unsigned int next_group = 0;
    if (last_of_bucket) {                                             // where the bucket goes in its worker's stream
      bool timed_out = false;
      const unsigned long long excl = lookback_prefix(row, (long long)b, lane, a.spin_limit, &timed_out);
      if (lane == 0) {
        st_status(row + b, kStPrefix | (excl + (unsigned long long)nwords));
        int skip = 0;
        if (timed_out) { latch_error(a.st, QGX_ERR_TIMEOUT); skip = 1; }
        if (excl + nwords > (unsigned long long)a.cap_words) { latch_error(a.st, QGX_ERR_CAPACITY); skip = 1; }
        a.offsets[k * a.nb + b] = (uint32_t)min(excl, (unsigned long long)0xffffffffu);
        s_base[gslot] = excl;
        s_skip[gslot] = skip;
        s_cnt[gslot] = 0u;
        if (slot == 0) next_group = (unsigned int)min(g + 3ull * gridDim.x, (unsigned long long)0xffffffffu);   // this buffer's next group
      }
    }
    team_sync(team);                                                  // all regions and stream offsets are in

    // ---- copy out: the header (whole words) by the bucket's first warp, then every warp its own region ----
    if (active && !s_skip[gslot]) {
      uint32_t* dst = a.stream + k * a.cap_words + s_base[gslot];
      const uint32_t before = s_pre[warp];
      if (wis == 0) {
        for (uint32_t m = (uint32_t)lane; m < hdr_words; m += 32u) {
          uint32_t v = __float_as_uint(norm);
          if (m > 0u) {
            const uint32_t sb = 2u * (m - 1u);                        // the word's first sub-block
            const uint32_t wr = stage_sa + 4u * (uint32_t)(buf * kStageCoords + (slot * wpb + (int)(sb / kSubPerWarp)) * kWarpCoords);
            v = lds32(wr + 4u * (kWarpHdrWord + (sb % kSubPerWarp) / 2u));
          }
          dst[m] = v;
        }
      }
      const uint32_t next_R = wis + 1 < wpb ? region + 4u * kWarpCoords : 0u;
      copy_segment(Segment{region, hdr_bits + before, s_tot[warp]}, next_R, dst, lane);
    }
    if (last_of_bucket && slot == 0 && lane == 0) s_next[team] = next_group;
    fence_before_bulk_copy();
    team_sync(team);                                                  // the buffer may be overwritten

    // ---- refill the buffer with the group just drawn: the other team will find it there ----
    if (loader) issue_load(buf, s_next[team]);
  }
}

}  // namespace qgx
