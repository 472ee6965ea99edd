// Device pieces of the prefix codec (Sec. 3.2 / App. J) shared by the stand-alone and the fused
// kernels: packing a quad's codewords, placing bits into a shared-memory image of a bucket, and a
// bounded bit reader with a table-driven decoder.
#pragma once

#include "qgx_common.cuh"

namespace qgx {

// shared-memory copy of the per-level stream bits: entry = bits | nbits << 16, where bits holds
// the codeword in stream order followed by the sign bit for a negative nonzero level
struct EncLut {
  uint32_t e[2 * QGX_MAX_LEVELS];        // index: level | sign << 5
};

__device__ __forceinline__ void fill_enc_lut(EncLut* lut, const CodeTable& ct) {
  for (int i = threadIdx.x; i < 2 * QGX_MAX_LEVELS; i += blockDim.x) {
    const int idx = i & 31, neg = i >> 5;
    uint32_t bits = 0, n = 0;
    if (idx < ct.nlev) {
      n = ct.len[idx];
      bits = ct.rev[idx];
      if (idx != 0) { bits |= (uint32_t)neg << n; n += 1; }
    }
    lut->e[i] = bits | (n << 16);
  }
}

// stream bits of the four symbols of a quad, concatenated in coordinate order
__device__ __forceinline__ void pack_quad(uint32_t packed_syms, int nvalid, const EncLut* lut, uint64_t* bits, uint32_t* nbits) {
  uint64_t acc = 0;
  uint32_t n = 0;
#pragma unroll
  for (int c = 0; c < kQuad; ++c) {
    if (c < nvalid) {
      const uint32_t s = (packed_syms >> (8 * c)) & 0xffu;
      const uint32_t e = lut->e[(s & 31u) | ((s >> 7) << 5)];
      acc |= (uint64_t)(e & 0xffffu) << n;
      n += e >> 16;
    }
  }
  *bits = acc;
  *nbits = n;
}

// Pair table: the stream bits of two consecutive symbols in one entry, bits | nbits << 26, indexed by
// the two 6-bit symbol codes (level | sign << 5) as first | second << 6.
constexpr int kPairLutSize = 64 * 64;
__device__ __forceinline__ void fill_pair_lut(uint32_t* pair, const EncLut* lut) {
  for (int i = threadIdx.x; i < kPairLutSize; i += blockDim.x) {
    const uint32_t a = lut->e[i & 63], b = lut->e[i >> 6];
    const uint32_t na = a >> 16, nb = b >> 16;
    pair[i] = ((a & 0xffffu) | ((b & 0xffffu) << na)) | ((na + nb) << 26);
  }
}

// stream bits of a full quad of 6-bit codes (level | sign << 5, one per byte) through the pair table
__device__ __forceinline__ void pack_quad_codes(uint32_t t, const uint32_t* pair, uint64_t* bits, uint32_t* nbits) {
  const uint32_t e01 = pair[(t & 0x3fu) | ((t >> 2) & 0xfc0u)];
  const uint32_t e23 = pair[((t >> 16) & 0x3fu) | ((t >> 18) & 0xfc0u)];
  const uint32_t b01 = e01 & 0x3ffffffu, n01 = e01 >> 26, b23 = e23 & 0x3ffffffu, n23 = e23 >> 26;
  const uint32_t lo = b01 | (b23 << n01);
  const uint32_t hi = __funnelshift_l(b23, 0u, n01);
  *bits = ((uint64_t)hi << 32) | lo;
  *nbits = n01 + n23;
}
// Pair table of the octet encoder: indexed by (first + 64 * second) mod 4096, first and second the signed level
// indices (negative for a negative coordinate) of two consecutive coordinates -- the low 12 bits of that sum as
// a two's complement number, which is how it comes out of the float arithmetic of the rounding.
__device__ __forceinline__ void fill_pair_lut_signed(uint32_t* pair, const EncLut* lut) {
  for (int i = threadIdx.x; i < kPairLutSize; i += blockDim.x) {
    const int lo6 = i & 63;
    const int first = lo6 >= 32 ? lo6 - 64 : lo6;
    const int hi6 = ((i - first) >> 6) & 63;
    const int second = hi6 >= 32 ? hi6 - 64 : hi6;
    const uint32_t a = lut->e[((first < 0 ? -first : first) & 31) | (first < 0 ? 32 : 0)];
    const uint32_t b = lut->e[((second < 0 ? -second : second) & 31) | (second < 0 ? 32 : 0)];
    const uint32_t na = a >> 16, nb = b >> 16;
    pair[i] = ((a & 0xffffu) | ((b & 0xffffu) << na)) | ((na + nb) << 26);
  }
}

// stream bits of four consecutive coordinates from their two pair-table entries
__device__ __forceinline__ void pack_pair_entries(uint32_t e01, uint32_t e23, uint64_t* bits, uint32_t* nbits) {
  const uint32_t b01 = e01 & 0x3ffffffu, n01 = e01 >> 26, b23 = e23 & 0x3ffffffu, n23 = e23 >> 26;
  const uint32_t lo = b01 | (b23 << n01);
  const uint32_t hi = __funnelshift_l(b23, 0u, n01);
  *bits = ((uint64_t)hi << 32) | lo;
  *nbits = n01 + n23;
}

// OR `nbits` (<= 52) bits into the bucket image at bit position pos (shared memory, zeroed before).
// Two words are always touched; a third only when the bits reach it.
__device__ __forceinline__ void put_bits(uint32_t* img, uint32_t pos, uint64_t bits, uint32_t nbits) {
  const uint32_t w = pos >> 5, sh = pos & 31u;
  const uint32_t blo = (uint32_t)bits, bhi = (uint32_t)(bits >> 32);
  atomicOr(&img[w], blo << sh);
  atomicOr(&img[w + 1], __funnelshift_l(blo, bhi, sh));
  if (sh + nbits > 64u) atomicOr(&img[w + 2], __funnelshift_l(bhi, 0u, sh));
}

// Two adjacent runs (a first, then b; each <= 52 bits) as one value of up to 104 bits.  Two words are
// always touched, further ones only when the bits reach them.
__device__ __forceinline__ void put_bits2(uint32_t* img, uint32_t pos, uint64_t a, uint32_t na, uint64_t b, uint32_t nb) {
  const uint64_t lo = a | (b << na);
  const uint64_t hi = (b >> 1) >> (63u - na);           // the bits of b past bit 63 (none when na == 0)
  const uint32_t n = na + nb;
  const uint32_t w = pos >> 5, sh = pos & 31u;
  const uint32_t m0 = (uint32_t)lo, m1 = (uint32_t)(lo >> 32), m2 = (uint32_t)hi, m3 = (uint32_t)(hi >> 32);
  atomicOr(&img[w], m0 << sh);
  atomicOr(&img[w + 1], __funnelshift_l(m0, m1, sh));
  if (sh + n > 64u) {
    atomicOr(&img[w + 2], __funnelshift_l(m1, m2, sh));
    if (sh + n > 96u) {
      atomicOr(&img[w + 3], __funnelshift_l(m2, m3, sh));
      if (sh + n > 128u) atomicOr(&img[w + 4], __funnelshift_l(m3, 0u, sh));
    }
  }
}

// Decoder table: index = next `maxlen` stream bits, entry = level | codeword length << 8 (0 = no
// codeword starts with these bits).
constexpr int kDecLutMax = 1 << QGX_MAX_CODE_LEN;

// Reads a bucket's words with every access bounded by nwords.
struct BitReader {
  const uint32_t* w;
  uint32_t nwords;
  uint32_t next;          // index of the next word to fetch
  uint64_t buf;           // bits not yet consumed, next bit at bit 0
  int avail;
  __device__ __forceinline__ uint32_t fetch(uint32_t i) const { return i < nwords ? w[i] : 0u; }
  __device__ __forceinline__ void seek(uint32_t bitpos) {
    next = bitpos >> 5;
    const uint32_t sh = bitpos & 31u;
    buf = (uint64_t)(fetch(next) >> sh);
    avail = 32 - (int)sh;
    ++next;
    refill();
  }
  __device__ __forceinline__ void refill() {
    if (avail <= 32) {
      buf |= (uint64_t)fetch(next) << avail;
      avail += 32;
      ++next;
    }
  }
  __device__ __forceinline__ void skip(int n) { buf >>= n; avail -= n; }
};

// decodes one symbol; returns false on an unassigned pattern.  *used accumulates consumed bits.
__device__ __forceinline__ bool decode_symbol(BitReader& br, const uint16_t* lut, uint32_t mask, uint32_t* sym, uint32_t* used) {
  br.refill();
  const uint32_t e = lut[(uint32_t)br.buf & mask];
  const int L = (int)(e >> 8);
  if (L == 0) return false;
  const uint32_t idx = e & 0xffu;
  br.skip(L);
  uint32_t neg = 0;
  if (idx != 0) { neg = (uint32_t)br.buf & 1u; br.skip(1); }
  *sym = idx | (neg << 7);
  *used += (uint32_t)L + (idx != 0 ? 1u : 0u);
  return true;
}

void build_dec_lut_host(const CodeTable& ct, uint16_t* lut /*[1 << maxlen]*/);

}  // namespace qgx
