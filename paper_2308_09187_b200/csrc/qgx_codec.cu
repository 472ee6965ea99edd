// qgx_encode and qgx_decode as separate steps: bucket bit lengths -> exclusive scan of the
// word-aligned lengths (offsets) -> bit scatter; and offsets -> bit gather.
#include "qgx_bucket.cuh"
#include "qgx_codec.cuh"

#include <mutex>
#include <vector>

namespace qgx {

// Scratch of qgx_encode_noalloc: bucket word offsets (u64 per bucket) followed by one overflow flag per
// worker.  It lives in the library image, so every GPU that loads the library carries these bytes
// until the process exits.
constexpr size_t kNoAllocMaxBuckets = 65536;            // K * nb
constexpr size_t kNoAllocMaxWorkers = 1024;             // K
constexpr size_t kNoAllocBytes = kNoAllocMaxBuckets * sizeof(uint64_t) + kNoAllocMaxWorkers * sizeof(uint32_t);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

void build_dec_lut_host(const CodeTable& ct, uint16_t* lut) {
  const int n = 1 << ct.maxlen;
  for (int i = 0; i < n; ++i) lut[i] = 0;
  for (int j = 0; j < ct.nlev; ++j) {
    const int L = ct.len[j];
    for (int hi = 0; hi < (1 << (ct.maxlen - L)); ++hi) lut[ct.rev[j] | (hi << L)] = (uint16_t)(j | (L << 8));
  }
}

__device__ __forceinline__ uint32_t load_quad_syms(const uint8_t* p, int nvalid, bool vec_ok) {
  if (nvalid == kQuad && vec_ok) return *reinterpret_cast<const uint32_t*>(p);
  uint32_t x = 0;
  for (int c = 0; c < nvalid; ++c) x |= (uint32_t)p[c] << (8 * c);
  return x;
}

// bucket_bits[k][b] = 32 + 16 * nsub + sum_i (len[idx_i] + [idx_i != 0])
__global__ void __launch_bounds__(512) k_bucket_bits(const uint8_t* __restrict__ sym, size_t d, int bucket, CodeTable ct,
                                                     bool vec_ok, uint32_t* __restrict__ bucket_bits, DevStatus* st) {
  __shared__ EncLut s_lut;
  __shared__ uint32_t s_sum;
  const size_t b = blockIdx.x, k = blockIdx.y, nb = gridDim.x;
  const size_t lo = b * (size_t)bucket;
  const int len = (int)min((size_t)bucket, d - lo);
  fill_enc_lut(&s_lut, ct);
  if (threadIdx.x == 0) s_sum = 0;
  __syncthreads();
  const uint8_t* src = sym + k * d + lo;
  uint32_t bits = 0;
  bool bad = false;
  const int nquads = (len + kQuad - 1) / kQuad;
  for (int q = threadIdx.x; q < nquads; q += blockDim.x) {
    const int nvalid = min(kQuad, len - q * kQuad);
    const uint32_t s4 = load_quad_syms(src + q * kQuad, nvalid, vec_ok);
    for (int c = 0; c < nvalid; ++c) bad = bad || (((s4 >> (8 * c)) & 31u) >= (uint32_t)ct.nlev);
    uint64_t pb;
    uint32_t n;
    pack_quad(s4, nvalid, &s_lut, &pb, &n);
    bits += n;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, o);
  if ((threadIdx.x & 31) == 0) atomicAdd(&s_sum, bits);
  if (bad) latch_error(st, QGX_ERR_CORRUPT);
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t nsub = ct.has_header ? (uint32_t)((len + ct.G - 1) / ct.G) : 0u;
    bucket_bits[k * nb + b] = kNormBits + 16u * nsub + s_sum;
  }
}

// One CTA per worker: off[k][b] = sum_{b' < b} ceil(bits[k][b'] / 32); total_bits[k]; a worker whose
// words exceed cap_words is flagged (flags[k] = 1) and err_code is latched.
__global__ void __launch_bounds__(256) k_scan_offsets(const uint32_t* __restrict__ bucket_bits, size_t nb, size_t cap_words,
                                                      uint64_t* __restrict__ off, uint64_t* __restrict__ total_bits,
                                                      uint32_t* __restrict__ flags, unsigned int err_code, DevStatus* st) {
  __shared__ uint64_t s_words[8], s_bits[8];
  __shared__ uint64_t s_carry_w, s_carry_b;
  const size_t k = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  if (threadIdx.x == 0) { s_carry_w = 0; s_carry_b = 0; }
  __syncthreads();
  for (size_t base = 0; base < nb; base += blockDim.x) {
    const size_t b = base + threadIdx.x;
    const uint64_t bits = b < nb ? (uint64_t)bucket_bits[k * nb + b] : 0ull;
    const uint64_t words = (bits + 31) >> 5;
    uint64_t iw = words, ib = bits;                     // warp-inclusive scans of words and bits
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint64_t yw = __shfl_up_sync(0xffffffffu, iw, o), yb = __shfl_up_sync(0xffffffffu, ib, o);
      if (lane >= o) { iw += yw; ib += yb; }
    }
    if (lane == 31) { s_words[warp] = iw; s_bits[warp] = ib; }
    __syncthreads();
    uint64_t before = s_carry_w;
    for (int w = 0; w < warp; ++w) before += s_words[w];
    if (b < nb) off[k * nb + b] = before + iw - words;
    __syncthreads();                                    // every thread has read the carry
    if (threadIdx.x == 0) {
      uint64_t tw = 0, tb = 0;
      for (int w = 0; w < nwarps; ++w) { tw += s_words[w]; tb += s_bits[w]; }
      s_carry_w += tw;
      s_carry_b += tb;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    if (total_bits) total_bits[k] = s_carry_b;
    const bool over = s_carry_w > (uint64_t)cap_words;
    flags[k] = over ? 1u : 0u;
    if (over) latch_error(st, err_code);
  }
}

// One CTA per (bucket, worker): builds the bucket's words in shared memory and copies them out.
template <int V4>
__global__ void __launch_bounds__(512) k_bit_scatter(const float* __restrict__ norms, const uint8_t* __restrict__ sym, size_t d,
                                                     int bucket, CodeTable ct, bool vec_ok, uint32_t* __restrict__ stream,
                                                     size_t cap_words, const uint32_t* __restrict__ bucket_bits,
                                                     const uint64_t* __restrict__ off, const uint32_t* __restrict__ flags) {
  extern __shared__ uint32_t s_dyn[];
  __shared__ EncLut s_lut;
  __shared__ uint32_t s_chunk[264];                     // bits per chunk of 32 quads, then their exclusive scan
  const size_t b = blockIdx.x, k = blockIdx.y, nb = gridDim.x;
  if (flags[k]) return;
  const size_t lo = b * (size_t)bucket;
  const int len = (int)min((size_t)bucket, d - lo);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const uint32_t nbits = bucket_bits[k * nb + b];
  const uint32_t nwords = (nbits + 31) >> 5;
  const int qps = ct.G / kQuad;                         // quads per sub-block
  const uint32_t nsub = ct.has_header ? (uint32_t)((len + ct.G - 1) / ct.G) : 0u;
  const uint32_t hdr_bits = kNormBits + 16u * nsub;
  uint32_t* s_img = s_dyn;                              // nwords (+2 slack) words
  uint32_t* s_sub = s_dyn + (((uint32_t)bucket * (uint32_t)(ct.maxlen + 1) + 16u * (uint32_t)(bucket / ct.G + 1) + kNormBits + 31u) >> 5) + 4;

  fill_enc_lut(&s_lut, ct);
  for (uint32_t i = threadIdx.x; i < nwords + 2; i += blockDim.x) s_img[i] = 0;
  __syncthreads();

  const uint8_t* src = sym + k * d + lo;
  uint64_t qbits[V4];
  uint32_t qn[V4], qexcl[V4];
#pragma unroll
  for (int j = 0; j < V4; ++j) {
    const int q = j * (int)blockDim.x + (int)threadIdx.x;
    const int nvalid = max(0, min(kQuad, len - q * kQuad));
    uint32_t s4 = 0;
    if (nvalid > 0) s4 = load_quad_syms(src + q * kQuad, nvalid, vec_ok);
    pack_quad(s4, nvalid, &s_lut, &qbits[j], &qn[j]);
    const uint32_t incl = warp_incl_scan(qn[j], lane);
    qexcl[j] = incl - qn[j];
    if (lane == 31) s_chunk[j * nwarps + warp] = incl;
  }
  __syncthreads();
  const int nchunks = V4 * nwarps;                      // <= 256
  if (warp == 0) {
    uint32_t carry = 0;
    for (int base = 0; base < nchunks; base += 32) {
      const int i = base + lane;
      const uint32_t x = i < nchunks ? s_chunk[i] : 0u;
      const uint32_t incl = warp_incl_scan(x, lane);
      if (i < nchunks) s_chunk[i] = carry + incl - x;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) s_chunk[nchunks] = carry;            // payload bits of the bucket
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < V4; ++j) {
    const int q = j * (int)blockDim.x + (int)threadIdx.x;
    const uint32_t p = s_chunk[j * nwarps + warp] + qexcl[j];
    if (nsub && q * kQuad < len && q % qps == 0) s_sub[q / qps] = p;
    put_bits(s_img, hdr_bits + p, qbits[j], qn[j]);
  }
  if (threadIdx.x == 0) {
    atomicOr(&s_img[0], __float_as_uint(norms[k * nb + b]));
    if (nsub) s_sub[nsub] = s_chunk[nchunks];
  }
  __syncthreads();
  for (uint32_t s = threadIdx.x; s < nsub; s += blockDim.x) {
    const uint32_t L = s_sub[s + 1] - s_sub[s];
    reinterpret_cast<uint16_t*>(s_img)[2 + s] = (uint16_t)(L & 0xffffu);
  }
  __syncthreads();
  uint32_t* dst = stream + k * cap_words + off[k * nb + b];
  for (uint32_t i = threadIdx.x; i < nwords; i += blockDim.x) dst[i] = s_img[i];
}

// One CTA per (bucket, worker); one thread per sub-block walks its part of the stream.
__global__ void __launch_bounds__(256) k_decode(const uint32_t* __restrict__ stream, size_t cap_words,
                                                const uint32_t* __restrict__ bucket_bits, const uint64_t* __restrict__ off,
                                                const uint32_t* __restrict__ flags, size_t d, int bucket, CodeTable ct,
                                                const uint16_t* __restrict__ g_lut, bool vec_ok, float* __restrict__ norms,
                                                uint8_t* __restrict__ sym, DevStatus* st) {
  extern __shared__ uint32_t s_dyn[];
  const size_t b = blockIdx.x, k = blockIdx.y, nb = gridDim.x;
  const size_t lo = b * (size_t)bucket;
  const int len = (int)min((size_t)bucket, d - lo);
  const int lane = threadIdx.x & 31;
  const uint32_t nsub = ct.has_header ? (uint32_t)((len + ct.G - 1) / ct.G) : 1u;
  const uint32_t hdr_bits = kNormBits + (ct.has_header ? 16u * nsub : 0u);
  uint32_t* s_start = s_dyn;                            // nsub + 1 payload-relative start bits
  uint16_t* s_lut = reinterpret_cast<uint16_t*>(s_dyn + (bucket / ct.G + 2));
  const int lut_n = 1 << ct.maxlen;
  for (int i = threadIdx.x; i < lut_n; i += blockDim.x) s_lut[i] = g_lut[i];

  uint8_t* out = sym + k * d + lo;
  const bool dead = flags[k] != 0;
  const uint32_t nbits = dead ? 0u : bucket_bits[k * nb + b];
  const uint32_t nwords = (nbits + 31) >> 5;
  const uint32_t* w = stream + k * cap_words + (dead ? 0 : off[k * nb + b]);
  bool bad = !dead && nbits < hdr_bits;
  if (dead || bad) {                                    // nothing trustworthy to read: zero output
    for (int i = threadIdx.x; i < len; i += blockDim.x) out[i] = 0;
    if (threadIdx.x == 0) { norms[k * nb + b] = 0.0f; if (bad) latch_error(st, QGX_ERR_CORRUPT); }
    return;
  }
  if (threadIdx.x == 0) norms[k * nb + b] = __uint_as_float(w[0]);
  // start bit of every sub-block: exclusive scan of the 16-bit header fields
  if (threadIdx.x < 32) {
    uint32_t carry = 0;
    if (ct.has_header) {
      for (uint32_t base = 0; base < nsub; base += 32) {
        const uint32_t s = base + lane;
        uint32_t L = 0;
        if (s < nsub) {
          const uint32_t bit = kNormBits + 16u * s;
          L = (w[bit >> 5] >> (bit & 31u)) & 0xffffu;   // inside the header, which nbits covers
        }
        const uint32_t incl = warp_incl_scan(L, lane);
        if (s < nsub) s_start[s] = carry + incl - L;
        carry += __shfl_sync(0xffffffffu, incl, 31);
      }
    } else {
      if (lane == 0) s_start[0] = 0;
      carry = nbits - hdr_bits;
    }
    if (lane == 0) s_start[nsub] = carry;
  }
  __syncthreads();
  if (s_start[nsub] != nbits - hdr_bits) bad = true;    // the lengths must add up to the bucket's payload
  const uint32_t mask = (uint32_t)lut_n - 1u;
  for (uint32_t s = threadIdx.x; s < nsub; s += blockDim.x) {
    const int first = (int)s * ct.G;
    const int count = min(ct.G, len - first);
    const uint32_t want = s_start[s + 1] - s_start[s];
    BitReader br;
    br.w = w;
    br.nwords = nwords;
    br.seek(hdr_bits + s_start[s]);
    uint32_t used = 0;
    bool ok = !bad;
    for (int i = 0; i < count; i += kQuad) {
      uint32_t packed = 0;
      const int nvalid = min(kQuad, count - i);
      for (int c = 0; c < nvalid; ++c) {
        uint32_t one = 0;
        if (ok) ok = decode_symbol(br, s_lut, mask, &one, &used) && used <= want;
        if (!ok) one = 0;
        packed |= one << (8 * c);
      }
      uint8_t* o = out + first + i;
      if (nvalid == kQuad && vec_ok) {
        *reinterpret_cast<uint32_t*>(o) = packed;
      } else {
        for (int c = 0; c < nvalid; ++c) o[c] = (uint8_t)(packed >> (8 * c));
      }
    }
    if (!ok || used != want) bad = true;
  }
  if (bad) latch_error(st, QGX_ERR_CORRUPT);
}

}  // namespace qgx

using namespace qgx;

static bool codec_args_ok(qgx_ctx* c, int K, size_t d, int bucket) {
  return c && K >= 1 && K <= 65535 && d >= 1 && bucket >= kQuad && bucket <= QGX_MAX_BUCKET && bucket % kQuad == 0;
}

extern "C" {

qgx_status qgx_encode(qgx_ctx* c, const float* norms, const uint8_t* sym, int K, size_t d, int bucket,
                      const qgx_codebook* cb, uint32_t* stream, size_t cap_words, uint32_t* bucket_bits,
                      uint64_t* total_bits) {
  if (!codec_args_ok(c, K, d, bucket) || !norms || !sym || !stream || !bucket_bits || !total_bits) return QGX_ERR_INVALID_ARG;
  CodeTable ct;
  qgx_status rc = make_code_table(cb, bucket, &ct);
  if (rc != QGX_OK) return rc;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  uint64_t* off = (uint64_t*)ws_get(c, 0, sizeof(uint64_t) * (size_t)K * nb);
  uint32_t* flags = (uint32_t*)ws_get(c, 1, sizeof(uint32_t) * (size_t)K);
  if (!off || !flags) return QGX_ERR_CUDA;
  const bool vec_ok = (d % kQuad == 0) && ((reinterpret_cast<uintptr_t>(sym) & 3u) == 0);
  const int v4 = bucket_v4(bucket);
  const int threads = bucket_threads(bucket, v4);
  const dim3 grid((unsigned)nb, (unsigned)K);
  k_bucket_bits<<<grid, threads, 0, c->stream>>>(sym, d, bucket, ct, vec_ok, bucket_bits, c->dstatus);
  k_scan_offsets<<<K, 256, 0, c->stream>>>(bucket_bits, nb, cap_words, off, total_bits, flags, QGX_ERR_CAPACITY, c->dstatus);
  const size_t img_words = (((size_t)bucket * (ct.maxlen + 1) + 16u * (bucket / ct.G + 1) + kNormBits + 31u) >> 5) + 4;
  const size_t smem = sizeof(uint32_t) * (img_words + (size_t)(bucket / ct.G) + 2);
#define QGX_LAUNCH_S(V)                                                                                         \
  do {                                                                                                          \
    cudaFuncSetAttribute(k_bit_scatter<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);             \
    k_bit_scatter<V><<<grid, threads, smem, c->stream>>>(norms, sym, d, bucket, ct, vec_ok, stream, cap_words,  \
                                                         bucket_bits, off, flags);                              \
  } while (0)
  switch (v4) {
    case 1: QGX_LAUNCH_S(1); break;
    case 2: QGX_LAUNCH_S(2); break;
    case 4: QGX_LAUNCH_S(4); break;
    default: QGX_LAUNCH_S(8); break;
  }
#undef QGX_LAUNCH_S
  count_launch(c, 3);
  return cuda_status(cudaGetLastError());
}

qgx_status qgx_decode(qgx_ctx* c, const uint32_t* stream, size_t cap_words, const uint32_t* bucket_bits, int K, size_t d,
                      int bucket, const qgx_codebook* cb, float* norms, uint8_t* sym) {
  if (!codec_args_ok(c, K, d, bucket) || !norms || !sym || !stream || !bucket_bits) return QGX_ERR_INVALID_ARG;
  CodeTable ct;
  qgx_status rc = make_code_table(cb, bucket, &ct);
  if (rc != QGX_OK) return rc;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  uint64_t* off = (uint64_t*)ws_get(c, 0, sizeof(uint64_t) * (size_t)K * nb);
  uint32_t* flags = (uint32_t*)ws_get(c, 1, sizeof(uint32_t) * (size_t)K);
  uint16_t* lut = (uint16_t*)ws_get(c, 2, sizeof(uint16_t) * kDecLutMax);
  if (!off || !flags || !lut) return QGX_ERR_CUDA;
  std::vector<uint16_t> h_lut((size_t)1 << ct.maxlen);
  build_dec_lut_host(ct, h_lut.data());
  // pageable source: the runtime stages it before returning, so the vector may go out of scope
  if (cudaMemcpyAsync(lut, h_lut.data(), h_lut.size() * sizeof(uint16_t), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
    return QGX_ERR_CUDA;
  const bool vec_ok = (d % kQuad == 0) && ((reinterpret_cast<uintptr_t>(sym) & 3u) == 0);
  k_scan_offsets<<<K, 256, 0, c->stream>>>(bucket_bits, nb, cap_words, off, nullptr, flags, QGX_ERR_CORRUPT, c->dstatus);
  const uint32_t nsub_max = (uint32_t)(bucket / ct.G);
  const int threads = (int)std::min<uint32_t>(256u, ((std::max<uint32_t>(nsub_max, 1u) + 31u) / 32u) * 32u);
  const size_t smem = sizeof(uint32_t) * (nsub_max + 2) + sizeof(uint16_t) * ((size_t)1 << ct.maxlen);
  const dim3 grid((unsigned)nb, (unsigned)K);
  k_decode<<<grid, threads, smem, c->stream>>>(stream, cap_words, bucket_bits, off, flags, d, bucket, ct, lut, vec_ok, norms,
                                               sym, c->dstatus);
  count_launch(c, 2);
  return cuda_status(cudaGetLastError());
}


// Device address of g_noalloc_scratch on the current device.  In host code the array's name only stands
// in for the symbol; the address a kernel can use has to be asked for, once per device.
static qgx_status noalloc_scratch_address(int device, unsigned char** out) {
  static std::mutex mu;
  static unsigned char* addr[64] = {nullptr};
  if (device < 0 || device >= 64) return QGX_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(mu);
  if (addr[device] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return QGX_ERR_CUDA;
    }
    addr[device] = static_cast<unsigned char*>(p);
  }
  *out = addr[device];
  return QGX_OK;
}

qgx_status qgx_encode_noalloc(qgx_ctx* c, const float* norms, const uint8_t* sym, int K, size_t d, int bucket,
                              const qgx_codebook* cb, uint32_t* stream, size_t cap_words, uint32_t* bucket_bits,
                              uint64_t* total_bits) {
  if (!codec_args_ok(c, K, d, bucket) || !norms || !sym || !stream || !bucket_bits || !total_bits) return QGX_ERR_INVALID_ARG;
  const size_t nb = (d + (size_t)bucket - 1) / (size_t)bucket;
  if ((size_t)K > kNoAllocMaxWorkers || (size_t)K * nb > kNoAllocMaxBuckets) return QGX_ERR_TOO_LARGE;
  CodeTable ct;
  qgx_status rc = make_code_table(cb, bucket, &ct);
  if (rc != QGX_OK) return rc;
  if (cudaSetDevice(c->device) != cudaSuccess) return QGX_ERR_CUDA;
  unsigned char* scratch = nullptr;
  rc = noalloc_scratch_address(c->device, &scratch);
  if (rc != QGX_OK) return rc;
  uint64_t* off = reinterpret_cast<uint64_t*>(scratch);
  uint32_t* flags = reinterpret_cast<uint32_t*>(scratch + kNoAllocMaxBuckets * sizeof(uint64_t));
  // Nothing in the scratch has to start at zero: the scan kernel writes every offset and every flag
  // that the scatter kernel reads.  The flags are cleared all the same, so that a stale "overflow"
  // of an earlier call can never be seen.
  if (cudaMemsetAsync(flags, 0, sizeof(uint32_t) * (size_t)K, c->stream) != cudaSuccess) return QGX_ERR_CUDA;
  const bool vec_ok = (d % kQuad == 0) && ((reinterpret_cast<uintptr_t>(sym) & 3u) == 0);
  const int v4 = bucket_v4(bucket);
  const int threads = bucket_threads(bucket, v4);
  const dim3 grid((unsigned)nb, (unsigned)K);
  k_bucket_bits<<<grid, threads, 0, c->stream>>>(sym, d, bucket, ct, vec_ok, bucket_bits, c->dstatus);
  k_scan_offsets<<<K, 256, 0, c->stream>>>(bucket_bits, nb, cap_words, off, total_bits, flags, QGX_ERR_CAPACITY, c->dstatus);
  const size_t img_words = (((size_t)bucket * (ct.maxlen + 1) + 16u * (bucket / ct.G + 1) + kNormBits + 31u) >> 5) + 4;
  const size_t smem = sizeof(uint32_t) * (img_words + (size_t)(bucket / ct.G) + 2);
#define QGX_LAUNCH_S(V)                                                                                         \
  do {                                                                                                          \
    cudaFuncSetAttribute(k_bit_scatter<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);             \
    k_bit_scatter<V><<<grid, threads, smem, c->stream>>>(norms, sym, d, bucket, ct, vec_ok, stream, cap_words,  \
                                                         bucket_bits, off, flags);                              \
  } while (0)
  switch (v4) {
    case 1: QGX_LAUNCH_S(1); break;
    case 2: QGX_LAUNCH_S(2); break;
    case 4: QGX_LAUNCH_S(4); break;
    default: QGX_LAUNCH_S(8); break;
  }
#undef QGX_LAUNCH_S
  count_launch(c, 3);
  return cuda_status(cudaGetLastError());
}

}  // extern "C"
