// Q-GenX reference oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-threaded C++17 restatement of the data-parallel hot path of
// Q-GenX ("Distributed Extra-gradient with Optimal Complexity and Communication
// Guarantees", arXiv 2308.09187), written from the paper and used only to check the
// CUDA library.  It shares no source, header, table or constant generator with the
// CUDA path and is reachable only from the tests, the smoke check and the benchmark's
// CPU-baseline leg.  Every function follows the paper's steps in the paper's order;
// there is no blocking, fusion or reordering.
//
// Arithmetic convention: data are fp32; every fp32 operation below is a single IEEE-754
// round-to-nearest operation (compile with -ffp-contract=off, never -ffast-math);
// accumulations that the text marks "fp64" are done in double, in index order.
//
// Parity status of the parts (what pins each one is in tests/test_oracle_*.py):
//   quantizer, codec, histogram, level fit, pmf, Huffman lengths, Philox, the update
//   recursion and the step-size identity are pinned.  The constants of the convergence
//   rates of Theorems 3 and 4 are big-O only: "rate constants: parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstring>
#include <string>
#include <vector>
#include <algorithm>
#include <limits>

namespace {

constexpr int kMaxLevels = 32;      // level index fits the low 5 bits of a symbol byte
constexpr int kMaxCodeLen = 12;     // longest admitted codeword
constexpr int kNormBits = 32;       // C_b: the norm is sent as a standard 32-bit float (App. E)

// status codes (values mirror the public library's so that tests can compare them)
enum {
  OK = 0, INVALID_ARG = 1, BAD_LEVELS = 2, CAPACITY = 3, CORRUPT = 4, NONFINITE = 5
};

// ---------------------------------------------------------------------------------
// Counter-based generator: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
// One round: two 32x32->64 multiplies of counter words 0 and 2 by fixed odd constants,
// a word permutation, and an xor with the round key; the key is bumped by the Weyl
// constants between rounds.  Ten rounds.
// ---------------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k0 += W0; k1 += W1; }
    const uint64_t p0 = M0 * (uint64_t)c0;
    const uint64_t p1 = M1 * (uint64_t)c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The 32-bit word that decides the rounding of element e of worker k in exchange xid:
// key = seed, counter = (e/4 low, e/4 high, worker, exchange id), word e mod 4.
uint32_t element_word(uint64_t seed, uint32_t worker, uint32_t xid, uint64_t e) {
  const uint64_t q = e >> 2;
  const uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), worker, xid};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  philox4x32_10(ctr, key, out);
  return out[e & 3];
}

// ---------------------------------------------------------------------------------
// Definition 1 (random quantization function), one normalized coordinate at a time.
// ---------------------------------------------------------------------------------
bool levels_ok(const float* lev, int nlev) {
  if (nlev < 2 || nlev > kMaxLevels) return false;
  if (!(lev[0] == 0.0f) || !(lev[nlev - 1] == 1.0f)) return false;
  for (int j = 0; j + 1 < nlev; ++j)
    if (!(lev[j] < lev[j + 1])) return false;
  return true;
}

// u_i = |v_i| / ||v||  (Sec. 3.2), one fp32 division, clamped to 1; a zero bucket gives u = 0.
float normalize(float v, float norm) {
  if (!(norm > 0.0f)) return 0.0f;
  float u = std::fabs(v) / norm;
  if (u > 1.0f) u = 1.0f;
  return u;
}

// tau(u): the index with l_tau <= u < l_{tau+1}; u = 1 takes the last interval.
int level_search(float u, const float* lev, int nlev) {
  int tau = 0;
  for (int j = 1; j <= nlev - 2; ++j)
    if (lev[j] <= u) tau = j;
  return tau;
}

// xi(u) = (u - l_tau) / (l_{tau+1} - l_tau): subtraction, subtraction, division in fp32.
float xi_of(float u, const float* lev, int tau) {
  const float num = u - lev[tau];
  const float den = lev[tau + 1] - lev[tau];
  return num / den;
}

// Round up with probability xi: the uniform variate is the top 24 bits of the word,
// r = (w >> 8) * 2^-24 in [0,1), and the upper level is taken iff r < xi.
int round_up(float xi, uint32_t word) {
  const float r = (float)(word >> 8) * 5.9604644775390625e-8f;  // exact: 24-bit integer * 2^-24
  return r < xi ? 1 : 0;
}

// symbol byte: bits 0..4 level index, bit 7 sign (set only for a nonzero level index)
uint8_t quantize_element(float v, float norm, const float* lev, int nlev, uint32_t word) {
  const float u = normalize(v, norm);
  const int tau = level_search(u, lev, nlev);
  const float xi = xi_of(u, lev, tau);
  const int idx = tau + round_up(xi, word);
  const bool neg = std::signbit(v) && idx != 0;
  return (uint8_t)(idx | (neg ? 0x80 : 0));
}

// Q_l(v) coordinate: ||v|| * s * l_idx  (Definition 1), one fp32 multiply.
float dequantize_element(uint8_t sym, float norm, const float* lev) {
  const int idx = sym & 31;
  const float val = norm * lev[idx];
  return (sym & 0x80) ? -val : val;
}

inline uint64_t n_buckets(uint64_t d, int bucket) { return (d + (uint64_t)bucket - 1) / (uint64_t)bucket; }

// Norm of one bucket: L2 = sqrt of the fp64 sum of squares in index order, rounded once
// to fp32; L-infinity = largest magnitude.
float bucket_norm(const float* v, uint64_t len, int norm_type) {
  if (norm_type == 1) {
    float m = 0.0f;
    bool bad = false;
    for (uint64_t i = 0; i < len; ++i) {
      const float a = std::fabs(v[i]);
      if (!(a == a)) bad = true;
      if (a > m) m = a;
    }
    return bad ? std::numeric_limits<float>::quiet_NaN() : m;
  }
  double s = 0.0;
  for (uint64_t i = 0; i < len; ++i) s += (double)v[i] * (double)v[i];
  return (float)std::sqrt(s);
}

// ---------------------------------------------------------------------------------
// Bit stream (Sec. 3.2 / App. J): LSB-first 32-bit words.
// ---------------------------------------------------------------------------------
struct BitWriter {
  uint32_t* w; uint64_t cap_bits; uint64_t pos; bool overflow;
  void put(uint32_t value, int nbits) {           // bit 0 of value is written first
    for (int b = 0; b < nbits; ++b) {
      if (pos >= cap_bits) { overflow = true; return; }
      if ((value >> b) & 1u) w[pos >> 5] |= (1u << (pos & 31));
      ++pos;
    }
  }
};
struct BitReader {
  const uint32_t* w; uint64_t end; uint64_t pos; bool overrun;
  int get() {
    if (pos >= end) { overrun = true; return 0; }
    const int b = (int)((w[pos >> 5] >> (pos & 31)) & 1u);
    ++pos;
    return b;
  }
};

}  // namespace

extern "C" {

struct qgxo_codebook {
  int32_t nlev;
  int32_t maxlen;
  int32_t subblock;        // elements per sub-block; <=0 or >= bucket: no sub-block header
  uint8_t len[32];         // codeword length of each level index
  uint32_t code[32];       // codeword as an integer; its most significant (len-th) bit is sent first
};

struct qgxo_operator {
  int32_t kind;            // 0 dense affine (M row-major d x d, b), 1 bilinear (A n x n, d = 2n), 2 diagonal (D)
  int32_t noise_model;     // how a worker's noise enters its dual vector: 0 V_k = A(x) + U_k, 1 V_k = A(x) .* U_k
  uint64_t d;
  const float* mat;        // M, A or D
  const float* bias;       // b (dense affine) or null
};

struct qgxo_eg_state {
  uint64_t d;
  int32_t K;
  int32_t t;               // iteration counter, starts at 1
  float* X;                // X_t
  float* Y;                // Y_t
  float* Xbar;             // running mean of X_{t+1/2}
  float* Xhalf;            // X_{t+1/2} of the last step
  const float* anchor;     // X_1
  double sum_sq;           // sum_{i<t} sum_k ||Vhat_{k,i} - Vhat_{k,i+1/2}||^2
  float gamma;             // gamma_t
  float pad;
};

// ------------------------------- RNG ----------------------------------------------
void qgxo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }
uint32_t qgxo_element_word(uint64_t seed, uint32_t worker, uint32_t xid, uint64_t e) { return element_word(seed, worker, xid, e); }

// ------------------------------- scalar pieces of Definition 1 ---------------------
int qgxo_check_levels(const float* lev, int nlev) { return levels_ok(lev, nlev) ? OK : BAD_LEVELS; }
float qgxo_normalize(float v, float norm) { return normalize(v, norm); }
int qgxo_level_search(float u, const float* lev, int nlev) { return level_search(u, lev, nlev); }
float qgxo_xi(float u, const float* lev, int tau) { return xi_of(u, lev, tau); }
int qgxo_round_up(float xi, uint32_t word) { return round_up(xi, word); }
// how many of the 2^24 equally likely variates round up (exhaustive)
uint64_t qgxo_count_up(float xi) {
  uint64_t n = 0;
  for (uint32_t m = 0; m < (1u << 24); ++m) n += (uint64_t)round_up(xi, m << 8);
  return n;
}

// ------------------------------- norms ---------------------------------------------
// norms[k][b] for v[k][d]; norm_type 0 = L2, 1 = L-infinity.  A non-finite norm is
// reported (NONFINITE) after all norms are written.
int qgxo_bucket_norms(const float* v, int K, uint64_t d, int bucket, int norm_type, float* norms) {
  if (K < 1 || bucket < 1 || (norm_type != 0 && norm_type != 1)) return INVALID_ARG;
  const uint64_t nb = n_buckets(d, bucket);
  int st = OK;
  for (int k = 0; k < K; ++k)
    for (uint64_t b = 0; b < nb; ++b) {
      const uint64_t lo = b * (uint64_t)bucket, hi = std::min<uint64_t>(d, lo + (uint64_t)bucket);
      const float n = bucket_norm(v + (uint64_t)k * d + lo, hi - lo, norm_type);
      norms[(uint64_t)k * nb + b] = n;
      if (!std::isfinite(n)) st = NONFINITE;
    }
  return st;
}

// ------------------------------- quantize ------------------------------------------
// sym[k][i] from v[k][i], the bucket norms and the Philox word of (seed, k, xid, coord_base + i).
// coord_base is where this vector starts inside a longer layer-wise dual vector (0 for a vector on its own):
// each tensor is quantized on its own (its own buckets, norms and levels), only the variates are indexed
// by the position in the whole vector.
int qgxo_quantize_at(const float* v, int K, uint64_t d, int bucket, const float* lev, int nlev,
                     const float* norms, uint64_t seed, uint32_t xid, uint64_t coord_base, uint8_t* sym) {
  if (K < 1 || bucket < 1) return INVALID_ARG;
  if (!levels_ok(lev, nlev)) return BAD_LEVELS;
  const uint64_t nb = n_buckets(d, bucket);
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) {
      const float norm = norms[(uint64_t)k * nb + i / (uint64_t)bucket];
      sym[(uint64_t)k * d + i] =
          quantize_element(v[(uint64_t)k * d + i], norm, lev, nlev, element_word(seed, (uint32_t)k, xid, coord_base + i));
    }
  return OK;
}

int qgxo_quantize(const float* v, int K, uint64_t d, int bucket, const float* lev, int nlev,
                  const float* norms, uint64_t seed, uint32_t xid, uint8_t* sym) {
  return qgxo_quantize_at(v, K, d, bucket, lev, nlev, norms, seed, xid, 0, sym);
}

// Same, with the random words supplied by the caller (words[k][i]); used to enumerate outcomes.
int qgxo_quantize_words(const float* v, int K, uint64_t d, int bucket, const float* lev, int nlev,
                        const float* norms, const uint32_t* words, uint8_t* sym) {
  if (K < 1 || bucket < 1) return INVALID_ARG;
  if (!levels_ok(lev, nlev)) return BAD_LEVELS;
  const uint64_t nb = n_buckets(d, bucket);
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) {
      const float norm = norms[(uint64_t)k * nb + i / (uint64_t)bucket];
      sym[(uint64_t)k * d + i] = quantize_element(v[(uint64_t)k * d + i], norm, lev, nlev, words[(uint64_t)k * d + i]);
    }
  return OK;
}

// vhat[k][i] = Q_l(v)_i
int qgxo_dequantize(const float* norms, const uint8_t* sym, int K, uint64_t d, int bucket,
                    const float* lev, int nlev, float* vhat) {
  if (K < 1 || bucket < 1) return INVALID_ARG;
  if (!levels_ok(lev, nlev)) return BAD_LEVELS;
  const uint64_t nb = n_buckets(d, bucket);
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) {
      const uint8_t s = sym[(uint64_t)k * d + i];
      if ((s & 31) >= nlev) return CORRUPT;
      vhat[(uint64_t)k * d + i] = dequantize_element(s, norms[(uint64_t)k * nb + i / (uint64_t)bucket], lev);
    }
  return OK;
}

// out[i] = (1/K) sum_k vhat[k][i]: fp32 running sum over k = 0..K-1, then one fp32 division.
int qgxo_average(const float* norms, const uint8_t* sym, int K, uint64_t d, int bucket,
                 const float* lev, int nlev, float* out) {
  if (K < 1 || bucket < 1) return INVALID_ARG;
  if (!levels_ok(lev, nlev)) return BAD_LEVELS;
  const uint64_t nb = n_buckets(d, bucket);
  for (uint64_t i = 0; i < d; ++i) {
    float acc = 0.0f;
    for (int k = 0; k < K; ++k) {
      const uint8_t s = sym[(uint64_t)k * d + i];
      if ((s & 31) >= nlev) return CORRUPT;
      acc = acc + dequantize_element(s, norms[(uint64_t)k * nb + i / (uint64_t)bucket], lev);
    }
    out[i] = acc / (float)K;
  }
  return OK;
}

// ------------------------------- codebooks (App. J) --------------------------------
static void canonical_codes(qgxo_codebook* cb) {
  // codes in increasing (length, index) order, each the previous plus one, shifted when the length grows
  std::vector<int> order(cb->nlev);
  for (int j = 0; j < cb->nlev; ++j) order[j] = j;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cb->len[a] < cb->len[b]; });
  uint32_t code = 0;
  int prev = cb->len[order[0]];
  cb->maxlen = 0;
  for (int r = 0; r < cb->nlev; ++r) {
    const int j = order[r];
    if (r > 0) { code = (code + 1u) << (cb->len[j] - prev); prev = cb->len[j]; }
    cb->code[j] = code;
    cb->maxlen = std::max<int>(cb->maxlen, cb->len[j]);
  }
}

// every level index gets ceil(log2 nlev) bits (at least one)
int qgxo_codebook_fixed(int nlev, int subblock, qgxo_codebook* cb) {
  if (nlev < 2 || nlev > kMaxLevels) return INVALID_ARG;
  std::memset(cb, 0, sizeof(*cb));
  int L = 1;
  while ((1 << L) < nlev) ++L;
  cb->nlev = nlev; cb->subblock = subblock;
  for (int j = 0; j < nlev; ++j) cb->len[j] = (uint8_t)L;
  canonical_codes(cb);
  return OK;
}

// Elias' recursive ("omega") code of the positive integer n, as a string of '0'/'1' in sending order
// (Elias 1975; the universal integer code that App. J names for an unknown symbol distribution):
// start from the single bit 0; while n > 1, put the binary expansion of n in front and replace n by
// the number of bits of that expansion minus one.
static std::string elias_omega(unsigned n) {
  std::string out = "0";
  while (n > 1) {
    std::string bin;
    for (unsigned m = n; m > 0; m >>= 1) bin.insert(bin.begin(), (m & 1u) ? '1' : '0');
    out = bin + out;
    n = (unsigned)bin.size() - 1;
  }
  return out;
}

// level index j is sent as the code of the integer j + 1: smaller levels get shorter codewords
int qgxo_codebook_elias(int nlev, int subblock, qgxo_codebook* cb) {
  if (nlev < 2 || nlev > kMaxLevels) return INVALID_ARG;
  std::memset(cb, 0, sizeof(*cb));
  cb->nlev = nlev; cb->subblock = subblock;
  for (int j = 0; j < nlev; ++j) {
    const std::string w = elias_omega((unsigned)j + 1u);
    uint32_t code = 0;
    for (char c : w) code = (code << 1) | (c == '1' ? 1u : 0u);     // first sent bit = most significant
    cb->len[j] = (uint8_t)w.size();
    cb->code[j] = code;
    cb->maxlen = std::max<int>(cb->maxlen, (int)w.size());
  }
  return OK;
}

// Huffman code lengths for weights p (repeatedly merge the two smallest weights; among equal
// weights the node created earlier / the lower index goes first).
static void huffman_lengths(const std::vector<double>& p, std::vector<int>& len) {
  const int n = (int)p.size();
  struct Node { double w; int left, right; };
  std::vector<Node> nodes;
  for (int j = 0; j < n; ++j) nodes.push_back({p[j], -1, -1});
  std::vector<int> live(n);
  for (int j = 0; j < n; ++j) live[j] = j;
  while (live.size() > 1) {
    int a = 0;
    for (size_t i = 1; i < live.size(); ++i) if (nodes[live[i]].w < nodes[live[a]].w) a = (int)i;
    const int na = live[a]; live.erase(live.begin() + a);
    int b = 0;
    for (size_t i = 1; i < live.size(); ++i) if (nodes[live[i]].w < nodes[live[b]].w) b = (int)i;
    const int nbn = live[b]; live.erase(live.begin() + b);
    nodes.push_back({nodes[na].w + nodes[nbn].w, na, nbn});
    live.push_back((int)nodes.size() - 1);
  }
  len.assign(n, 0);
  std::vector<std::pair<int, int>> stack;           // (node, depth)
  stack.push_back({live[0], 0});
  while (!stack.empty()) {
    auto [id, dep] = stack.back(); stack.pop_back();
    if (nodes[id].left < 0) { len[id] = std::max(dep, 1); continue; }
    stack.push_back({nodes[id].left, dep + 1});
    stack.push_back({nodes[id].right, dep + 1});
  }
}

// Huffman codebook for the symbol weights p[0..nlev); if the longest codeword exceeds 12
// bits the weights are flattened by adding 2^(m-16), m = 0,1,2,..., to each until it fits.
int qgxo_codebook_huffman(const double* p, int nlev, int subblock, qgxo_codebook* cb) {
  if (nlev < 2 || nlev > kMaxLevels) return INVALID_ARG;
  for (int j = 0; j < nlev; ++j) if (!(p[j] >= 0.0) || !std::isfinite(p[j])) return INVALID_ARG;
  std::memset(cb, 0, sizeof(*cb));
  cb->nlev = nlev; cb->subblock = subblock;
  std::vector<double> w(p, p + nlev);
  std::vector<int> len;
  for (int m = 0;; ++m) {
    huffman_lengths(w, len);
    const int mx = *std::max_element(len.begin(), len.end());
    if (mx <= kMaxCodeLen) break;
    const double add = std::ldexp(1.0, m - 16);
    for (int j = 0; j < nlev; ++j) w[j] = p[j] + add;
  }
  for (int j = 0; j < nlev; ++j) cb->len[j] = (uint8_t)len[j];
  canonical_codes(cb);
  return OK;
}

// ------------------------------- choice of the code (App. J) -----------------------
// App. J names two families of codes: Huffman's when the frequencies of the levels are known or can be estimated,
// Elias' recursive code when they are not.  What decides between candidate codes here is what an exchange would
// have cost under each: counts[j] = how many coordinates of the last exchange were sent as level j; a code costs
// sum_j counts[j] * (len_j + [j != 0]) bits on them (codeword, plus the sign bit of a nonzero level; the bucket
// headers are the same under every code).
int qgxo_level_counts(const uint8_t* sym, int K, uint64_t d, int nlev, uint64_t* counts) {
  if (K < 1 || nlev < 2 || nlev > kMaxLevels) return INVALID_ARG;
  for (int j = 0; j < kMaxLevels; ++j) counts[j] = 0;
  for (uint64_t i = 0; i < (uint64_t)K * d; ++i) {
    const int idx = sym[i] & 31;
    if (idx >= nlev) return CORRUPT;
    counts[idx] += 1;
  }
  return OK;
}

uint64_t qgxo_code_bits(const uint64_t* counts, const qgxo_codebook* cb) {
  uint64_t bits = 0;
  for (int j = 0; j < cb->nlev; ++j) bits += counts[j] * (uint64_t)(cb->len[j] + (j != 0 ? 1 : 0));
  return bits;
}

// Candidates, in this order: 0 the code in use; 1 a Huffman code built from the counts themselves (only if
// allow_rebuild); 2 Elias' recursive code; 3 the fixed-length code.  bits[c] receives each candidate's cost
// (~0 for a candidate that is not allowed); the cheapest wins, the earlier candidate on ties; *chosen receives
// its codebook.  Returns the winner's number, or a negative status.
int qgxo_choose_code(const uint64_t* counts, int nlev, const qgxo_codebook* current, int allow_rebuild, uint64_t* bits,
                     qgxo_codebook* chosen) {
  if (nlev < 2 || nlev > kMaxLevels || current->nlev != nlev) return -INVALID_ARG;
  qgxo_codebook cand[4];
  cand[0] = *current;
  uint64_t total = 0;
  for (int j = 0; j < nlev; ++j) total += counts[j];
  bool have[4] = {true, allow_rebuild != 0 && total > 0, true, true};
  if (have[1]) {
    std::vector<double> p(nlev);
    for (int j = 0; j < nlev; ++j) p[j] = (double)counts[j] / (double)total;
    if (qgxo_codebook_huffman(p.data(), nlev, current->subblock, &cand[1]) != OK) have[1] = false;
  }
  if (qgxo_codebook_elias(nlev, current->subblock, &cand[2]) != OK) have[2] = false;
  if (qgxo_codebook_fixed(nlev, current->subblock, &cand[3]) != OK) have[3] = false;
  int best = 0;
  for (int c = 0; c < 4; ++c) {
    bits[c] = have[c] ? qgxo_code_bits(counts, &cand[c]) : ~(uint64_t)0;
    if (have[c] && bits[c] < bits[best]) best = c;
  }
  *chosen = cand[best];
  return best;
}

// ------------------------------- stream geometry -----------------------------------
static inline int eff_subblock(int bucket, int subblock) { return (subblock <= 0 || subblock >= bucket) ? bucket : subblock; }

// worst-case words of one worker's stream
uint64_t qgxo_capacity_words(uint64_t d, int bucket, int subblock, int maxlen) {
  const uint64_t nb = n_buckets(d, bucket);
  const int G = eff_subblock(bucket, subblock);
  uint64_t words = 0;
  for (uint64_t b = 0; b < nb; ++b) {
    const uint64_t len = std::min<uint64_t>(d, (b + 1) * (uint64_t)bucket) - b * (uint64_t)bucket;
    const uint64_t nsub = (G < bucket) ? (len + G - 1) / G : 0;
    const uint64_t bits = kNormBits + 16 * nsub + len * (uint64_t)(maxlen + 1);
    words += (bits + 31) / 32;
  }
  return words;
}

// ------------------------------- CODE o Q ------------------------------------------
// Per bucket, in this order: the 32 bits of the norm; if the bucket is cut into
// sub-blocks, one 16-bit length (in bits) per sub-block; then for each coordinate in
// order its codeword (first code bit first) followed by one sign bit iff the level
// index is nonzero.  Each bucket starts on a word boundary; unused bits are zero.
int qgxo_encode(const float* norms, const uint8_t* sym, int K, uint64_t d, int bucket,
                const qgxo_codebook* cb, uint32_t* stream, uint64_t cap_words,
                uint32_t* bucket_bits, uint64_t* total_bits) {
  if (K < 1 || bucket < 1 || cb->nlev < 2 || cb->nlev > kMaxLevels) return INVALID_ARG;
  const uint64_t nb = n_buckets(d, bucket);
  const int G = eff_subblock(bucket, cb->subblock);
  for (int k = 0; k < K; ++k) {
    uint32_t* w = stream + (uint64_t)k * cap_words;
    std::memset(w, 0, cap_words * sizeof(uint32_t));
    BitWriter bw{w, cap_words * 32, 0, false};
    uint64_t sum_bits = 0;
    for (uint64_t b = 0; b < nb; ++b) {
      bw.pos = (bw.pos + 31) & ~(uint64_t)31;               // word boundary
      const uint64_t start = bw.pos;
      const uint64_t lo = b * (uint64_t)bucket, hi = std::min<uint64_t>(d, lo + (uint64_t)bucket);
      uint32_t nbits;
      std::memcpy(&nbits, &norms[(uint64_t)k * nb + b], 4);
      bw.put(nbits, kNormBits);
      const uint64_t nsub = (G < bucket) ? (hi - lo + G - 1) / G : 0;
      const uint64_t header_pos = bw.pos;
      bw.pos += 16 * nsub;                                  // the length fields are written once the payload is known
      if (bw.overflow || bw.pos > bw.cap_bits) return CAPACITY;
      std::vector<uint32_t> sublen(nsub, 0);
      for (uint64_t i = lo; i < hi; ++i) {
        const uint8_t s = sym[(uint64_t)k * d + i];
        const int idx = s & 31;
        if (idx >= cb->nlev) return INVALID_ARG;
        const uint64_t before = bw.pos;
        const int L = cb->len[idx];
        for (int c = L - 1; c >= 0; --c) bw.put((cb->code[idx] >> c) & 1u, 1);   // first code bit first
        if (idx != 0) bw.put((s >> 7) & 1u, 1);                                   // sign of a nonzero coordinate
        if (bw.overflow) return CAPACITY;
        if (nsub) sublen[(i - lo) / (uint64_t)G] += (uint32_t)(bw.pos - before);
      }
      const uint64_t payload_end = bw.pos;
      for (uint64_t sb = 0; sb < nsub; ++sb) {
        if (sublen[sb] > 0xFFFFu) return INVALID_ARG;
        bw.pos = header_pos + 16 * sb;
        bw.put(sublen[sb], 16);
      }
      bw.pos = payload_end;
      const uint64_t used = bw.pos - start;
      bucket_bits[(uint64_t)k * nb + b] = (uint32_t)used;
      sum_bits += used;
    }
    total_bits[k] = sum_bits;
  }
  return OK;
}

// ------------------------------- DEQ o CODE ----------------------------------------
// Exact inverse, bucket by bucket; the bucket's bit length bounds every read.
int qgxo_decode(const uint32_t* stream, uint64_t cap_words, const uint32_t* bucket_bits,
                int K, uint64_t d, int bucket, const qgxo_codebook* cb, float* norms, uint8_t* sym) {
  if (K < 1 || bucket < 1 || cb->nlev < 2 || cb->nlev > kMaxLevels) return INVALID_ARG;
  const uint64_t nb = n_buckets(d, bucket);
  const int G = eff_subblock(bucket, cb->subblock);
  for (int k = 0; k < K; ++k) {
    const uint32_t* w = stream + (uint64_t)k * cap_words;
    uint64_t word_off = 0;
    for (uint64_t b = 0; b < nb; ++b) {
      const uint64_t bits = bucket_bits[(uint64_t)k * nb + b];
      if (word_off + (bits + 31) / 32 > cap_words) return CORRUPT;
      BitReader br{w, word_off * 32 + bits, word_off * 32, false};
      const uint64_t lo = b * (uint64_t)bucket, hi = std::min<uint64_t>(d, lo + (uint64_t)bucket);
      uint32_t nbits = 0;
      for (int q = 0; q < kNormBits; ++q) nbits |= (uint32_t)br.get() << q;
      float norm;
      std::memcpy(&norm, &nbits, 4);
      norms[(uint64_t)k * nb + b] = norm;
      const uint64_t nsub = (G < bucket) ? (hi - lo + G - 1) / G : 0;
      std::vector<uint32_t> sublen(nsub);
      for (uint64_t sb = 0; sb < nsub; ++sb) {
        uint32_t L = 0;
        for (int q = 0; q < 16; ++q) L |= (uint32_t)br.get() << q;
        sublen[sb] = L;
      }
      if (br.overrun) return CORRUPT;
      uint64_t sb_start = br.pos;
      for (uint64_t i = lo; i < hi; ++i) {
        // walk the prefix code one bit at a time
        uint32_t acc = 0;
        int L = 0, idx = -1;
        while (idx < 0) {
          acc = (acc << 1) | (uint32_t)br.get();
          ++L;
          if (br.overrun || L > kMaxCodeLen) return CORRUPT;
          for (int j = 0; j < cb->nlev; ++j)
            if (cb->len[j] == L && cb->code[j] == acc) { idx = j; break; }
        }
        int neg = 0;
        if (idx != 0) neg = br.get();
        if (br.overrun) return CORRUPT;
        sym[(uint64_t)k * d + i] = (uint8_t)(idx | (neg ? 0x80 : 0));
        if (nsub && ((i - lo + 1) % (uint64_t)G == 0 || i + 1 == hi)) {
          const uint64_t sb = (i - lo) / (uint64_t)G;
          if (br.pos - sb_start != sublen[sb]) return CORRUPT;
          sb_start = br.pos;
        }
      }
      if (br.pos != br.end) return CORRUPT;
      word_off += (bits + 31) / 32;
    }
  }
  return OK;
}

// ------------------------------- sufficient statistics (Sec. 3.3) ------------------
// hist[bin(u_i)] += lambda, lambda = ||bucket||^2 (weighted) or 1 (unweighted),
// bin(u) = min(floor(u * nbins), nbins-1), over all workers, buckets, coordinates in order.
int qgxo_histogram(const float* v, int K, uint64_t d, int bucket, int norm_type, int nbins,
                   int weighted, double* hist) {
  if (K < 1 || bucket < 1 || nbins < 1) return INVALID_ARG;
  const uint64_t nb = n_buckets(d, bucket);
  for (int j = 0; j < nbins; ++j) hist[j] = 0.0;
  int st = OK;
  for (int k = 0; k < K; ++k)
    for (uint64_t b = 0; b < nb; ++b) {
      const uint64_t lo = b * (uint64_t)bucket, hi = std::min<uint64_t>(d, lo + (uint64_t)bucket);
      const float* vb = v + (uint64_t)k * d + lo;
      const float norm = bucket_norm(vb, hi - lo, norm_type);
      if (!std::isfinite(norm)) { st = NONFINITE; continue; }
      const double wgt = weighted ? (double)norm * (double)norm : 1.0;
      for (uint64_t i = 0; i < hi - lo; ++i) {
        const float u = normalize(vb[i], norm);
        int bin = (int)std::floor(u * (float)nbins);
        if (bin > nbins - 1) bin = nbins - 1;
        hist[bin] += wgt;
      }
    }
  return st;
}

}  // extern "C"

namespace {

// F~ as a piecewise-uniform density: bin j spreads its mass evenly over [j/n, (j+1)/n).
// Moments M_r(x) = int_0^x u^r dF~(u), r = 0, 1, 2, from running sums over whole bins plus
// the exact integral over the part of the bin that contains x.
struct Cdf {
  int n; std::vector<double> m, P0, P1, P2;
  Cdf(const double* hist, int nbins) : n(nbins), m(hist, hist + nbins), P0(nbins + 1, 0.0), P1(nbins + 1, 0.0), P2(nbins + 1, 0.0) {
    for (int j = 0; j < n; ++j) {
      const double a = (double)j / n, b = (double)(j + 1) / n, dens = m[j] * n;
      P0[j + 1] = P0[j] + m[j];
      P1[j + 1] = P1[j] + dens * (b * b - a * a) / 2.0;
      P2[j + 1] = P2[j] + dens * (b * b * b - a * a * a) / 3.0;
    }
  }
  double moment(int r, double x) const {
    if (x <= 0.0) return 0.0;
    if (x >= 1.0) return r == 0 ? P0[n] : (r == 1 ? P1[n] : P2[n]);
    int j = (int)std::floor(x * n);
    if (j > n - 1) j = n - 1;
    const double a = (double)j / n, dens = m[j] * n;
    if (r == 0) return P0[j] + dens * (x - a);
    if (r == 1) return P1[j] + dens * (x * x - a * a) / 2.0;
    return P2[j] + dens * (x * x * x - a * a * a) / 3.0;
  }
  // int_lo^hi (c - u)(u - a) dF~ = -M2 + (a + c) M1 - a c M0 over [lo, hi]
  double var_integral(double a, double c, double lo, double hi) const {
    const double d0 = moment(0, hi) - moment(0, lo), d1 = moment(1, hi) - moment(1, lo), d2 = moment(2, hi) - moment(2, lo);
    return -d2 + (a + c) * d1 - a * c * d0;
  }
};

// the QAda objective: sum over intervals of int sigma_Q^2(u; l) dF~(u), sigma_Q^2 = (l_{i+1}-u)(u-l_i)
double objective(const Cdf& F, const std::vector<double>& lev) {
  double s = 0.0;
  for (size_t i = 0; i + 1 < lev.size(); ++i) s += F.var_integral(lev[i], lev[i + 1], lev[i], lev[i + 1]);
  return s;
}

// derivative of the objective in one level l with its neighbours a < l < c fixed:
// g(l) = int_a^l (u - a) dF~ - int_l^c (c - u) dF~   (non-decreasing in l)
double stationarity(const Cdf& F, double a, double c, double l) {
  const double left = (F.moment(1, l) - F.moment(1, a)) - a * (F.moment(0, l) - F.moment(0, a));
  const double right = c * (F.moment(0, c) - F.moment(0, l)) - (F.moment(1, c) - F.moment(1, l));
  return left - right;
}

}  // namespace

extern "C" {

double qgxo_objective(const double* hist, int nbins, const float* lev, int nlev) {
  Cdf F(hist, nbins);
  std::vector<double> l(lev, lev + nlev);
  return objective(F, l);
}

double qgxo_stationarity(const double* hist, int nbins, double a, double c, double l) {
  Cdf F(hist, nbins);
  return stationarity(F, a, c, l);
}

// Level fit: coordinate descent on the QAda objective, one level at a time, each level
// moved to the root of g on [a, c] by bisection.  first_fit != 0 starts from the mass
// quantiles of F~ at j/(nlev-1); otherwise from the levels passed in.  At most 32 sweeps,
// stops when no level moved by 1e-7 or more.  Levels are kept 2^-20 apart, rounded to fp32.
// obj_trace (may be null) receives the objective before the first sweep and after every sweep
// (length up to 33); *n_sweeps the number of sweeps made.
int qgxo_fit_levels(const double* hist, int nbins, float* lev, int nlev, int first_fit,
                    double* obj_trace, int* n_sweeps) {
  if (nlev < 2 || nlev > kMaxLevels || nbins < 1) return INVALID_ARG;
  Cdf F(hist, nbins);
  const double total = F.P0[nbins];
  const double gap = std::ldexp(1.0, -20);
  std::vector<double> l(nlev);
  if (first_fit) {
    l[0] = 0.0; l[nlev - 1] = 1.0;
    for (int j = 1; j <= nlev - 2; ++j) {
      // smallest x with F~(x) >= (j/(nlev-1)) * total, by bisection on the cdf
      const double target = total * (double)j / (double)(nlev - 1);
      double lo = 0.0, hi = 1.0;
      for (int it = 0; it < 60; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (F.moment(0, mid) >= target) hi = mid; else lo = mid;
      }
      l[j] = hi;
    }
  } else {
    if (!levels_ok(lev, nlev)) return BAD_LEVELS;
    for (int j = 0; j < nlev; ++j) l[j] = (double)lev[j];
  }
  // keep a valid, separated table from the start
  for (int j = 1; j <= nlev - 2; ++j) l[j] = std::max(l[j], l[j - 1] + gap);
  for (int j = nlev - 2; j >= 1; --j) l[j] = std::min(l[j], l[j + 1] - gap);
  int sweeps = 0;
  if (obj_trace) obj_trace[0] = objective(F, l);
  if (total > 0.0) {
    for (int sweep = 0; sweep < 32; ++sweep) {
      double moved = 0.0;
      for (int j = 1; j <= nlev - 2; ++j) {
        const double a = l[j - 1], c = l[j + 1];
        if (!(F.moment(0, c) - F.moment(0, a) > 0.0)) continue;      // no mass between the neighbours
        double lo = a, hi = c;
        for (int it = 0; it < 80; ++it) {
          const double mid = 0.5 * (lo + hi);
          if (stationarity(F, a, c, mid) >= 0.0) hi = mid; else lo = mid;
        }
        double nl = 0.5 * (lo + hi);
        nl = std::min(std::max(nl, a + gap), c - gap);
        moved = std::max(moved, std::fabs(nl - l[j]));
        l[j] = nl;
      }
      ++sweeps;
      if (obj_trace) obj_trace[sweeps] = objective(F, l);
      if (moved < 1e-7) break;
    }
  }
  if (n_sweeps) *n_sweeps = sweeps;
  lev[0] = 0.0f; lev[nlev - 1] = 1.0f;
  for (int j = 1; j <= nlev - 2; ++j) lev[j] = (float)l[j];
  return levels_ok(lev, nlev) ? OK : BAD_LEVELS;
}

// Symbol weights (Proposition on the code pmf, App. E), normalised by the total mass:
// p_j = int_{l_{j-1}}^{l_j} (u - l_{j-1})/(l_j - l_{j-1}) dF~ + int_{l_j}^{l_{j+1}} (l_{j+1} - u)/(l_{j+1} - l_j) dF~,
// with only the second term for j = 0 and only the first for the last level.
int qgxo_symbol_pmf(const double* hist, int nbins, const float* lev, int nlev, double* p) {
  if (!levels_ok(lev, nlev) || nbins < 1) return BAD_LEVELS;
  Cdf F(hist, nbins);
  const double total = F.P0[nbins];
  for (int j = 0; j < nlev; ++j) {
    double s = 0.0;
    if (j > 0) {
      const double a = lev[j - 1], c = lev[j];
      s += ((F.moment(1, c) - F.moment(1, a)) - a * (F.moment(0, c) - F.moment(0, a))) / (c - a);
    }
    if (j < nlev - 1) {
      const double a = lev[j], c = lev[j + 1];
      s += (c * (F.moment(0, c) - F.moment(0, a)) - (F.moment(1, c) - F.moment(1, a))) / (c - a);
    }
    p[j] = total > 0.0 ? s / total : (j == 0 ? 1.0 : 0.0);
  }
  return OK;
}

// ------------------------------- operator A(x) -------------------------------------
// dense affine: out_i = fp32( sum_j M_ij x_j + b_i ), fp64 accumulation in j order;
// bilinear game min_x max_y x^T A y with z = (x, y): out = (A y, -A^T x), fp64 accumulation;
// diagonal: out_i = D_i * x_i (one fp32 multiply).
int qgxo_apply_operator(const qgxo_operator* op, const float* x, float* out) {
  const uint64_t d = op->d;
  if (op->kind == 0) {
    for (uint64_t i = 0; i < d; ++i) {
      double s = 0.0;
      for (uint64_t j = 0; j < d; ++j) s += (double)op->mat[i * d + j] * (double)x[j];
      if (op->bias) s += (double)op->bias[i];
      out[i] = (float)s;
    }
    return OK;
  }
  if (op->kind == 1) {
    if (d % 2) return INVALID_ARG;
    const uint64_t n = d / 2;
    const float* xs = x; const float* ys = x + n;
    for (uint64_t i = 0; i < n; ++i) {
      double s = 0.0;
      for (uint64_t j = 0; j < n; ++j) s += (double)op->mat[i * n + j] * (double)ys[j];
      out[i] = (float)s;
    }
    for (uint64_t j = 0; j < n; ++j) {
      double s = 0.0;
      for (uint64_t i = 0; i < n; ++i) s += (double)op->mat[i * n + j] * (double)xs[i];
      out[n + j] = (float)(-s);
    }
    return OK;
  }
  if (op->kind == 2) {
    for (uint64_t i = 0; i < d; ++i) out[i] = op->mat[i] * x[i];
    return OK;
  }
  return INVALID_ARG;
}

// Stochastic dual vectors of the K workers at one point: V_k = A(x) + U_k (Eq. "oracle"),
// one fp32 addition per coordinate; U null means no noise.
// The relative-noise oracles of Assumption 3 (random coordinate descent, random player updating: App. on
// examples): worker k sees A(x) through a random non-negative scale, V_k = A(x) .* S_k with E[S_k] = 1 (S_k = 0 on
// the coordinates that are not drawn, 1/p on those drawn with probability p), so the noise V_k - A(x) vanishes
// where A does.  One fp32 multiplication per coordinate; S null means no noise.
void qgxo_form_dual_vectors_relative(const float* a, const float* S, int K, uint64_t d, float* V) {
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) V[(uint64_t)k * d + i] = S ? a[i] * S[(uint64_t)k * d + i] : a[i];
}

void qgxo_form_dual_vectors(const float* a, const float* U, int K, uint64_t d, float* V) {
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) V[(uint64_t)k * d + i] = U ? a[i] + U[(uint64_t)k * d + i] : a[i];
}

static void form_by_model(const qgxo_operator* op, const float* a, const float* noise, int K, uint64_t d, float* V) {
  if (op->noise_model == 1) qgxo_form_dual_vectors_relative(a, noise, K, d, V);
  else qgxo_form_dual_vectors(a, noise, K, d, V);
}

// One exchange of Algorithm 1: every worker quantizes and encodes its vector, every stream is
// decoded again, and the decoded vectors vhat[K][d] (may be null) and their mean are returned.
// quantizer_off != 0 bypasses quantization and coding (vhat = V), for the textbook reduction.
int qgxo_exchange_full(const float* V, int K, uint64_t d, int bucket, int norm_type,
                       const float* lev, int nlev, const qgxo_codebook* cb, uint64_t seed, uint32_t xid,
                       int quantizer_off, float* vhat_out, float* mean, uint64_t* total_bits) {
  const uint64_t nb = n_buckets(d, bucket);
  std::vector<float> vhat_local;
  float* vhat = vhat_out;
  if (!vhat) { vhat_local.resize((uint64_t)K * d); vhat = vhat_local.data(); }
  if (quantizer_off) {
    for (uint64_t q = 0; q < (uint64_t)K * d; ++q) vhat[q] = V[q];
    if (total_bits) for (int k = 0; k < K; ++k) total_bits[k] = 0;
  } else {
    std::vector<float> norms((uint64_t)K * nb), norms2((uint64_t)K * nb);
    std::vector<uint8_t> sym((uint64_t)K * d), sym2((uint64_t)K * d);
    int st = qgxo_bucket_norms(V, K, d, bucket, norm_type, norms.data());
    if (st) return st;
    st = qgxo_quantize(V, K, d, bucket, lev, nlev, norms.data(), seed, xid, sym.data());
    if (st) return st;
    const uint64_t cap = qgxo_capacity_words(d, bucket, cb->subblock, cb->maxlen);
    std::vector<uint32_t> stream((uint64_t)K * cap), bbits((uint64_t)K * nb);
    std::vector<uint64_t> tot(K);
    st = qgxo_encode(norms.data(), sym.data(), K, d, bucket, cb, stream.data(), cap, bbits.data(), tot.data());
    if (st) return st;
    st = qgxo_decode(stream.data(), cap, bbits.data(), K, d, bucket, cb, norms2.data(), sym2.data());
    if (st) return st;
    st = qgxo_dequantize(norms2.data(), sym2.data(), K, d, bucket, lev, nlev, vhat);
    if (st) return st;
    if (total_bits) for (int k = 0; k < K; ++k) total_bits[k] = tot[k];
  }
  for (uint64_t i = 0; i < d; ++i) {
    float acc = 0.0f;
    for (int k = 0; k < K; ++k) acc = acc + vhat[(uint64_t)k * d + i];
    mean[i] = acc / (float)K;
  }
  return OK;
}

// Level refit at an update step t in U (Algorithm 1, first loop): the sufficient statistic is
// the norm^2-weighted histogram of all buckets of the K current dual vectors; the levels are
// refitted (from quantiles on the first fit, from the current levels afterwards) and, for
// code_type 1, the Huffman code is rebuilt from the symbol weights; code_type 0 keeps the
// fixed-length code, code_type 2 Elias' recursive code (neither depends on the weights).
int qgxo_refit(const float* V, int K, uint64_t d, int bucket, int norm_type, int nbins, int first_fit,
               int code_type, float* lev, int nlev, qgxo_codebook* cb, double* hist_out) {
  std::vector<double> hist(nbins), p(nlev);
  int st = qgxo_histogram(V, K, d, bucket, norm_type, nbins, 1, hist.data());
  if (st) return st;
  st = qgxo_fit_levels(hist.data(), nbins, lev, nlev, first_fit, nullptr, nullptr);
  if (st) return st;
  const int sub = cb->subblock;
  if (code_type == 1) {
    st = qgxo_symbol_pmf(hist.data(), nbins, lev, nlev, p.data());
    if (st) return st;
    st = qgxo_codebook_huffman(p.data(), nlev, sub, cb);
  } else if (code_type == 2) {
    st = qgxo_codebook_elias(nlev, sub, cb);
  } else {
    st = qgxo_codebook_fixed(nlev, sub, cb);
  }
  if (hist_out) for (int j = 0; j < nbins; ++j) hist_out[j] = hist[j];
  return st;
}

// One iteration of Algorithm 1 in its dual-extrapolation instance (two oracle calls):
//   [t in U: refit levels and code on V_{k,t}]
//   X_{t+1/2} = X_t - gamma_t * mean_k Vhat_{k,t}
//   Y_{t+1}   = Y_t - mean_k Vhat_{k,t+1/2}
//   sum_sq   += sum_k ||Vhat_{k,t} - Vhat_{k,t+1/2}||^2          (fp32 differences, fp64 sum)
//   gamma_{t+1} = K / sqrt(1 + sum_sq)
//   X_{t+1}   = anchor + gamma_{t+1} * Y_{t+1}                   (anchor = X_1; the paper takes X_1 = 0)
//   Xbar     += (X_{t+1/2} - Xbar) / t
// Exchange ids 2t and 2t+1 key the two independent quantizer draws.
// refit: 0 none, 1 refit from the current levels, 2 first fit (quantile start).
// Optional outputs (may be null): the two means and the two sets of decoded vectors.
// The iteration with its own level table and code for each of the two exchanges (footnote of Sec. 3.3: one
// sequence of adaptive levels for the V_{k,t} and another one for the V_{k,t+1/2}); lev_t == lev_h and cb_t == cb_h
// give the single-table iteration.  At an update step each table is refitted on its own dual vectors.
static int eg_step_core(qgxo_eg_state* st, const qgxo_operator* op, const float* noise_t, const float* noise_half,
                        int bucket, int norm_type, float* lev_t, int nlev_t, qgxo_codebook* cb_t,
                        float* lev_h, int nlev_h, qgxo_codebook* cb_h,
                        uint64_t seed, int quantizer_off, int refit, int code_type, int nbins, uint64_t* bits_out) {
  const uint64_t d = st->d; const int K = st->K;
  const bool two = (lev_h != lev_t) || (cb_h != cb_t);
  std::vector<float> a(d), V((uint64_t)K * d), vhat1((uint64_t)K * d), vhat2((uint64_t)K * d), mean(d);
  std::vector<uint64_t> tb1(K), tb2(K);
  int rc = qgxo_apply_operator(op, st->X, a.data());
  if (rc) return rc;
  form_by_model(op, a.data(), noise_t, K, d, V.data());
  if (refit && !quantizer_off) {
    rc = qgxo_refit(V.data(), K, d, bucket, norm_type, nbins, refit == 2, code_type, lev_t, nlev_t, cb_t, nullptr);
    if (rc) return rc;
  }
  rc = qgxo_exchange_full(V.data(), K, d, bucket, norm_type, lev_t, nlev_t, cb_t, seed, 2u * (uint32_t)st->t,
                          quantizer_off, vhat1.data(), mean.data(), tb1.data());
  if (rc) return rc;
  for (uint64_t i = 0; i < d; ++i) { const float step = st->gamma * mean[i]; st->Xhalf[i] = st->X[i] - step; }
  rc = qgxo_apply_operator(op, st->Xhalf, a.data());
  if (rc) return rc;
  form_by_model(op, a.data(), noise_half, K, d, V.data());
  if (two && refit && !quantizer_off) {
    rc = qgxo_refit(V.data(), K, d, bucket, norm_type, nbins, refit == 2, code_type, lev_h, nlev_h, cb_h, nullptr);
    if (rc) return rc;
  }
  rc = qgxo_exchange_full(V.data(), K, d, bucket, norm_type, lev_h, nlev_h, cb_h, seed, 2u * (uint32_t)st->t + 1u,
                          quantizer_off, vhat2.data(), mean.data(), tb2.data());
  if (rc) return rc;
  for (uint64_t i = 0; i < d; ++i) st->Y[i] = st->Y[i] - mean[i];
  double s = 0.0;
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) {
      const float diff = vhat1[(uint64_t)k * d + i] - vhat2[(uint64_t)k * d + i];
      s += (double)diff * (double)diff;
    }
  st->sum_sq += s;
  st->gamma = (float)((double)K / std::sqrt(1.0 + st->sum_sq));
  for (uint64_t i = 0; i < d; ++i) { const float gy = st->gamma * st->Y[i]; st->X[i] = st->anchor[i] + gy; }
  const float tf = (float)st->t;
  for (uint64_t i = 0; i < d; ++i) { const float diff = st->Xhalf[i] - st->Xbar[i]; st->Xbar[i] = st->Xbar[i] + diff / tf; }
  st->t += 1;
  if (bits_out) { uint64_t b = 0; for (int k = 0; k < K; ++k) b += tb1[k] + tb2[k]; *bits_out = b; }
  return OK;
}

int qgxo_eg_step(qgxo_eg_state* st, const qgxo_operator* op, const float* noise_t, const float* noise_half,
                 int bucket, int norm_type, float* lev, int nlev, qgxo_codebook* cb,
                 uint64_t seed, int quantizer_off, int refit, int code_type, int nbins, uint64_t* bits_out) {
  return eg_step_core(st, op, noise_t, noise_half, bucket, norm_type, lev, nlev, cb, lev, nlev, cb, seed, quantizer_off,
                      refit, code_type, nbins, bits_out);
}

int qgxo_eg_step_two_tables(qgxo_eg_state* st, const qgxo_operator* op, const float* noise_t, const float* noise_half,
                            int bucket, int norm_type, float* lev_t, int nlev_t, qgxo_codebook* cb_t,
                            float* lev_h, int nlev_h, qgxo_codebook* cb_h,
                            uint64_t seed, int quantizer_off, int refit, int code_type, int nbins, uint64_t* bits_out) {
  if (lev_t == lev_h || cb_t == cb_h) return INVALID_ARG;
  return eg_step_core(st, op, noise_t, noise_half, bucket, norm_type, lev_t, nlev_t, cb_t, lev_h, nlev_h, cb_h, seed,
                      quantizer_off, refit, code_type, nbins, bits_out);
}

// The two other members of the family named in Sec. 3.1, one oracle call and one exchange per iteration.
// method 1, quantized dual averaging (Vhat_{k,t} = 0, hence X_{t+1/2} = X_t):
//   g_{k,t} = Q(A(X_t) + U_{k,t});  Y_{t+1} = Y_t - mean_k g_{k,t};  sum_sq += sum_k ||0 - g_{k,t}||^2
// method 2, quantized optimistic dual averaging (Vhat_{k,t} = g_{k,t-1/2}, the vectors of the previous iteration,
// taken as zero in the first iteration):
//   X_{t+1/2} = X_t - gamma_t * mean_k g_{k,t-1/2};  g_{k,t+1/2} = Q(A(X_{t+1/2}) + U_{k,t+1/2});
//   Y_{t+1} = Y_t - mean_k g_{k,t+1/2};  sum_sq += sum_k ||g_{k,t-1/2} - g_{k,t+1/2}||^2
// both: gamma_{t+1} = K / sqrt(1 + sum_sq), X_{t+1} = anchor + gamma_{t+1} Y_{t+1}, Xbar += (X_{t+1/2} - Xbar) / t.
// A refit (t in U) uses the iteration's only dual vectors.  The exchange id is 2t + 1 (the draw of the second
// exchange of Algorithm 1).  g_prev [K][d] and mean_prev [d] carry g_{k,t-1/2} and its mean from call to call
// (method 2; zero before the first call) and are overwritten.
int qgxo_family_step(qgxo_eg_state* st, int method, const qgxo_operator* op, const float* noise,
                     int bucket, int norm_type, float* lev, int nlev, qgxo_codebook* cb,
                     uint64_t seed, int quantizer_off, int refit, int code_type, int nbins,
                     float* g_prev, float* mean_prev, uint64_t* bits_out) {
  if (method != 1 && method != 2) return INVALID_ARG;
  if (method == 2 && (!g_prev || !mean_prev)) return INVALID_ARG;
  const uint64_t d = st->d; const int K = st->K;
  std::vector<float> a(d), V((uint64_t)K * d), g((uint64_t)K * d), mean(d);
  std::vector<uint64_t> tb(K);
  for (uint64_t i = 0; i < d; ++i) {
    if (method == 2) { const float step = st->gamma * mean_prev[i]; st->Xhalf[i] = st->X[i] - step; }
    else st->Xhalf[i] = st->X[i];
  }
  int rc = qgxo_apply_operator(op, st->Xhalf, a.data());
  if (rc) return rc;
  form_by_model(op, a.data(), noise, K, d, V.data());
  if (refit && !quantizer_off) {
    rc = qgxo_refit(V.data(), K, d, bucket, norm_type, nbins, refit == 2, code_type, lev, nlev, cb, nullptr);
    if (rc) return rc;
  }
  rc = qgxo_exchange_full(V.data(), K, d, bucket, norm_type, lev, nlev, cb, seed, 2u * (uint32_t)st->t + 1u,
                          quantizer_off, g.data(), mean.data(), tb.data());
  if (rc) return rc;
  for (uint64_t i = 0; i < d; ++i) st->Y[i] = st->Y[i] - mean[i];
  double s = 0.0;
  for (int k = 0; k < K; ++k)
    for (uint64_t i = 0; i < d; ++i) {
      const float before = method == 2 ? g_prev[(uint64_t)k * d + i] : 0.0f;
      const float diff = before - g[(uint64_t)k * d + i];
      s += (double)diff * (double)diff;
    }
  st->sum_sq += s;
  st->gamma = (float)((double)K / std::sqrt(1.0 + st->sum_sq));
  for (uint64_t i = 0; i < d; ++i) { const float gy = st->gamma * st->Y[i]; st->X[i] = st->anchor[i] + gy; }
  const float tf = (float)st->t;
  for (uint64_t i = 0; i < d; ++i) { const float diff = st->Xhalf[i] - st->Xbar[i]; st->Xbar[i] = st->Xbar[i] + diff / tf; }
  st->t += 1;
  if (method == 2) {
    for (uint64_t i = 0; i < (uint64_t)K * d; ++i) g_prev[i] = g[i];
    for (uint64_t i = 0; i < d; ++i) mean_prev[i] = mean[i];
  }
  if (bits_out) { uint64_t b = 0; for (int k = 0; k < K; ++k) b += tb[k]; *bits_out = b; }
  return OK;
}

}  // extern "C"
