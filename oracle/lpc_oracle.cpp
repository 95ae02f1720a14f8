// CPU oracle for the LPC-SVRG / ALPC-SVRG per-iteration path (arXiv 1901.08924).
//
// THIS IS TEST INFRASTRUCTURE, not the product.  It is a plain, slow, single-threaded
// restatement of what the paper defines, written to be checked against the paper by eye.
// Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may call it;
// the CUDA library never does, and the two share no source, header, table or helper.
//
// Arithmetic convention: "fp32" below means every operation is one IEEE-754 binary32
// round-to-nearest-even operation with no contraction into fused multiply-add (this file
// must be compiled with -ffp-contract=off and without -ffast-math).  Where fp64 is used
// it is said so.
//
// Pins (see tests/test_oracle_*.py): Philox known-answer vectors; exhaustive enumeration of
// the 16-bit rounding variable for the quantizer's mean and variance (Section 3.2 rule (1),
// Lemma 1); end points and projection (rule (2)); the vector error bound of the
// supplement's Lemma 3; pack/unpack round trips and the bit counts of Table 1; the prox
// against a brute-force scalar minimisation; the SVRG estimator at the snapshot and its
// batch expectation on tiny problems; b=32 against an independently written prox-SVRG loop;
// pairwise sums against fp64.  The b=1 codebook and the c*std clip threshold are extensions
// that the paper does not define: they are pinned by enumeration only ("parity unpinned"
// against the paper for those two readings).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

constexpr int ORC_OK = 0;
constexpr int ORC_ERR_INVALID = -1;
constexpr int ORC_ERR_NONFINITE = -3;

constexpr int LOSS_LOGISTIC = 0;
constexpr int LOSS_LEAST_SQUARES = 1;

constexpr int CLIP_NONE = 0;    // T = ||u||_inf              (Eq. 2 with lambda = 1)
constexpr int CLIP_LAMBDA = 1;  // T = lambda * ||u||_inf     (Eq. 2)
constexpr int CLIP_STD = 2;     // T = min(c * std(u), ||u||_inf)  (the [-c sigma, c sigma] region of Section 3.1)

constexpr uint32_t TAG_ROUND = 0;    // stochastic-rounding stream
constexpr uint32_t TAG_BATCH = 1;    // per-worker minibatch i_B
constexpr uint32_t TAG_BATCH_J = 2;  // shared minibatch J of the double sampling
constexpr uint32_t TAG_REQUANT = 4;   // the server's rounding variables under scheme (c)

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
// SC'11): a 128-bit counter and a 64-bit key go through ten rounds; each round multiplies
// two counter words by fixed odd constants and mixes high/low halves with the key, which
// is advanced by two Weyl constants between rounds.
// ---------------------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
  const uint64_t mul_a = 0xD2511F53u;
  const uint64_t mul_b = 0xCD9E8D57u;
  const uint32_t weyl_a = 0x9E3779B9u;
  const uint32_t weyl_b = 0xBB67AE85u;
  uint32_t c[4] = {ctr_in[0], ctr_in[1], ctr_in[2], ctr_in[3]};
  uint32_t k[2] = {key_in[0], key_in[1]};
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k[0] += weyl_a;
      k[1] += weyl_b;
    }
    const uint64_t prod_a = mul_a * (uint64_t)c[0];
    const uint64_t prod_b = mul_b * (uint64_t)c[2];
    const uint32_t n0 = (uint32_t)(prod_b >> 32) ^ c[1] ^ k[0];
    const uint32_t n1 = (uint32_t)prod_b;
    const uint32_t n2 = (uint32_t)(prod_a >> 32) ^ c[3] ^ k[1];
    const uint32_t n3 = (uint32_t)prod_a;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
  }
  for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// Counter layout used by every stream of the method: word 0 = block index within the
// stream, words 1 and 3 = low and high half of the global iteration k, word 2 = worker
// index in the low 24 bits and the stream tag in the high 8.  The key is the 64-bit seed.
void stream_block(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block,
                  uint32_t out[4]) {
  const uint32_t ctr[4] = {block, (uint32_t)k, (worker & 0xFFFFFFu) | (tag << 24),
                           (uint32_t)(k >> 32)};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  philox4x32_10(ctr, key, out);
}

// The 16-bit rounding variable of coordinate j: eight coordinates share one Philox block;
// coordinate j takes 16-bit lane (j mod 8), lanes numbered from the low half of word 0.
uint32_t rounding_bits(uint64_t seed, uint32_t worker, uint64_t k, uint32_t block_base, int64_t j) {
  uint32_t w[4];
  stream_block(seed, TAG_ROUND, worker, k, block_base + (uint32_t)(j >> 3), w);
  const int lane = (int)(j & 7);
  return (w[lane >> 1] >> (16 * (lane & 1))) & 0xFFFFu;
}

// ---------------------------------------------------------------------------------------
// Pairwise (balanced binary tree) summation in fp32 over the index range padded with
// zeros to the next power of two.  This fixes the rounding order of every fp32 sum the
// method needs, independent of how a parallel machine partitions the range into aligned
// power-of-two blocks.
// ---------------------------------------------------------------------------------------
int64_t next_pow2(int64_t n) {
  int64_t p = 1;
  while (p < n) p <<= 1;
  return p;
}

template <class Leaf>
float tree_reduce(int64_t lo, int64_t width, int64_t n, Leaf leaf) {
  if (lo >= n) return 0.0f;  // padding
  if (width == 1) return leaf(lo);
  const int64_t half = width / 2;
  const float left = tree_reduce(lo, half, n, leaf);
  const float right = tree_reduce(lo + half, half, n, leaf);
  return left + right;
}

float tree_sum(const float* v, int64_t n) {
  if (n <= 0) return 0.0f;
  return tree_reduce(0, next_pow2(n), n, [&](int64_t j) { return v[j]; });
}

float tree_sumsq(const float* v, int64_t n) {
  if (n <= 0) return 0.0f;
  return tree_reduce(0, next_pow2(n), n, [&](int64_t j) { return v[j] * v[j]; });
}

float tree_dot(const float* a, const float* b, int64_t n) {
  if (n <= 0) return 0.0f;
  return tree_reduce(0, next_pow2(n), n, [&](int64_t j) { return a[j] * b[j]; });
}

// ---------------------------------------------------------------------------------------
// Quantizer Q_(delta,b) of Section 2.2 with the scale of Eq. 2.
// ---------------------------------------------------------------------------------------
struct Scale {
  float M = 0.0f;       // ||u||_inf
  float S1 = 0.0f;      // pairwise sum of u        (CLIP_STD only)
  float S2 = 0.0f;      // pairwise sum of u*u      (CLIP_STD only)
  float T = 0.0f;       // clip threshold = largest positive codebook value in exact arithmetic
  float delta = 0.0f;   // codebook spacing (b=1: the magnitude T of the two code points)
  float rdelta = 0.0f;  // 1/delta  (b=1: 1/T)
  bool degenerate = true;
};

int levels(int b) { return (1 << (b - 1)) - 1; }  // number of positive codebook points

int compute_scale(const float* u, int64_t len, int b, int clip_mode, float clip_value, Scale* sc) {
  *sc = Scale();
  float M = 0.0f;
  for (int64_t j = 0; j < len; ++j) {
    if (!std::isfinite(u[j])) return ORC_ERR_NONFINITE;
    const float a = std::fabs(u[j]);
    if (a > M) M = a;
  }
  sc->M = M;
  float T = M;
  if (clip_mode == CLIP_LAMBDA) {
    T = clip_value * M;
  } else if (clip_mode == CLIP_STD) {
    sc->S1 = tree_sum(u, len);
    sc->S2 = tree_sumsq(u, len);
    // fp64 from here to T
    const double mean = (double)sc->S1 / (double)len;
    double var = (double)sc->S2 / (double)len - mean * mean;
    if (var < 0.0) var = 0.0;
    double t = (double)clip_value * std::sqrt(var);
    if (t > (double)M) t = (double)M;  // keeps the effective lambda = T/M inside (0,1]
    T = (float)t;
  }
  sc->T = T;
  if (b == 32) {  // full-precision bypass: no grid, the "code" is the number itself
    sc->delta = 1.0f;
    sc->rdelta = 1.0f;
    sc->degenerate = false;
    return ORC_OK;
  }
  const float delta = (b == 1) ? T : T / (float)levels(b);
  const float rdelta = 1.0f / delta;
  if (M == 0.0f || T == 0.0f || delta == 0.0f || !std::isfinite(rdelta)) {
    // Eq. 2 gives delta = 0 (e.g. u = 0 at the first step of every epoch): send zeros.
    sc->delta = 0.0f;
    sc->rdelta = 0.0f;
    sc->degenerate = true;
    return ORC_OK;
  }
  sc->delta = delta;
  sc->rdelta = rdelta;
  sc->degenerate = false;
  return ORC_OK;
}

// One coordinate, given 1/delta and the 16-bit rounding variable r16 in [0, 65536).
// Returns the signed grid index kq in [-2^(b-1), 2^(b-1)-1]  (b=1: the bit, 0 or 1).
int quantize_coord(float u, float rdelta, int b, uint32_t r16) {
  if (b == 1) {
    float s = u * rdelta;  // u / T
    if (s < -1.0f) s = -1.0f;
    if (s > 1.0f) s = 1.0f;
    const float f = (s + 1.0f) * 0.5f;  // position between the two code points -T and +T
    const bool up = ((float)r16 + 0.5f) < f * 65536.0f;
    return up ? 1 : 0;
  }
  const float lo = -(float)(1 << (b - 1));
  const float hi = (float)levels(b);
  float s = u * rdelta;
  if (s < lo) s = lo;  // rule (2): outside the hull -> smallest ...
  if (s > hi) s = hi;  //                            ... or largest codebook value
  const float fl = std::floor(s);
  // rule (1): round up with probability (x - z)/delta = s - floor(s), realised on a 2^-16 grid.  The
  // fraction is taken in fp64, where it is exact for every fp32 s (an fp32 subtraction would round it
  // when s is negative), and so is the comparison.
  const double f = (double)s - (double)fl;
  const bool up = ((double)r16 + 0.5) < f * 65536.0;
  return (int)fl + (up ? 1 : 0);
}

uint32_t code_of(int kq, int b) { return (b == 1) ? (uint32_t)kq : (uint32_t)(kq + (1 << (b - 1))); }
int index_of(uint32_t code, int b) { return (b == 1) ? 2 * (int)code - 1 : (int)code - (1 << (b - 1)); }

int64_t packed_words(int64_t len, int b) { return (len * (int64_t)b + 31) / 32; }

// Little-endian bit stream: code j occupies stream bits [j*b, (j+1)*b); stream bit p lives
// in word p/32 at bit position p%32.  Unused tail bits are zero.
void put_code(uint32_t* words, int64_t j, int b, uint32_t code) {
  for (int bit = 0; bit < b; ++bit) {
    const int64_t p = j * b + bit;
    if ((code >> bit) & 1u) words[p >> 5] |= (1u << (p & 31));
  }
}

uint32_t get_code(const uint32_t* words, int64_t j, int b) {
  uint32_t code = 0;
  for (int bit = 0; bit < b; ++bit) {
    const int64_t p = j * b + bit;
    if ((words[p >> 5] >> (p & 31)) & 1u) code |= (1u << bit);
  }
  return code;
}

float bits_to_float(uint32_t w) { float f; std::memcpy(&f, &w, 4); return f; }
uint32_t float_to_bits(float f) { uint32_t w; std::memcpy(&w, &f, 4); return w; }

// Decoded value of one received coordinate: delta * index  (b=32: the number itself).
float decode_value(const uint32_t* words, int64_t j, int b, float delta) {
  if (b == 32) return delta * bits_to_float(words[j]);
  return delta * (float)index_of(get_code(words, j, b), b);
}

float soft_threshold(float w, float kappa) {
  float a = std::fabs(w) - kappa;
  if (a < 0.0f) a = 0.0f;
  return std::copysign(a, w);
}

// ---------------------------------------------------------------------------------------
// Linear-model losses of the experiments (Section 5.1): f_a(x) = loss(<X_a, x>, y_a).
// ---------------------------------------------------------------------------------------
float loss_deriv(int loss, float m, float y) {
  if (loss == LOSS_LEAST_SQUARES) return m - y;  // d/dm of (m-y)^2/2
  // logistic log(1+exp(-y m)): derivative -y/(1+exp(y m)), evaluated in fp64, rounded once
  const double t = (double)y * (double)m;
  return (float)(-(double)y / (1.0 + std::exp(t)));
}

double loss_value(int loss, float m, float y) {  // fp64
  if (loss == LOSS_LEAST_SQUARES) {
    const double r = (double)m - (double)y;
    return 0.5 * r * r;
  }
  const double t = (double)y * (double)m;
  return (t > 0.0) ? std::log1p(std::exp(-t)) : (-t + std::log1p(std::exp(t)));
}

}  // namespace

extern "C" {

void orc_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

void orc_stream_block(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block,
                      uint32_t* out) {
  stream_block(seed, tag, worker, k, block, out);
}

uint32_t orc_rounding_bits(uint64_t seed, uint32_t worker, uint64_t k, uint32_t block_base, int64_t j) {
  return rounding_bits(seed, worker, k, block_base, j);
}

float orc_tree_sum(const float* v, int64_t n) { return tree_sum(v, n); }
float orc_tree_sumsq(const float* v, int64_t n) { return tree_sumsq(v, n); }
float orc_tree_dot(const float* a, const float* b, int64_t n) { return tree_dot(a, b, n); }

int64_t orc_packed_words(int64_t len, int b) { return packed_words(len, b); }

// Bits of one worker message (Section 3.2: b bits per coordinate plus one float).
uint64_t orc_message_bits(int64_t len, int b) { return 32u + (uint64_t)b * (uint64_t)len; }
// Bits of one communication step 2 under scheme (a) (Table 1, broadcast row).
uint64_t orc_broadcast_bits(int64_t len, int b, int N) {
  return orc_message_bits(len, b) * (uint64_t)N * (uint64_t)(N - 1);
}

// Scale of Eq. 2.  out = {M, S1, S2, T, delta, rdelta}; *degenerate_out = 1 when delta = 0.
int orc_scale(const float* u, int64_t len, int b, int clip_mode, float clip_value, float* out,
              int* degenerate_out) {
  Scale sc;
  const int rc = compute_scale(u, len, b, clip_mode, clip_value, &sc);
  if (rc != ORC_OK) return rc;
  out[0] = sc.M; out[1] = sc.S1; out[2] = sc.S2; out[3] = sc.T; out[4] = sc.delta; out[5] = sc.rdelta;
  if (degenerate_out) *degenerate_out = sc.degenerate ? 1 : 0;
  return ORC_OK;
}

int orc_quantize_coord(float u, float rdelta, int b, uint32_t r16) {
  return quantize_coord(u, rdelta, b, r16);
}

void orc_pack(const uint32_t* codes, int64_t len, int b, uint32_t* words_out) {
  const int64_t W = packed_words(len, b);
  for (int64_t w = 0; w < W; ++w) words_out[w] = 0;
  for (int64_t j = 0; j < len; ++j) put_code(words_out, j, b, codes[j]);
}

void orc_unpack(const uint32_t* words, int64_t len, int b, uint32_t* codes_out) {
  for (int64_t j = 0; j < len; ++j) codes_out[j] = get_code(words, j, b);
}

// Quantization step (Algorithm 1, step 7) of one worker's vector u (or of one tensor
// segment of it) followed by packing.
//   words_out  : packed_words(len,b) words, fully overwritten
//   delta_out  : the transmitted float (delta; for b=1 the magnitude T; for b=32 1.0)
//   clipped_out: d_lambda, the number of coordinates outside the hull [-(T+delta), T]
//   index_out  : nullable, the signed grid index of every coordinate
int orc_quantize_pack(const float* u, int64_t len, int b, int clip_mode, float clip_value,
                      uint64_t seed, uint32_t worker, uint64_t k, uint32_t block_base,
                      uint32_t* words_out, float* delta_out, uint32_t* clipped_out, int32_t* index_out) {
  if (len < 0 || !((b >= 1 && b <= 16) || b == 32)) return ORC_ERR_INVALID;
  const int64_t W = packed_words(len, b);
  for (int64_t w = 0; w < W; ++w) words_out[w] = 0;
  Scale sc;
  const int rc = compute_scale(u, len, b, clip_mode, clip_value, &sc);
  if (rc != ORC_OK) return rc;
  *delta_out = sc.delta;
  uint32_t clipped = 0;
  for (int64_t j = 0; j < len; ++j) {
    if (b == 32) {
      float v = u[j];
      if (clip_mode != CLIP_NONE) {
        if (v > sc.T) { v = sc.T; ++clipped; }
        if (v < -sc.T) { v = -sc.T; ++clipped; }
      }
      words_out[j] = float_to_bits(v);
      if (index_out) index_out[j] = 0;
      continue;
    }
    int kq;
    if (sc.degenerate) {
      kq = 0;  // b=1 has no zero code point: bit 0, whose decoded value is -0*... = 0 since delta=0
    } else {
      const uint32_t r16 = rounding_bits(seed, worker, k, block_base, j);
      kq = quantize_coord(u[j], sc.rdelta, b, r16);
      const float lower = (b == 1) ? -sc.T : -(sc.T + sc.delta);
      if (u[j] > sc.T || u[j] < lower) ++clipped;
    }
    put_code(words_out, j, b, code_of(kq, b));
    if (index_out) index_out[j] = (b == 1) ? 2 * kq - 1 : kq;
  }
  if (clipped_out) *clipped_out = clipped;
  return ORC_OK;
}

// Scheme (a) (Eq. 3): decode every worker's message with its own delta, average, then
// Algorithm 1 steps 9-10 with h = lambda_l1*||.||_1:
//   v = u~ + mu ;  x+ = prox_{eta h}(x - eta v) = soft-threshold(x - eta v, eta*lambda_l1)
// words: N streams, stream i starts at words + i*stride_words.  mu nullable (= 0).
void orc_unpack_average_prox(const uint32_t* words, int64_t stride_words, const float* delta, int N,
                             int64_t len, int b, const float* mu, float* x_inout, float eta,
                             float lambda_l1, float* v_out, float* utilde_out) {
  const float invN = 1.0f / (float)N;
  const float kappa = eta * lambda_l1;
  for (int64_t j = 0; j < len; ++j) {
    float acc = 0.0f;
    for (int i = 0; i < N; ++i) acc = acc + decode_value(words + (int64_t)i * stride_words, j, b, delta[i]);
    const float ut = acc * invN;
    const float v = ut + (mu ? mu[j] : 0.0f);
    const float w = x_inout[j] - eta * v;
    x_inout[j] = soft_threshold(w, kappa);
    if (v_out) v_out[j] = v;
    if (utilde_out) utilde_out[j] = ut;
  }
}

float orc_soft_threshold(float w, float kappa) { return soft_threshold(w, kappa); }

}  // extern "C"

// ---------------------------------------------------------------------------------------
// Parameter-server schemes (b) and (c) of Section 3.2.
//
// Both unify the scale first: delta_t = max_i delta_t^i, and every worker quantizes with delta_t in
// step 7.  delta^i = T^i / levels is monotone in the threshold T^i, so the
// shared scale is the scale of the worker with the largest threshold; a worker whose own vector is all
// zero then simply sends zero codes on the shared grid.  If every worker is degenerate so is the result.
//
// (b) The server adds the signed grid indices, K_j = sum_i k_ij, which takes the ceil(log2 N) more bits
//     per coordinate that the scheme grants the sum, and sends the sums back; a worker recovers
//     u~_j = (delta_t * K_j) / N  (Eq. 3 with a common delta).  The sum is stored like any other code
//     stream, in offset binary with b' = b + ceil(log2 N) bits: K_j + 2^(b'-1).
// (c) The server averages and quantizes again with the same grid, u~ = Q_(delta_t,b)(avg) (Eq. 4):
//     in grid units the average is s_j = K_j / N (one fp32 division), already inside the hull, and
//     rule (1) of Section 2.2 rounds it with the server's own rounding stream; b bits go back.
// The two-point extension b = 1 and the bypass b = 32 have no integer grid to add on: not offered.
// ---------------------------------------------------------------------------------------
int ceil_log2(int N) {
  int r = 0;
  while ((1 << r) < N) ++r;
  return r;
}

extern "C" {

int orc_sum_bits_per_coordinate(int b, int N) { return b + ceil_log2(N); }

// Table 1: bits of one communication step 2.  scheme 0: (a) broadcast (32+bd)N(N-1);
// 1: (b) N(64 + 2bd + d ceil(log N));  2: (c) N(64 + 2bd).
uint64_t orc_scheme_bits(int scheme, int64_t d, int b, int N) {
  const uint64_t bd = (uint64_t)b * (uint64_t)d;
  if (scheme == 0) return (32u + bd) * (uint64_t)N * (uint64_t)(N - 1);
  if (scheme == 1) return (uint64_t)N * (64u + 2u * bd + (uint64_t)d * (uint64_t)ceil_log2(N));
  return (uint64_t)N * (64u + 2u * bd);
}

// Step 7 of Algorithm 1 for all N workers with the unified scale.  U: N vectors, vector i at U + i*ld.
// words_out: N streams, stream i at words_out + i*stride_words.  delta_out: the one shared float.
// clipped_out (nullable): N counts of coordinates outside the shared hull.  block_base: first block of
// the rounding streams (a tensor segment of a longer vector continues the count of its predecessors).
int orc_quantize_pack_shared(const float* U, int N, int64_t len, int64_t ld, int b, int clip_mode,
                             float clip_value, uint64_t seed, uint64_t k, uint32_t block_base, uint32_t* words_out,
                             int64_t stride_words, float* delta_out, uint32_t* clipped_out) {
  if (len < 0 || N < 1 || b < 2 || b > 16) return ORC_ERR_INVALID;
  Scale best;
  bool have = false;
  for (int i = 0; i < N; ++i) {
    Scale sc;
    const int rc = compute_scale(U + (int64_t)i * ld, len, b, clip_mode, clip_value, &sc);
    if (rc != ORC_OK) return rc;
    if (!sc.degenerate && (!have || sc.T > best.T)) { best = sc; have = true; }
  }
  *delta_out = have ? best.delta : 0.0f;
  const int64_t W = packed_words(len, b);
  for (int i = 0; i < N; ++i) {
    const float* u = U + (int64_t)i * ld;
    uint32_t* words = words_out + (int64_t)i * stride_words;
    for (int64_t w = 0; w < W; ++w) words[w] = 0;
    uint32_t clipped = 0;
    for (int64_t j = 0; j < len; ++j) {
      int kq = 0;
      if (have) {
        kq = quantize_coord(u[j], best.rdelta, b, rounding_bits(seed, (uint32_t)i, k, block_base, j));
        if (u[j] > best.T || u[j] < -(best.T + best.delta)) ++clipped;
      }
      put_code(words, j, b, code_of(kq, b));
    }
    if (clipped_out) clipped_out[i] = clipped;
  }
  return ORC_OK;
}

// The server of schemes (b) (requantize = 0) and (c) (requantize = 1).  out: one stream of
// b + ceil(log2 N) bits per coordinate (b), or of b bits (c).
int orc_server_reduce(const uint32_t* words, int64_t stride_words, int N, int64_t len, int b,
                      int requantize, uint64_t seed, uint64_t k, uint32_t block_base, uint32_t* out) {
  if (len < 0 || N < 1 || b < 2 || b > 16) return ORC_ERR_INVALID;
  const int bo = requantize ? b : b + ceil_log2(N);
  if (bo > 16) return ORC_ERR_INVALID;
  const int64_t W = packed_words(len, bo);
  for (int64_t w = 0; w < W; ++w) out[w] = 0;
  for (int64_t j = 0; j < len; ++j) {
    int K = 0;
    for (int i = 0; i < N; ++i) K += index_of(get_code(words + (int64_t)i * stride_words, j, b), b);
    if (!requantize) {
      put_code(out, j, bo, code_of(K, bo));
    } else {
      const float s = (float)K / (float)N;  // the average in grid units
      uint32_t w4[4];
      stream_block(seed, TAG_REQUANT, 0, k, block_base + (uint32_t)(j >> 3), w4);
      const int lane = (int)(j & 7);
      const uint32_t r16 = (w4[lane >> 1] >> (16 * (lane & 1))) & 0xFFFFu;
      put_code(out, j, b, code_of(quantize_coord(s, 1.0f, b, r16), b));
    }
  }
  return ORC_OK;
}

// ---------------------------------------------------------------------------------------
// Entropy coding of a message (Section 5.1: the experiments pass the codes through Huffman's code
// [huffman1952method] to cut the traffic further).  The paper gives no format; what is counted here is
// the payload alone: from the histogram of a message's 2^b code values, (i) the empirical entropy
// n * H = -sum_c count_c * log2(count_c / n), the bound no symbol code can beat, and (ii) the length of
// the message under a Huffman code built for that histogram, sum_c count_c * len_c.  The code table and
// the 32-bit scale are not included.  A message with one distinct value still spends one bit per
// coordinate under (ii) (a code word cannot be empty).
// ---------------------------------------------------------------------------------------
// hist_out: 2^b counts.
int orc_code_histogram(const uint32_t* words, int64_t len, int b, uint64_t* hist_out) {
  if (len < 0 || b < 1 || b > 16) return ORC_ERR_INVALID;
  for (int c = 0; c < (1 << b); ++c) hist_out[c] = 0;
  for (int64_t j = 0; j < len; ++j) hist_out[get_code(words, j, b)] += 1;
  return ORC_OK;
}

// n * H in bits (fp64) for a histogram of `bins` counts.
double orc_entropy_bits(const uint64_t* hist, int bins) {
  uint64_t n = 0;
  for (int c = 0; c < bins; ++c) n += hist[c];
  double bits = 0.0;
  for (int c = 0; c < bins; ++c)
    if (hist[c] > 0) bits -= (double)hist[c] * std::log2((double)hist[c] / (double)n);
  return bits;
}

// Total length in bits under Huffman's construction: repeatedly merge the two lightest subtrees; every
// merge adds the merged weight once (each symbol below it gets one bit longer).
uint64_t orc_huffman_bits(const uint64_t* hist, int bins) {
  uint64_t w[1 << 16];
  int m = 0;
  for (int c = 0; c < bins; ++c)
    if (hist[c] > 0) w[m++] = hist[c];
  if (m == 0) return 0;
  if (m == 1) return w[0];
  uint64_t total = 0;
  while (m > 1) {
    int a = 0, b2 = 1;  // indices of the two smallest weights, by plain search
    if (w[b2] < w[a]) { a = 1; b2 = 0; }
    for (int i = 2; i < m; ++i) {
      if (w[i] < w[a]) { b2 = a; a = i; }
      else if (w[i] < w[b2]) { b2 = i; }
    }
    const uint64_t merged = w[a] + w[b2];
    total += merged;
    const int hi = a > b2 ? a : b2, lo = a > b2 ? b2 : a;
    w[lo] = merged;
    w[hi] = w[m - 1];
    --m;
  }
  return total;
}

// A worker's side after the server's message: u~_j = (delta * index_j) / divisor, then Algorithm 1
// steps 9-10 as in orc_unpack_average_prox.  Scheme (b): bits = b + ceil(log2 N), divisor = N;
// scheme (c): bits = b, divisor = 1.
void orc_unpack_scaled_prox(const uint32_t* words, float delta, int64_t len, int bits, int divisor,
                            const float* mu, float* x_inout, float eta, float lambda_l1, float* v_out,
                            float* utilde_out) {
  const float inv = 1.0f / (float)divisor;
  const float kappa = eta * lambda_l1;
  for (int64_t j = 0; j < len; ++j) {
    const float acc = 0.0f + decode_value(words, j, bits, delta);
    const float ut = acc * inv;
    const float v = ut + (mu ? mu[j] : 0.0f);
    const float w = x_inout[j] - eta * v;
    x_inout[j] = soft_threshold(w, kappa);
    if (v_out) v_out[j] = v;
    if (utilde_out) utilde_out[j] = ut;
  }
}

}  // extern "C"

extern "C" {


// ---- linear model ---------------------------------------------------------------------

float orc_margin(const float* Xa, const float* x, int64_t d) { return tree_dot(Xa, x, d); }
float orc_loss_deriv(int loss, float m, float y) { return loss_deriv(loss, m, y); }
double orc_loss_value(int loss, float m, float y) { return loss_value(loss, m, y); }

// Communication step 1 (Algorithm 1, step 4): mu = grad f(x) = (1/n) sum_a l'(<X_a,x>, y_a) X_a,
// accumulated in fp64 and rounded once; also the margins and f(x) = (1/n) sum_a f_a(x) (fp64).
void orc_full_grad(const float* X, const float* y, int64_t n, int64_t d, int loss, const float* x,
                   float* mu_out, float* margins_out, double* f_out) {
  std::vector<double> acc((size_t)d, 0.0);
  double fsum = 0.0;
  for (int64_t a = 0; a < n; ++a) {
    const float* Xa = X + a * d;
    const float m = tree_dot(Xa, x, d);
    if (margins_out) margins_out[a] = m;
    const double g = (double)loss_deriv(loss, m, y[a]);
    fsum += loss_value(loss, m, y[a]);
    for (int64_t j = 0; j < d; ++j) acc[(size_t)j] += g * (double)Xa[j];
  }
  if (mu_out)
    for (int64_t j = 0; j < d; ++j) mu_out[j] = (float)(acc[(size_t)j] / (double)n);
  if (f_out) *f_out = fsum / (double)n;
}

// P(x) = f(x) + lambda_l1 ||x||_1  (Eq. 1), fp64.
double orc_objective(const float* X, const float* y, int64_t n, int64_t d, int loss, const float* x,
                     float lambda_l1) {
  double f = 0.0;
  orc_full_grad(X, y, n, d, loss, x, nullptr, nullptr, &f);
  double l1 = 0.0;
  for (int64_t j = 0; j < d; ++j) l1 += std::fabs((double)x[j]);
  return f + (double)lambda_l1 * l1;
}

// Minibatch of size B, uniform with replacement (Algorithm 1, step 6) from the row range
// [lo, lo+span): slot a uses word 0 of block a of the (tag, worker, k) stream.
void orc_sample_batch(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, int B, int64_t lo,
                      int64_t span, int64_t* idx_out) {
  for (int a = 0; a < B; ++a) {
    uint32_t w[4];
    stream_block(seed, tag, worker, k, (uint32_t)a, w);
    idx_out[a] = lo + (int64_t)(((uint64_t)w[0] * (uint64_t)span) >> 32);
  }
}

// Coefficients c_a = l'(<X_a,x>,y_a) - l'(<X_a,x~>,y_a) of the SVRG difference.
void orc_svrg_coef(const float* X, const float* y, int64_t d, int loss, const int64_t* idx, int B,
                   const float* x, const float* xs, float* coef_out) {
  for (int a = 0; a < B; ++a) {
    const float* Xa = X + idx[a] * d;
    const float g_cur = loss_deriv(loss, tree_dot(Xa, x, d), y[idx[a]]);
    const float g_snap = loss_deriv(loss, tree_dot(Xa, xs, d), y[idx[a]]);
    coef_out[a] = g_cur - g_snap;
  }
}

// u = (1/B) sum_a c_a X_a (Algorithm 1, step 6), summed in batch order, fp32.
void orc_svrg_diff_from_coef(const float* X, int64_t d, const int64_t* idx, int B, const float* coef,
                             float* u_out) {
  const float invB = 1.0f / (float)B;
  for (int64_t j = 0; j < d; ++j) {
    float acc = 0.0f;
    for (int a = 0; a < B; ++a) acc = acc + coef[a] * X[idx[a] * d + j];
    u_out[j] = acc * invB;
  }
}

// One inner iteration of Algorithm 1 (steps 6-10) for all N workers under scheme (a).
//   x_inout: x_t in, x_{t+1} out.  xs = snapshot, mu = grad f(snapshot).
//   partition_local != 0: worker i samples from its contiguous row block of n/N rows;
//   otherwise from all n rows (the paper's data-parallel setting).
//   Outputs (all nullable): idx N*B, coef N*B, u N*d, words N*stride_words, delta N,
//   clipped N, v d.
int orc_lpc_inner_step(const float* X, const float* y, int64_t n, int64_t d, int loss, float lambda_l1,
                       int N, int B, int b, int clip_mode, float clip_value, uint64_t seed,
                       int partition_local, uint64_t k, float eta, const float* xs, const float* mu,
                       float* x_inout, int64_t* idx_out, float* coef_out, float* u_out,
                       uint32_t* words_out, int64_t stride_words, float* delta_out,
                       uint32_t* clipped_out, float* v_out) {
  const int64_t W = packed_words(d, b);
  if (words_out && stride_words < W) return ORC_ERR_INVALID;
  const int64_t stride = words_out ? stride_words : W;
  std::vector<uint32_t> words_local;
  uint32_t* words = words_out;
  if (!words) { words_local.assign((size_t)(stride * N), 0u); words = words_local.data(); }
  std::vector<float> delta((size_t)N), u((size_t)d), coef((size_t)B);
  std::vector<int64_t> idx((size_t)B);
  const int64_t n_i = n / N;
  for (int i = 0; i < N; ++i) {
    const int64_t lo = partition_local ? (int64_t)i * n_i : 0;
    const int64_t span = partition_local ? n_i : n;
    orc_sample_batch(seed, TAG_BATCH, (uint32_t)i, k, B, lo, span, idx.data());
    orc_svrg_coef(X, y, d, loss, idx.data(), B, x_inout, xs, coef.data());
    orc_svrg_diff_from_coef(X, d, idx.data(), B, coef.data(), u.data());
    for (int64_t w = 0; w < stride; ++w) words[(int64_t)i * stride + w] = 0;
    uint32_t clipped = 0;
    const int rc = orc_quantize_pack(u.data(), d, b, clip_mode, clip_value, seed, (uint32_t)i, k, 0u,
                                     words + (int64_t)i * stride, &delta[(size_t)i], &clipped, nullptr);
    if (rc != ORC_OK) return rc;
    if (idx_out) for (int a = 0; a < B; ++a) idx_out[(int64_t)i * B + a] = idx[(size_t)a];
    if (coef_out) for (int a = 0; a < B; ++a) coef_out[(int64_t)i * B + a] = coef[(size_t)a];
    if (u_out) for (int64_t j = 0; j < d; ++j) u_out[(int64_t)i * d + j] = u[(size_t)j];
    if (delta_out) delta_out[i] = delta[(size_t)i];
    if (clipped_out) clipped_out[i] = clipped;
  }
  orc_unpack_average_prox(words, stride, delta.data(), N, d, b, mu, x_inout, eta, lambda_l1, v_out, nullptr);
  return ORC_OK;
}

// One inner iteration of Algorithm 2 (steps 5-13), h = lambda_l1*||.||_1.
//   coupling   x = tau1*z + tau2*xs + (1-tau1-tau2)*y
//   v          low-precision estimator at x (as in Algorithm 1)
//   v^         full-precision estimator on the shared batch J drawn from all n rows
//   y+ = argmin 2L||y-x||^2 + <v,y> + h(y)        = soft(x - v/(4L), lambda_l1/(4L))
//   z+ = argmin ||z-z_k||^2/(2 alpha) + <v^,z> + h = soft(z - alpha v^, alpha*lambda_l1)
//   ysum += y+   (Algorithm 3's snapshot is the mean of the epoch's y iterates)
//
// Strongly convex case (Algorithm 2 as printed): h(x) = lambda_l1*||x||_1 + (sigma/2)*||x||^2.  Completing the
// square in the two argmins gives the plain soft-threshold results divided by (1 + sigma/(4L)) and by
// (1 + alpha*sigma):
//   y+ = soft(x - v/(4L), lambda_l1/(4L)) * cy,   cy = 1 / (1 + sigma*inv4L)
//   z+ = soft(z - alpha v^, alpha*lambda_l1) * cz, cz = 1 / (1 + alpha*sigma)
// and the snapshot of Algorithm 2's last step weighs y_{sm+t+1} by (1 + alpha*sigma)^t: the caller passes that
// weight (1, theta, theta*theta, ... formed by repeated fp32 multiplication) and ysum += weight * y+.
// sigma = 0, weight = 1 multiply by exactly 1 and reproduce the general convex step bit for bit.
int orc_alpc_step_sc(const float* X, const float* y, int64_t n, int64_t d, int loss, float lambda_l1, int N,
                     int B, int b, int clip_mode, float clip_value, uint64_t seed, int partition_local,
                     uint64_t k, float tau1, float tau2, float alpha, float inv4L, float sigma, float weight,
                     const float* xs, const float* mu, float* y_inout, float* z_inout, float* ysum_inout,
                     float* x_out, float* v_out, float* vhat_out, uint32_t* words_out, int64_t stride_words,
                     float* delta_out) {
  const float tau3 = (1.0f - tau1) - tau2;
  std::vector<float> x((size_t)d), xq((size_t)d), v((size_t)d), uj((size_t)d), coef((size_t)B);
  std::vector<int64_t> idx((size_t)B);
  for (int64_t j = 0; j < d; ++j)
    x[(size_t)j] = (tau1 * z_inout[j] + tau2 * xs[j]) + tau3 * y_inout[j];
  // low-precision estimator: run Algorithm 1's steps 6-9 at x with eta = 0 and no prox effect,
  // taking only v from them
  xq = x;
  const int rc = orc_lpc_inner_step(X, y, n, d, loss, 0.0f, N, B, b, clip_mode, clip_value, seed,
                                    partition_local, k, 0.0f, xs, mu, xq.data(), nullptr, nullptr, nullptr,
                                    words_out, stride_words, delta_out, nullptr, v.data());
  if (rc != ORC_OK) return rc;
  // double sampling: the same J on every worker, full precision, nothing transmitted
  orc_sample_batch(seed, TAG_BATCH_J, 0u, k, B, 0, n, idx.data());
  orc_svrg_coef(X, y, d, loss, idx.data(), B, x.data(), xs, coef.data());
  orc_svrg_diff_from_coef(X, d, idx.data(), B, coef.data(), uj.data());
  const float kappa_y = inv4L * lambda_l1;
  const float kappa_z = alpha * lambda_l1;
  const float cy = 1.0f / (1.0f + sigma * inv4L);
  const float cz = 1.0f / (1.0f + alpha * sigma);
  for (int64_t j = 0; j < d; ++j) {
    const float vhat = uj[(size_t)j] + mu[j];
    const float ynew = soft_threshold(x[(size_t)j] - inv4L * v[(size_t)j], kappa_y) * cy;
    const float znew = soft_threshold(z_inout[j] - alpha * vhat, kappa_z) * cz;
    y_inout[j] = ynew;
    z_inout[j] = znew;
    if (ysum_inout) ysum_inout[j] = ysum_inout[j] + weight * ynew;
    if (x_out) x_out[j] = x[(size_t)j];
    if (v_out) v_out[j] = v[(size_t)j];
    if (vhat_out) vhat_out[j] = vhat;
  }
  return ORC_OK;
}

// The general convex step (Algorithm 3 runs it with its own tau1, alpha per epoch): h = lambda_l1*||.||_1.
int orc_alpc_step(const float* X, const float* y, int64_t n, int64_t d, int loss, float lambda_l1, int N,
                  int B, int b, int clip_mode, float clip_value, uint64_t seed, int partition_local,
                  uint64_t k, float tau1, float tau2, float alpha, float inv4L, const float* xs,
                  const float* mu, float* y_inout, float* z_inout, float* ysum_inout, float* x_out,
                  float* v_out, float* vhat_out, uint32_t* words_out, int64_t stride_words,
                  float* delta_out) {
  return orc_alpc_step_sc(X, y, n, d, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, partition_local, k,
                          tau1, tau2, alpha, inv4L, 0.0f, 1.0f, xs, mu, y_inout, z_inout, ysum_inout, x_out,
                          v_out, vhat_out, words_out, stride_words, delta_out);
}

// Algorithm 2's snapshot: x~ = (sum_t w_t)^-1 * sum_t w_t y_{sm+t+1}, given the weighted sum and the weights'
// sum (both accumulated in fp32 in step order): one reciprocal, one multiplication per coordinate.
void orc_weighted_snapshot(const float* ysum, float wsum, int64_t d, float* xs_out) {
  const float inv = 1.0f / wsum;
  for (int64_t j = 0; j < d; ++j) xs_out[j] = ysum[j] * inv;
}

// Algorithm 3 (general convex case), its outer rule.  Epoch s runs Algorithm 2's steps 3-14 with
//   tau_{1,s} = 2/(s+4),   alpha_s = 1/(6 L tau_{1,s})      (step 3; evaluated in fp64, rounded to fp32 once each)
// and tau_2 as given; its snapshot is the plain mean of the epoch's m iterates y (step 5), taken as the running
// fp32 sum of the y's in step order times the fp32 reciprocal of m.  y and z carry over from epoch to epoch.
void orc_alpc3_epoch_params(int64_t s, double L, float* tau1_out, float* alpha_out) {
  const double tau1 = 2.0 / (double)(s + 4);
  *tau1_out = (float)tau1;
  *alpha_out = (float)(1.0 / (6.0 * L * tau1));
}

void orc_alpc3_mean_snapshot(const float* ysum, int64_t m, int64_t d, float* xs_out) {
  const float inv_m = 1.0f / (float)m;
  for (int64_t j = 0; j < d; ++j) xs_out[j] = ysum[j] * inv_m;
}

// One epoch of Algorithm 3 after communication step 1 (mu = grad f(xs) is given): m steps k = s*m .. s*m + m - 1 with
// the epoch's parameters, then the mean snapshot.  inv4L = 1/(4L) rounded to fp32.
int orc_alpc3_epoch(const float* X, const float* y, int64_t n, int64_t d, int loss, float lambda_l1, int N, int B,
                    int b, int clip_mode, float clip_value, uint64_t seed, int partition_local, int64_t s, int64_t m,
                    double L, float tau2, const float* xs, const float* mu, float* y_inout, float* z_inout,
                    float* xs_next_out) {
  float tau1, alpha;
  orc_alpc3_epoch_params(s, L, &tau1, &alpha);
  const float inv4L = (float)(1.0 / (4.0 * L));
  std::vector<float> ysum((size_t)d, 0.0f);
  for (int64_t t = 0; t < m; ++t) {
    const int rc = orc_alpc_step(X, y, n, d, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, partition_local,
                                 (uint64_t)(s * m + t), tau1, tau2, alpha, inv4L, xs, mu, y_inout, z_inout,
                                 ysum.data(), nullptr, nullptr, nullptr, nullptr, 0, nullptr);
    if (rc != ORC_OK) return rc;
  }
  orc_alpc3_mean_snapshot(ysum.data(), m, d, xs_next_out);
  return ORC_OK;
}

// P(x) with the elastic-net regulariser: the objective of Eq. 1 plus (sigma/2)*||x||^2 (fp64 sum).
double orc_ridge_term(const float* x, int64_t d, float sigma) {
  double s2 = 0.0;
  for (int64_t j = 0; j < d; ++j) s2 += (double)x[j] * (double)x[j];
  return 0.5 * (double)sigma * s2;
}

}  // extern "C"
