// Communication step 2 under scheme (a) (Eq. 3) fused with Algorithm 1 steps 9-10: every worker's
// packed message is decoded with its own delta, the decoded vectors are averaged, the snapshot
// gradient is added and the proximal (soft-threshold) step is applied, in one pass.  The same
// kernel, in its second mode, applies Algorithm 2's y- and z-updates instead.
//
// A thread owns 8 consecutive coordinates per sweep: per worker it loads the 8*b bits that hold
// their codes (b whole bytes, naturally aligned when b is 1, 2, 4, 8 or 16), and accumulates
// delta_i * index in worker order, every operation a separate fp32 round-to-nearest operation.
#include "lpc_device.cuh"
#include "lpc_kernels.h"

namespace lpc {
namespace {

constexpr int AT = 256;
constexpr int AGROUP = AT * 8;
constexpr int AITER = TILE / AGROUP;

__device__ __forceinline__ bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__device__ __forceinline__ void load8f(const float* __restrict__ p, int64_t j, int64_t len, bool vec, float* v) {
  if (vec && j + 8 <= len) {
    const float4 a = *reinterpret_cast<const float4*>(p + j);
    const float4 c = *reinterpret_cast<const float4*>(p + j + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = (j + e < len) ? p[j + e] : 0.f;
  }
}
__device__ __forceinline__ void store8f(float* __restrict__ p, int64_t j, int64_t len, bool vec, const float* v) {
  if (vec && j + 8 <= len) {
    *reinterpret_cast<float4*>(p + j) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(p + j + 4) = make_float4(v[4], v[5], v[6], v[7]);
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (j + e < len) p[j + e] = v[e];
  }
}

// The 8*b bits of coordinate group j/8 of one worker's segment stream, as (lo, hi).
template <int BITS>
__device__ __forceinline__ void load_chunk(const uint32_t* __restrict__ w, int64_t g, int b, int64_t pad_words,
                                           uint64_t& lo, uint64_t& hi) {
  hi = 0;
  if (BITS == 8) {
    const uint2 t = *reinterpret_cast<const uint2*>(w + g * 2);
    lo = (uint64_t)t.x | ((uint64_t)t.y << 32);
  } else if (BITS == 4) {
    lo = w[g];
  } else if (BITS == 2) {
    lo = reinterpret_cast<const uint16_t*>(w)[g];
  } else if (BITS == 1) {
    lo = reinterpret_cast<const uint8_t*>(w)[g];
  } else if (BITS == 3) {
    // three bytes at byte 3 g: from the aligned word that holds the first and, where they run over, the next one
    const int64_t idx = (3 * g) >> 2;
    const int sh = (int)((3 * g) & 3) * 8;
    const uint32_t w0 = w[idx], w1 = (sh > 8 && idx + 1 < pad_words) ? w[idx + 1] : 0u;
    lo = __funnelshift_r(w0, w1, sh) & 0xFFFFFFu;
  } else {
    const uint8_t* bytes = reinterpret_cast<const uint8_t*>(w);
    const int64_t b0 = g * b, limit = pad_words * 4;
    lo = 0;
    for (int i = 0; i < b; ++i) {
      const uint64_t v = (b0 + i < limit) ? bytes[b0 + i] : 0;
      if (i < 8) lo |= v << (8 * i); else hi |= v << (8 * (i - 8));
    }
  }
}

__device__ __forceinline__ uint32_t extract(uint64_t lo, uint64_t hi, int pos, int b) {
  uint64_t v;
  if (pos < 64) {
    v = lo >> pos;
    if (pos + b > 64) v |= hi << (64 - pos);
  } else {
    v = hi >> (pos - 64);
  }
  return (uint32_t)v & ((1u << b) - 1u);
}

template <int BITS>  // 1, 2, 3, 4, 8: fixed width; 0: b in 1..16 from the arguments; 32: floats
__global__ void __launch_bounds__(AT) unpack_average_prox_kernel(AggArgs a) {
  // a.split CTAs share a tile (each takes AITER / split of its sweeps): short vectors still fill the machine
  const int tile = blockIdx.x / a.split, part = blockIdx.x % a.split;
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  const SegInfo s = a.segs[seg];
  const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
  const int tid = threadIdx.x;
  const int b = (BITS == 0) ? a.b : BITS;

  extern __shared__ float sdelta[];
  for (int i = tid; i < a.N; i += AT) sdelta[i] = a.delta[(int64_t)i * a.nseg + seg];
  __syncthreads();

  const float invN = __fdiv_rn(1.0f, (float)a.divisor);
  float* xs = a.x + s.off;
  const float* mus = a.mu ? a.mu + s.off : nullptr;
  float* vs = a.v_out ? a.v_out + s.off : nullptr;
  const bool vec = aligned16(xs) && (!mus || aligned16(mus)) && (!vs || aligned16(vs)) &&
                   (a.mode == 0 || (aligned16(a.y + s.off) && aligned16(a.z + s.off) && aligned16(a.ysum + s.off) &&
                                    aligned16(a.vhat + s.off)));

#pragma unroll 1
  for (int it = part * (AITER / a.split); it < (part + 1) * (AITER / a.split); ++it) {
    const int64_t j = tstart + (int64_t)it * AGROUP + tid * 8;
    if (j >= s.len) break;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    const uint32_t* w = a.codes + s.word_off;
    if constexpr (BITS == 32) {
#pragma unroll 2
      for (int i = 0; i < a.N; ++i) {
        const uint32_t* wi = w + (int64_t)i * a.stride_words;
        const float di = sdelta[i];
        float val[8];
        load8f(reinterpret_cast<const float*>(wi), j, s.len, true, val);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = add_rn(acc[e], mul_rn(di, val[e]));
      }
    } else {
#pragma unroll 8
      for (int i = 0; i < a.N; ++i) {
        uint64_t lo, hi;
        load_chunk<BITS>(w + (int64_t)i * a.stride_words, j >> 3, b, s.pad_words, lo, hi);
        const float di = sdelta[i];
        float kf[8];
        if constexpr (BITS == 0) {
#pragma unroll
          for (int e = 0; e < 8; ++e) kf[e] = index_as_float(extract(lo, hi, e * b, b), b);
        } else {
          decode8<(BITS == 0 || BITS == 32) ? 1 : BITS>(lo, kf);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = add_scaled_index<BITS>(acc[e], di, kf[e]);
      }
    }
    float xv[8], mv[8], vv[8];
    load8f(xs, j, s.len, vec, xv);
    if (mus) {
      load8f(mus, j, s.len, vec, mv);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) mv[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) vv[e] = add_rn(mul_rn(acc[e], invN), mv[e]);
    if (vs) store8f(vs, j, s.len, vec, vv);
    if (a.mode == 0) {
      const float kappa = mul_rn(a.eta, a.lambda_l1);
#pragma unroll
      for (int e = 0; e < 8; ++e) xv[e] = soft_threshold(__fsub_rn(xv[e], mul_rn(a.eta, vv[e])), kappa);
      store8f(xs, j, s.len, vec, xv);
    } else {
      float zv[8], hv[8], sv[8], yv[8];
      load8f(a.z + s.off, j, s.len, vec, zv);
      load8f(a.vhat + s.off, j, s.len, vec, hv);
      load8f(a.ysum + s.off, j, s.len, vec, sv);
      const float ky = mul_rn(a.inv4L, a.lambda_l1), kz = mul_rn(a.alpha, a.lambda_l1);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        yv[e] = mul_rn(soft_threshold(__fsub_rn(xv[e], mul_rn(a.inv4L, vv[e])), ky), a.cy);
        zv[e] = mul_rn(soft_threshold(__fsub_rn(zv[e], mul_rn(a.alpha, hv[e])), kz), a.cz);
        sv[e] = add_rn(sv[e], mul_rn(a.wy, yv[e]));
      }
      store8f(a.y + s.off, j, s.len, vec, yv);
      store8f(a.z + s.off, j, s.len, vec, zv);
      store8f(a.ysum + s.off, j, s.len, vec, sv);
    }
  }
  if (a.k_counter && blockIdx.x == 0 && tid == 0) *a.k_counter += 1;
}

// The server of schemes (b) and (c) (Section 3.2).  A thread owns 8 consecutive coordinates per sweep: it adds the
// codes of the N streams as integers, then either stores the index sums K_j in offset binary with b_out =
// b + ceil(log2 N) bits (scheme (b) grants the sum that many more bits), or rounds the average K_j / N back to the
// b-bit grid with rule (1) of Section 2.2 and the server's own rounding stream (scheme (c), Eq. 4).  The 8 * b_out
// output bits of a thread are b_out whole bytes, staged through shared memory and written out as words.
// One worker's 8 * BITS bits of coordinate group g (fixed widths), and their addition into packed integer lanes:
// 2-bit codes in byte lanes of four half words, 4-bit codes in byte lanes of two words (even and odd codes), 8-bit
// codes in half-word lanes of four words.
template <int BITS>
__device__ __forceinline__ uint2 load_codes(const uint32_t* __restrict__ w, int64_t g) {
  if constexpr (BITS == 8) return __ldcs(reinterpret_cast<const uint2*>(w + g * 2));
  else if constexpr (BITS == 4) return make_uint2(__ldcs(w + g), 0u);
  else return make_uint2((uint32_t)__ldcs(reinterpret_cast<const uint16_t*>(w) + g), 0u);
}
template <int BITS>
__device__ __forceinline__ void add_lanes(uint32_t* acc, uint2 c) {
  if constexpr (BITS == 8) {  // codes (0, 2), (1, 3), (4, 6), (5, 7)
    acc[0] += c.x & 0x00FF00FFu; acc[1] += (c.x >> 8) & 0x00FF00FFu;
    acc[2] += c.y & 0x00FF00FFu; acc[3] += (c.y >> 8) & 0x00FF00FFu;
  } else if constexpr (BITS == 4) {  // codes 0, 2, 4, 6 and 1, 3, 5, 7, one per byte
    acc[0] += c.x & 0x0F0F0F0Fu; acc[1] += (c.x >> 4) & 0x0F0F0F0Fu;
  } else {  // codes 0, 4 | 1, 5 | 2, 6 | 3, 7 in the low and high byte of a half word
    acc[0] += c.x & 0x0303u; acc[1] += (c.x >> 2) & 0x0303u; acc[2] += (c.x >> 4) & 0x0303u; acc[3] += (c.x >> 6) & 0x0303u;
  }
}
template <int BITS>
__device__ __forceinline__ void spread_lanes(const uint32_t* acc, int* K) {
  if constexpr (BITS == 8) {
    K[0] += (int)(acc[0] & 0xFFFFu); K[2] += (int)(acc[0] >> 16); K[1] += (int)(acc[1] & 0xFFFFu); K[3] += (int)(acc[1] >> 16);
    K[4] += (int)(acc[2] & 0xFFFFu); K[6] += (int)(acc[2] >> 16); K[5] += (int)(acc[3] & 0xFFFFu); K[7] += (int)(acc[3] >> 16);
  } else if constexpr (BITS == 4) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      K[2 * q] += (int)((acc[0] >> (8 * q)) & 0xFFu);
      K[2 * q + 1] += (int)((acc[1] >> (8 * q)) & 0xFFu);
    }
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      K[q] += (int)(acc[q] & 0xFFu);
      K[q + 4] += (int)((acc[q] >> 8) & 0xFFu);
    }
  }
}

// Sums of the codes of the N streams at the 8 coordinates of group gA and of group gB (K += sum_i code_i).  Eight
// workers per round, and the words of both groups are requested before the first is used: sixteen loads in flight
// per thread.  Eight codes of at most 8 bits cannot overflow a lane.
template <int BITS>
__device__ __forceinline__ void sum_codes8x2(const uint32_t* __restrict__ w, int64_t stride_words, int N, int64_t gA,
                                             int64_t gB, bool doA, bool doB, int b, int64_t pad_words, int* KA, int* KB) {
  if constexpr (BITS != 0) {
    for (int i0 = 0; i0 < N; i0 += 8) {
      uint2 ca[8], cb[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const bool live = i0 + q < N;
        const uint32_t* wi = w + (int64_t)(i0 + q) * stride_words;
        ca[q] = (live && doA) ? load_codes<BITS>(wi, gA) : make_uint2(0u, 0u);
        cb[q] = (live && doB) ? load_codes<BITS>(wi, gB) : make_uint2(0u, 0u);
      }
      uint32_t aa[4] = {0, 0, 0, 0}, ab[4] = {0, 0, 0, 0};
#pragma unroll
      for (int q = 0; q < 8; ++q) { add_lanes<BITS>(aa, ca[q]); add_lanes<BITS>(ab, cb[q]); }
      spread_lanes<BITS>(aa, KA);
      spread_lanes<BITS>(ab, KB);
    }
  } else {
#pragma unroll 2
    for (int i = 0; i < N; ++i) {
      uint64_t lo, hi;
      if (doA) {
        load_chunk<0>(w + (int64_t)i * stride_words, gA, b, pad_words, lo, hi);
#pragma unroll
        for (int e = 0; e < 8; ++e) KA[e] += (int)extract(lo, hi, e * b, b);
      }
      if (doB) {
        load_chunk<0>(w + (int64_t)i * stride_words, gB, b, pad_words, lo, hi);
#pragma unroll
        for (int e = 0; e < 8; ++e) KB[e] += (int)extract(lo, hi, e * b, b);
      }
    }
  }
}

// The server of schemes (b) and (c) (Section 3.2).  A thread owns 8 consecutive coordinates per sweep and takes two
// sweeps at a time: it adds the codes of the N streams as integers, then either stores the index sums K_j in offset
// binary with b_out = b + ceil(log2 N) bits (scheme (b) grants the sum that many more bits), or rounds the average
// K_j / N back to the b-bit grid with rule (1) of Section 2.2 and the server's own rounding stream (scheme (c),
// Eq. 4).  The 8 * b_out output bits of a thread are b_out whole bytes: one or two words stored directly when b_out
// is 4 or 8, else staged through shared memory and written out as words.
template <int BITS>  // input width: 2, 4, 8 fixed; 0: b in 2..16 from the arguments
__global__ void __launch_bounds__(AT, 4) server_reduce_kernel(ServerArgs a) {
  const int tile = blockIdx.x;
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  const SegInfo s = a.segs[seg];
  const SegInfo so = a.segs_out[seg];
  const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
  const int tid = threadIdx.x;
  const int b = (BITS == 0) ? a.b : BITS;
  const int bo = a.b_out;
  const int bias_in = a.N << (b - 1);  // sum of the offsets of N codes
  const float fN = (float)a.N;
  const bool pow2 = (a.N & (a.N - 1)) == 0;
  const float invN = __fdiv_rn(1.0f, fN);  // exact when N is a power of two: then K * invN is the division K / N
  const bool direct = (bo == 4 || bo == 8);
  __shared__ __align__(16) uint8_t stage[AT * 16];
  const uint32_t* w = a.codes + s.word_off;
  uint32_t* out = a.out + so.word_off;

  // the packed output bits of one group from its sums
  auto encode = [&](const int* K, int64_t j, int nvalid, uint64_t& olo, uint64_t& ohi) {
    olo = 0; ohi = 0;
    if (nvalid <= 0) return;
    U4 r = U4{0, 0, 0, 0};
    if (a.requantize) r = stream_block(a.seed, TAG_REQUANT, 0u, a.k, s.block_base + (uint32_t)(j >> 3));
    if constexpr (BITS != 0) {
      if (a.requantize) {
        uint32_t w0 = 0, w1 = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float avg = pow2 ? mul_rn((float)K[e], invN) : __fdiv_rn((float)K[e], fN);
          const uint32_t code = quantize_code<BITS ? BITS : 2>(avg, 1.0f, lane16(r, e));
          if (e * BITS < 32) w0 |= code << ((e * BITS) & 31);
          else w1 |= code << ((e * BITS) & 31);
        }
        olo = (uint64_t)w0 | ((uint64_t)w1 << 32);
        if (nvalid < 8) olo &= (1ull << (nvalid * BITS)) - 1ull;
        return;
      }
    }
    if (!a.requantize && bo <= 8) {
      // eight sums of at most 8 bits: one 64-bit word, built from the last code down with one uniform shift each
      const uint32_t bias_out = 1u << (bo - 1);
      uint64_t wv = 0;
#pragma unroll
      for (int e = 7; e >= 0; --e) wv = (wv << bo) | (uint64_t)((e < nvalid) ? (uint32_t)K[e] + bias_out : 0u);
      olo = wv;
      return;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (e < nvalid) {
        uint32_t code;
        if (a.requantize) {
          const float avg = pow2 ? mul_rn((float)K[e], invN) : __fdiv_rn((float)K[e], fN);
          code = quantize_code_rt(avg, 1.0f, lane16(r, e), b);
        } else {
          code = (uint32_t)(K[e] + (1 << (bo - 1)));
        }
        const int pos = e * bo;
        if (pos < 64) {
          olo |= (uint64_t)code << pos;
          if (pos + bo > 64) ohi |= (uint64_t)code >> (64 - pos);
        } else {
          ohi |= (uint64_t)code << (pos - 64);
        }
      }
    }
  };
  bool staged_before = false;
  auto emit = [&](int64_t sweep0, int64_t j, uint64_t olo, uint64_t ohi) {  // called by all threads of the block together
    if (direct) {  // uniform for the launch
      const int64_t g = j >> 3;
      if (bo == 4) {
        if (g < so.pad_words) out[g] = (uint32_t)olo;
      } else {
        if (2 * g < so.pad_words) *reinterpret_cast<uint2*>(out + 2 * g) = make_uint2((uint32_t)olo, (uint32_t)(olo >> 32));
      }
    } else {
      if (staged_before) __syncthreads();
      staged_before = true;
      if (bo <= 8) {
        const uint32_t l32 = (uint32_t)olo, h32 = (uint32_t)(olo >> 32);
        uint8_t* dst = stage + tid * bo;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (i < bo) dst[i] = (uint8_t)(((i < 4) ? l32 : h32) >> (8 * (i & 3)));
      } else {
        for (int i = 0; i < bo; ++i) stage[tid * bo + i] = (uint8_t)((i < 8) ? (olo >> (8 * i)) : (ohi >> (8 * (i - 8))));
      }
      __syncthreads();
      const int64_t w0 = (sweep0 >> 5) * bo;  // sweep0 is a multiple of 2048, so this is exact
      const uint32_t* stw = reinterpret_cast<const uint32_t*>(stage);
      for (int q = tid; q < (AGROUP / 32) * bo; q += AT)
        if (w0 + q < so.pad_words) out[w0 + q] = stw[q];
    }
  };

#pragma unroll 1
  for (int it = 0; it < AITER; it += 2) {
    const int64_t sweepA = tstart + (int64_t)it * AGROUP, sweepB = sweepA + AGROUP;
    if (sweepA >= s.len) break;  // uniform for the block
    const bool haveB = sweepB < s.len;  // uniform for the block
    const int64_t jA = sweepA + tid * 8, jB = sweepB + tid * 8;
    const int nvA = (jA < s.len) ? (int)min((int64_t)8, s.len - jA) : 0;
    const int nvB = (jB < s.len) ? (int)min((int64_t)8, s.len - jB) : 0;
    int KA[8], KB[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { KA[e] = -bias_in; KB[e] = -bias_in; }
    sum_codes8x2<BITS>(w, a.stride_words, a.N, jA >> 3, jB >> 3, nvA > 0, nvB > 0, b, s.pad_words, KA, KB);
    uint64_t olo, ohi;
    encode(KA, jA, nvA, olo, ohi);
    emit(sweepA, jA, olo, ohi);
    if (haveB) {
      encode(KB, jB, nvB, olo, ohi);
      emit(sweepB, jB, olo, ohi);
    }
  }
}

// The server for 4-bit codes of at most 16 workers (sums of at most 8 bits).  A thread owns 32 consecutive coordinates:
// per worker that is one 16-byte load, and its output -- 32 sums of BO bits, or 32 re-quantized 4-bit codes -- is BO (or
// 4) whole words, so nothing is staged or exchanged.  The codes are added in byte lanes (even and odd codes of a word
// apart), every load of the thread in flight at once; the sums are placed in the output words by multiply-adds with
// constant powers of two (the low part of the product is the shifted value, the high part its spill into the next word).
template <int BO, bool REQ>
__global__ void __launch_bounds__(AT, 4) server_reduce4_kernel(ServerArgs a) {
  constexpr int OW = REQ ? 4 : BO;  // output words per thread
  const int tile = blockIdx.x, tid = threadIdx.x;
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  const SegInfo s = a.segs[seg];
  const SegInfo so = a.segs_out[seg];
  const int64_t j = (int64_t)(tile - s.tile_first) * TILE + tid * 32;  // this thread's first coordinate (segment-local)
  if (j >= s.len) return;
  const int nv = (int)min((int64_t)32, s.len - j);
  const uint32_t* w = a.codes + s.word_off + (j >> 3);  // its four words of every stream: inside the padded stream
  uint32_t ev[4] = {0, 0, 0, 0}, od[4] = {0, 0, 0, 0};  // sums of the codes 8q + 2r in byte r of ev[q], of 8q + 2r + 1 in od[q]
#pragma unroll 1
  for (int i0 = 0; i0 < a.N; i0 += 8) {  // eight workers per round, their loads in flight together (uniform trip count)
    uint4 c[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      c[i] = (i0 + i < a.N) ? __ldcs(reinterpret_cast<const uint4*>(w + (int64_t)(i0 + i) * a.stride_words)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int i = 0; i < 8; ++i) {  // 16 codes of at most 15: a byte lane cannot overflow
      const uint32_t x[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        ev[q] += x[q] & 0x0F0F0F0Fu;
        od[q] += (x[q] >> 4) & 0x0F0F0F0Fu;
      }
    }
  }
  uint32_t out[OW];
#pragma unroll
  for (int i = 0; i < OW; ++i) out[i] = 0u;
  if constexpr (REQ) {
    // scheme (c), Eq. 4: the average K / N in grid units, rounded by rule (1) with the server's own rounding stream
    const float fN = (float)a.N;
    const bool pow2 = (a.N & (a.N - 1)) == 0;
    const float invN = __fdiv_rn(1.0f, fN);
    const float magic = 8388608.f + (float)(a.N << 3);  // 2^23 + the offsets of N codes: as_float(2^23 | sum) - magic = K exactly
    float dummy = 0.f;
    auto requantize = [&](auto average) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t sum = (((e & 1) ? od[q] : ev[q]) >> (8 * (e >> 1))) & 0xFFu;
          v[e] = average(__fsub_rn(__uint_as_float(0x4B000000u | sum), magic));
        }
        const U4 r = stream_block(a.seed, TAG_REQUANT, 0u, a.k, s.block_base + (uint32_t)(j >> 3) + (uint32_t)q);
        out[q] = (uint32_t)quantize_group8<4, false>(v, 1.0f, r, 0.f, 0.f, dummy);
      }
    };
    if (pow2) {
      // N a power of two: K / N is exact in fp32 and Z = ceil(s * 2^17) of the rounding rule (lpc_device.cuh) is the
      // integer K * (2^17 / N); the average of N hull points lies in the hull, so nothing is clamped.  The code
      // floor((Z + 131070 + 2^17 * 8 - 2 r16) / 2^17) then takes integer operations only:
      //   (sum * c1 + c0 - 2 r16) >> 17,   c1 = 2^17 / N,   c0 = 131070 + 2^20 - 8 N c1.
      const uint32_t c1 = 131072u / (uint32_t)a.N, c0 = 131070u + (1u << 20) - 8u * (uint32_t)a.N * c1;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const U4 r = stream_block(a.seed, TAG_REQUANT, 0u, a.k, s.block_base + (uint32_t)(j >> 3) + (uint32_t)q);
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t sum = (((e & 1) ? od[q] : ev[q]) >> (8 * (e >> 1))) & 0xFFu;
          word += ((sum * c1 + c0 - 2u * lane16(r, e)) >> 17) << (4 * e);
        }
        out[q] = word;
      }
    } else {
      requantize([&](float K) { return __fdiv_rn(K, fN); });
    }
  } else {
    // scheme (b): the index sums in offset binary; sum of codes - 8 N + 2^(BO-1) >= 0 since 2^(BO-1) >= 8 N
    const uint32_t shift = (1u << (BO - 1)) - ((uint32_t)a.N << 3);
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const int q = e >> 3, r = (e & 7) >> 1;
      const uint32_t val = ((((e & 1) ? od[q] : ev[q]) >> (8 * r)) & 0xFFu) + shift;
      const int pos = e * BO, wi = pos >> 5, sh = pos & 31;
      out[wi] += val << sh;
      if (sh + BO > 32) out[wi + 1] += val >> (32 - sh);
    }
  }
  if (nv < 32) {  // nothing but zeros past the end of the segment
    const int bits = nv * (REQ ? 4 : BO);
#pragma unroll
    for (int i = 0; i < OW; ++i) {
      const int left = bits - 32 * i;
      if (left <= 0) out[i] = 0u;
      else if (left < 32) out[i] &= (1u << left) - 1u;
    }
  }
  uint32_t* o = a.out + so.word_off + (j >> 5) * OW;
#pragma unroll
  for (int i = 0; i < OW; ++i)
    if ((j >> 5) * OW + i < so.pad_words) o[i] = out[i];
}

constexpr int HRUN = 32;  // tiles per CTA: the counts reach the message's histogram (a few hot addresses) once per run and segment

// Histogram of a message's code values, the input of the entropy-coding count (Section 5.1: the experiments pass the
// codes through Huffman's code).
//
// Widths 1, 2 and 4 are counted without looking at single codes.  A thread takes 16 bytes of the stream at a time and
// keeps one counter per code value in registers:
//   b = 4: the four words hold 32 codes.  A 4 x 4 bit transpose across the words (two rounds of masked swaps) gives
//          R_k, whose bit 4 i + r is bit k of code i of word r; the codes equal to v are the bits of
//          AND_k (v_k ? R_k : ~R_k), and their number is one population count -- about 2.3 instructions per code
//          instead of an extraction, an address and a shared-memory read-modify-write for each;
//   b = 2: two bit planes per word, four masks and population counts per 16 codes;
//   b = 1: the population count of the word.
// A CTA takes a run of tiles of one worker; the thread counters are added up by warp reductions when the run or
// the tensor segment ends, and one 64-bit atomic per value, run and segment reaches the message's histogram.  Codes
// of a ragged end (less than 16 bytes of valid codes) are counted one by one.
template <int BITS>
__device__ __forceinline__ void count_unit(uint4 q, uint32_t* cnt) {
  if constexpr (BITS == 4) {
    uint32_t a = q.x, b = q.y, c = q.z, d = q.w, t;
    t = ((a >> 1) ^ b) & 0x55555555u; b ^= t; a ^= t << 1;
    t = ((c >> 1) ^ d) & 0x55555555u; d ^= t; c ^= t << 1;
    t = ((a >> 2) ^ c) & 0x33333333u; c ^= t; a ^= t << 2;
    t = ((b >> 2) ^ d) & 0x33333333u; d ^= t; b ^= t << 2;
#pragma unroll
    for (int v = 0; v < 8; ++v) {  // the low three bits of the value, then both settings of the fourth
      const uint32_t m = ((v & 1) ? a : ~a) & ((v & 2) ? b : ~b) & ((v & 4) ? c : ~c);
      cnt[v] += __popc(m & ~d);
      cnt[v + 8] += __popc(m & d);
    }
  } else if constexpr (BITS == 2) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t lo = w[i] & 0x55555555u, hi = (w[i] >> 1) & 0x55555555u;
      cnt[0] += __popc(~(lo | hi) & 0x55555555u);
      cnt[1] += __popc(lo & ~hi);
      cnt[2] += __popc(hi & ~lo);
      cnt[3] += __popc(lo & hi);
    }
  } else {
    const uint32_t ones = __popc(q.x) + __popc(q.y) + __popc(q.z) + __popc(q.w);
    cnt[1] += ones;
    cnt[0] += 128u - ones;
  }
}

template <int BITS>  // 1, 2, 4
__global__ void __launch_bounds__(AT) code_histogram_swar_kernel(HistArgs a) {
  constexpr int BINS = 1 << BITS, CPU = 128 / BITS;  // codes per 16-byte unit
  const int worker = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
  const int tile0 = blockIdx.x * HRUN, tile1 = min(tile0 + HRUN, a.ntiles);
  __shared__ unsigned int total[BINS];
  if (tid < BINS) total[tid] = 0u;
  __syncthreads();
  uint32_t cnt[BINS];
#pragma unroll
  for (int v = 0; v < BINS; ++v) cnt[v] = 0u;
  int tile = tile0;
  while (tile < tile1) {  // one pass per tensor segment that the run touches
    const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
    const SegInfo s = a.segs[seg];
    const int tend = min(tile1, s.tile_first + s.tile_count);  // the run's tiles of this segment: [tile, tend)
    const int64_t j0 = (int64_t)(tile - s.tile_first) * TILE;
    const int64_t n = min(s.len, (int64_t)(tend - s.tile_first) * TILE) - j0;  // codes to count
    const uint32_t* w = a.codes + (int64_t)worker * a.stride_words + s.word_off + (j0 >> 5) * BITS;  // 16-byte aligned
    const int64_t units = n / CPU;
    const uint4* wu = reinterpret_cast<const uint4*>(w);
    int64_t u = tid;
    for (; u + 3 * AT < units; u += 4 * AT) {  // four loads in flight
      const uint4 q0 = __ldcs(wu + u), q1 = __ldcs(wu + u + AT), q2 = __ldcs(wu + u + 2 * AT), q3 = __ldcs(wu + u + 3 * AT);
      count_unit<BITS>(q0, cnt); count_unit<BITS>(q1, cnt); count_unit<BITS>(q2, cnt); count_unit<BITS>(q3, cnt);
    }
    for (; u < units; u += AT) count_unit<BITS>(__ldcs(wu + u), cnt);
    for (int64_t j = units * CPU + tid; j < n; j += AT) {  // the ragged end, code by code
      const uint32_t code = (w[(j * BITS) >> 5] >> ((j * BITS) & 31)) & (uint32_t)(BINS - 1);
      atomicAdd(&total[code], 1u);
    }
    // the segment's counts of this run go to its histogram
#pragma unroll
    for (int v = 0; v < BINS; ++v) {
      const uint32_t sum = __reduce_add_sync(0xFFFFFFFFu, cnt[v]);
      if (lane == 0 && sum) atomicAdd(&total[v], sum);
      cnt[v] = 0u;
    }
    __syncthreads();
    if (tid < BINS && total[tid]) {
      atomicAdd(&a.hist[((int64_t)worker * a.nseg + seg) * BINS + tid], (unsigned long long)total[tid]);
      total[tid] = 0u;
    }
    __syncthreads();
    tile = tend;
  }
}

// Widths without a bit-sliced count (8 bits, and the odd widths): every thread counts the 32 codes it reads in counters
// of its own in shared memory -- one byte per code value, four values to a 32-bit word, word[value / 4][thread] -- so
// that counting needs no atomic operation however skewed the codes are and a warp's accesses fall on 32 different banks.
// The block then adds the columns up with warp reductions and sends the tile's count of every value to the message's
// histogram with one atomic addition each.
template <int BITS>  // 1, 2, 4, 8: code width known at compile time; 0: b in 1..8 from the arguments
__global__ void __launch_bounds__(AT) code_histogram_kernel(HistArgs a) {
  const int worker = blockIdx.y;
  const int tile0 = blockIdx.x * HRUN, tile1 = min(tile0 + HRUN, a.ntiles);
  const int tid = threadIdx.x;
  const int b = BITS ? BITS : a.b, bins = 1 << b;
  const int rows = (bins + 3) / 4;  // words per thread and copy
  // Narrow codes keep NCH copies of the counters, one per coordinate position modulo NCH: the eight increments of a
  // group then form NCH independent chains of read-modify-writes instead of one (they may hit the same counter, so
  // the chain of one copy cannot be reordered)
  constexpr int NCH = (BITS >= 1 && BITS <= 4) ? 4 : 1;
  extern __shared__ __align__(16) uint32_t cw[];  // NCH x rows x AT words
  uint8_t* mine = reinterpret_cast<uint8_t*>(cw + tid);  // this thread's counter of value c in copy q: mine[((q * rows + c / 4) * AT) * 4 + c % 4]
  __shared__ unsigned int total[256];
  for (int c = tid; c < bins; c += AT) total[c] = 0u;
  int cur_seg = -1;
  auto flush = [&]() {  // the counts gathered for segment cur_seg go to its histogram (all threads call this)
    __syncthreads();
    if (cur_seg >= 0)
      for (int c = tid; c < bins; c += AT) {
        if (total[c]) atomicAdd(&a.hist[((int64_t)worker * a.nseg + cur_seg) * bins + c], (unsigned long long)total[c]);
        total[c] = 0u;
      }
    __syncthreads();
  };
#pragma unroll 1
  for (int tile = tile0; tile < tile1; ++tile) {
    const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
    if (seg != cur_seg) {
      flush();
      cur_seg = seg;
    }
    const SegInfo s = a.segs[seg];
    const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
    for (int i = tid; i < NCH * rows * AT; i += AT) cw[i] = 0u;  // a thread clears and uses its own column only
    const uint32_t* w = a.codes + (int64_t)worker * a.stride_words + s.word_off;
    if constexpr (BITS != 0) {
      // fixed widths: which thread counts which code does not matter, so a thread takes whole words of the tile's
      // stream, BITS of them, AT words apart (coalesced), all requested before the first is used
      constexpr int CPW = 32 / BITS;  // codes per word
      const int64_t nvalid_tile = min((int64_t)TILE, s.len - tstart);
      const uint32_t* wt = w + (tstart >> 5) * BITS;
      uint32_t cwords[BITS];
#pragma unroll
      for (int i = 0; i < BITS; ++i) {
        const int wi = i * AT + tid;
        cwords[i] = ((int64_t)wi * CPW < nvalid_tile) ? __ldcs(wt + wi) : 0u;
      }
#pragma unroll
      for (int i = 0; i < BITS; ++i) {
        const int wi = i * AT + tid;
        const int64_t left = nvalid_tile - (int64_t)wi * CPW;  // codes of this word that exist
        if (left >= CPW) {
#pragma unroll
          for (int e = 0; e < CPW; ++e) {
            const uint32_t code = (cwords[i] >> (e * BITS)) & (uint32_t)(bins - 1);
            mine[((((e % NCH) * rows + (code >> 2)) * (AT * 4))) | (code & 3u)] += 1;
          }
        } else {
          for (int e = 0; e < (int)left; ++e) {
            const uint32_t code = (cwords[i] >> (e * BITS)) & (uint32_t)(bins - 1);
            mine[((((e % NCH) * rows + (code >> 2)) * (AT * 4))) | (code & 3u)] += 1;
          }
        }
      }
    } else {
#pragma unroll 1
      for (int it = 0; it < AITER; ++it) {  // a thread sees at most AITER * 8 = 32 codes: a byte counter cannot overflow
        const int64_t j = tstart + (int64_t)it * AGROUP + tid * 8;
        if (j >= s.len) break;
        const int nvalid = (int)min((int64_t)8, s.len - j);
        uint64_t lo, hi;
        load_chunk<0>(w, j >> 3, b, s.pad_words, lo, hi);  // 8 * b <= 64 bits: all in lo
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (e < nvalid) {
            const uint32_t code = (uint32_t)(lo >> (e * b)) & (uint32_t)(bins - 1);
            mine[((code >> 2) * (AT * 4)) | (code & 3u)] += 1;
          }
        }
      }
    }
    // the tile's columns add up: a word's four byte counters (each <= 32) widen to two words of 16-bit lanes, a warp
    // adds them with one integer reduction each (32 lanes * 32 fits 16 bits), lane 0 adds the sums to the run's totals
    for (int r = 0; r < rows; ++r) {
      uint32_t v = cw[r * AT + tid];
#pragma unroll
      for (int q = 1; q < NCH; ++q) v += cw[(q * rows + r) * AT + tid];  // byte lanes: at most 32 in all, no carry
      const uint32_t even = __reduce_add_sync(0xFFFFFFFFu, v & 0x00FF00FFu);         // values 4r, 4r+2
      const uint32_t odd = __reduce_add_sync(0xFFFFFFFFu, (v >> 8) & 0x00FF00FFu);   // values 4r+1, 4r+3
      if ((tid & 31) == 0) {
        if (even & 0xFFFFu) atomicAdd(&total[4 * r], even & 0xFFFFu);
        if (even >> 16) atomicAdd(&total[4 * r + 2], even >> 16);
        if (odd & 0xFFFFu) atomicAdd(&total[4 * r + 1], odd & 0xFFFFu);
        if (odd >> 16) atomicAdd(&total[4 * r + 3], odd >> 16);
      }
    }
  }
  flush();
}

}  // namespace

cudaError_t launch_code_histogram(const HistArgs& a, cudaStream_t st) {
  if (a.ntiles <= 0 || a.N <= 0) return cudaSuccess;
  const size_t sh = (size_t)(a.b <= 4 && (a.b == 1 || a.b == 2 || a.b == 4) ? 4 : 1) * (size_t)(((1 << a.b) + 3) / 4) * AT * sizeof(uint32_t);
  const dim3 grid((unsigned)((a.ntiles + HRUN - 1) / HRUN), (unsigned)a.N);
  auto go = [&](auto kernel) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
    if (e != cudaSuccess) return e;
    kernel<<<grid, AT, sh, st>>>(a);
    return cudaGetLastError();
  };
  switch (a.b) {
    case 1: code_histogram_swar_kernel<1><<<grid, AT, 0, st>>>(a); return cudaGetLastError();
    case 2: code_histogram_swar_kernel<2><<<grid, AT, 0, st>>>(a); return cudaGetLastError();
    case 4: code_histogram_swar_kernel<4><<<grid, AT, 0, st>>>(a); return cudaGetLastError();
    case 8: return go(code_histogram_kernel<8>);
    default: return go(code_histogram_kernel<0>);
  }
}

cudaError_t launch_server_reduce(const ServerArgs& a, cudaStream_t st) {
  if (a.ntiles <= 0) return cudaSuccess;
  const dim3 grid((unsigned)a.ntiles), block(AT);
  if (a.b == 4 && a.N <= 16) {  // sums of at most 8 bits: whole words per thread
    if (a.requantize) { server_reduce4_kernel<4, true><<<grid, block, 0, st>>>(a); return cudaGetLastError(); }
    switch (a.b_out) {
      case 4: server_reduce4_kernel<4, false><<<grid, block, 0, st>>>(a); return cudaGetLastError();
      case 5: server_reduce4_kernel<5, false><<<grid, block, 0, st>>>(a); return cudaGetLastError();
      case 6: server_reduce4_kernel<6, false><<<grid, block, 0, st>>>(a); return cudaGetLastError();
      case 7: server_reduce4_kernel<7, false><<<grid, block, 0, st>>>(a); return cudaGetLastError();
      case 8: server_reduce4_kernel<8, false><<<grid, block, 0, st>>>(a); return cudaGetLastError();
      default: break;
    }
  }
  switch (a.b) {
    case 2: server_reduce_kernel<2><<<grid, block, 0, st>>>(a); break;
    case 4: server_reduce_kernel<4><<<grid, block, 0, st>>>(a); break;
    case 8: server_reduce_kernel<8><<<grid, block, 0, st>>>(a); break;
    default: server_reduce_kernel<0><<<grid, block, 0, st>>>(a); break;
  }
  return cudaGetLastError();
}

int aggregate_split(int ntiles, int sm_count) {
  const int wave = 4 * (sm_count > 0 ? sm_count : 148);  // resident CTAs of this kernel
  return (ntiles >= 2 * wave) ? 1 : (ntiles >= wave) ? 2 : AITER;
}

cudaError_t launch_unpack_average_prox(const AggArgs& a, cudaStream_t st) {
  if (a.ntiles <= 0) return cudaSuccess;
  if (!(a.split == 1 || a.split == 2 || a.split == AITER)) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)(a.ntiles * a.split)), block(AT);
  const size_t sh = (size_t)a.N * sizeof(float);
  switch (a.b) {
    case 1: unpack_average_prox_kernel<1><<<grid, block, sh, st>>>(a); break;
    case 2: unpack_average_prox_kernel<2><<<grid, block, sh, st>>>(a); break;
    case 3: unpack_average_prox_kernel<3><<<grid, block, sh, st>>>(a); break;
    case 4: unpack_average_prox_kernel<4><<<grid, block, sh, st>>>(a); break;
    case 8: unpack_average_prox_kernel<8><<<grid, block, sh, st>>>(a); break;
    case 32: unpack_average_prox_kernel<32><<<grid, block, sh, st>>>(a); break;
    default: unpack_average_prox_kernel<0><<<grid, block, sh, st>>>(a); break;
  }
  return cudaGetLastError();
}

}  // namespace lpc
