// Device-side building blocks shared by the kernels of the library: the counter-based random
// streams, the fixed-order fp32 reductions, the per-coordinate quantizer and small PTX wrappers.
//
// Arithmetic contract.  The packed codes are a deterministic function of the input floats, so every
// fp32 operation on the way to a code is an explicit round-to-nearest intrinsic (__fmul_rn, __fadd_rn,
// __fdiv_rn) that the compiler can neither contract into an FMA nor reorder.  The files are also
// compiled with -fmad=false.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "lpc_status.h"

namespace lpc {

// ---- stream tags ---------------------------------------------------------------------------------
constexpr uint32_t TAG_ROUND = 0;
constexpr uint32_t TAG_BATCH = 1;
constexpr uint32_t TAG_BATCH_J = 2;
constexpr uint32_t TAG_REQUANT = 4;  // the server's rounding variables under scheme (c) of Section 3.2

// Philox4x32-10 (Salmon et al., SC'11).  Ten rounds; each round multiplies counter words 0 and 2 by
// two fixed constants, xors the high halves with the other two words and the key, and the key
// advances by two Weyl increments between rounds.
struct U4 { uint32_t x, y, z, w; };

__device__ __forceinline__ U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                            uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // the two halves of each 32x32 product as separate multiplies: fewer instructions here than the 64-bit form
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return U4{c0, c1, c2, c3};
}

// Block `block` of stream (tag, worker, k): counter = (block, k_lo, worker | tag<<24, k_hi), key = seed.
__device__ __forceinline__ U4 stream_block(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k,
                                           uint32_t block) {
  return philox4x32_10(block, (uint32_t)k, (worker & 0xFFFFFFu) | (tag << 24), (uint32_t)(k >> 32),
                       (uint32_t)seed, (uint32_t)(seed >> 32));
}

// ---- fixed-order (balanced binary tree over the coordinate index) fp32 sums ------------------------
__device__ __forceinline__ float add_rn(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float mul_rn(float a, float b) { return __fmul_rn(a, b); }

__device__ __forceinline__ float tree8(const float* v) {
  return add_rn(add_rn(add_rn(v[0], v[1]), add_rn(v[2], v[3])), add_rn(add_rn(v[4], v[5]), add_rn(v[6], v[7])));
}
__device__ __forceinline__ float tree4(float a, float b, float c, float d) {
  return add_rn(add_rn(a, b), add_rn(c, d));
}

// All 32 lanes end with the tree sum of the 32 lane values (lane order = leaf order).
__device__ __forceinline__ float warp_tree_sum(float v) {
#pragma unroll
  for (int m = 1; m < 32; m <<= 1) v = add_rn(v, __shfl_xor_sync(0xFFFFFFFFu, v, m));
  return v;
}
__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) { return __reduce_max_sync(0xFFFFFFFFu, v); }

// Warp reduction of V values per lane by recursive halving.  At the stage with lane mask 1<<S a lane
// keeps one half of its values and receives the partner's partial sums for that half; lanes with the bit
// clear keep the lower half.  After log2(V) stages one value is left, and the remaining stages are plain
// butterflies.  Partner sums are added in lane order, which is the balanced tree over the 32 lanes.
template <int V, int S>
struct WarpHalving {
  static __device__ __forceinline__ void run(float* v, int lane) {
    if constexpr (S < 5) {
      if constexpr (V > 1) {
        const bool up = (lane >> S) & 1;
#pragma unroll
        for (int i = 0; i < V / 2; ++i) {
          const float send = up ? v[i] : v[i + V / 2];
          const float keep = up ? v[i + V / 2] : v[i];
          v[i] = add_rn(keep, __shfl_xor_sync(0xFFFFFFFFu, send, 1 << S));
        }
        WarpHalving<V / 2, S + 1>::run(v, lane);
      } else {
        v[0] = add_rn(v[0], __shfl_xor_sync(0xFFFFFFFFu, v[0], 1 << S));
        WarpHalving<1, S + 1>::run(v, lane);
      }
    }
  }
};

// Index q (0 <= q < 2^LOGV) of the value that WarpHalving leaves in a lane: its bits, most significant first,
// are the lane's low bits.  Lanes with (lane >> LOGV) != 0 hold copies.
template <int LOGV>
__device__ __forceinline__ int halving_index(int lane) {
  int q = 0;
#pragma unroll
  for (int s = 0; s < LOGV; ++s) q |= ((lane >> s) & 1) << (LOGV - 1 - s);
  return q;
}

// Tree sum of N floats (N a power of two) stored in order in memory, evaluated by one thread: the recursive definition,
// unrolled, so the operands stay in registers and independent additions overlap.
template <int N>
__device__ __forceinline__ float tree_sum_n(const float* v) {
  if constexpr (N == 1) return v[0];
  else return add_rn(tree_sum_n<N / 2>(v), tree_sum_n<N / 2>(v + N / 2));
}
// The same for a count known only at run time (a power of two, <= 32: cross-warp and cross-CTA partial sums).
__device__ __forceinline__ float smem_tree_sum(const float* v, int count) {
  switch (count) {
    case 1: return v[0];
    case 2: return tree_sum_n<2>(v);
    case 4: return tree_sum_n<4>(v);
    case 8: return tree_sum_n<8>(v);
    case 16: return tree_sum_n<16>(v);
    default: return tree_sum_n<32>(v);
  }
}

// ---- scale (Eq. 2) -----------------------------------------------------------------------------------
struct Scale {
  float delta;   // transmitted float: codebook spacing (b=1: T; b=32: 1)
  float rdelta;  // 1/delta (0 when degenerate)
  float T;       // clip threshold
  float lower;   // lower end of the hull: -(T+delta)  (b=1: -T)
  uint32_t flags;  // bit0 degenerate (send zeros), bit1 non-finite input
};

constexpr int CLIP_NONE = 0, CLIP_LAMBDA = 1, CLIP_STD = 2;

// max_bits = max over coordinates of the bit pattern of |u| (monotone in |u|; NaN/Inf >= 0x7F800000).
__device__ __forceinline__ Scale make_scale(uint32_t max_bits, float S1, float S2, int64_t len, int b,
                                            int clip_mode, float clip_value) {
  Scale sc;
  if (max_bits >= 0x7F800000u) {
    sc.delta = __int_as_float(0x7FC00000);
    sc.rdelta = 0.f; sc.T = 0.f; sc.lower = 0.f; sc.flags = 3u;
    return sc;
  }
  const float M = __uint_as_float(max_bits);
  float T = M;
  if (clip_mode == CLIP_LAMBDA) {
    T = mul_rn(clip_value, M);
  } else if (clip_mode == CLIP_STD) {
    double mean, ex2;
    if (len > 0 && (len & (len - 1)) == 0) {
      // a power-of-two length: multiplying by 2^-log2(len) is the same exact operation as the division
      const double inv = __longlong_as_double((long long)(1023 - (63 - __clzll(len))) << 52);
      mean = __dmul_rn((double)S1, inv);
      ex2 = __dmul_rn((double)S2, inv);
    } else {
      mean = __ddiv_rn((double)S1, (double)len);
      ex2 = __ddiv_rn((double)S2, (double)len);
    }
    double var = __dsub_rn(ex2, __dmul_rn(mean, mean));
    if (var < 0.0) var = 0.0;
    double t = __dmul_rn((double)clip_value, __dsqrt_rn(var));
    if (t > (double)M) t = (double)M;
    T = __double2float_rn(t);
  }
  sc.T = T;
  if (b == 32) {
    sc.delta = 1.f; sc.rdelta = 1.f; sc.lower = -T; sc.flags = 0u;
    return sc;
  }
  const float Lv = (float)((1 << (b - 1)) - 1);
  const float delta = (b == 1) ? T : __fdiv_rn(T, Lv);
  const float rdelta = __fdiv_rn(1.0f, delta);
  if (M == 0.f || T == 0.f || delta == 0.f || isinf(rdelta) || isnan(rdelta)) {
    sc.delta = 0.f; sc.rdelta = 0.f; sc.lower = 0.f; sc.flags = 1u;
    return sc;
  }
  sc.delta = delta;
  sc.rdelta = rdelta;
  sc.lower = (b == 1) ? -T : -add_rn(T, delta);
  sc.flags = 0u;
  return sc;
}

// ---- quantizer of Section 2.2 for one coordinate -----------------------------------------------------
// Returns the stored code c = k + 2^(b-1) (b=1: the bit).  r16 is the coordinate's 16-bit random lane.
// s = u/delta (fp32) is clamped to the hull first (rule 2), then rounded down or up with probability
// frac(s) = s - floor(s), taken exactly (rule 1):   up  <=>  r16 + 0.5 < frac(s) * 65536.
//
// The decision is evaluated in fixed point, exactly and with few instructions (the quantize pass is bound
// by instruction issue, and there by the integer/logic pipe).  With Z = ceil(s * 2^17), which is exact
// (a power-of-two scaling and one directed rounding),
//   A := ceil(s * 65536 - 1/2) = floor(Z / 2),
//   r16 + 1/2 < frac(s) * 65536   <=>   r16 < A - 65536 * floor(s)          (r16 is an integer),
//   floor(s) + [r16 < A - 65536 floor(s)] = floor((A + 65535 - r16) / 65536)  (0 <= r16 <= 65535)
//                                         = floor((Z + 131070 - 2 r16) / 2^17),
// and the floor is a right shift.
//
// b <= 4: Z is formed in the mantissa of a float instead of by a conversion.  One fused multiply-add with
// round-up, t = RU(s * 2^17 + K), has an exact product and a single directed rounding; K is an integer
// that keeps t inside the binade [2^23, 2^24) where floats are the integers, so t = K + Z and the bit
// pattern of t is bits(K) + Z.  K also carries the constants 131070 and 2^17 * 2^(b-1), and bits(1.5 * 2^23)
// = 0x4B400000 = 0x25A0 * 2^17, hence
//   (bits(t) - 2 r16) >> 17  =  0x25A0 + code,        code = floor(s) + up + 2^(b-1).
// quantize_raw returns that biased value; QRAW_BIAS is removed once per packed word.
constexpr uint32_t QRAW_BIAS = 0x25A0u;

template <int B_>
__device__ __forceinline__ uint32_t quantize_raw(float u, float rdelta, uint32_t r16) {
  static_assert(B_ >= 1 && B_ <= 4, "the mantissa form covers b <= 4");
  float s = mul_rn(u, rdelta);
  if constexpr (B_ == 1) {
    // two code points: position between them ((s + 1) / 2) * 65536 = (s + 1) * 32768, s + 1 rounded to fp32
    s = add_rn(fminf(fmaxf(s, -1.f), 1.f), 1.f);
    const float t = __fmaf_ru(s, 65536.f, 12582912.f + 131070.f);
    return (__float_as_uint(t) - 2u * r16) >> 17;
  } else {
    constexpr float lo = -(float)(1 << (B_ - 1));
    constexpr float hi = (float)((1 << (B_ - 1)) - 1);
    constexpr float K = 12582912.f + 131070.f + (float)(131072 << (B_ - 1));
    s = fminf(fmaxf(s, lo), hi);  // projection onto the hull (rule 2)
    const float t = __fmaf_ru(s, 131072.f, K);
    return (__float_as_uint(t) - 2u * r16) >> 17;
  }
}

template <int B_>
__device__ __forceinline__ uint32_t quantize_code(float u, float rdelta, uint32_t r16) {
  static_assert(B_ >= 1 && B_ <= 8, "32-bit fixed point covers b <= 8");
  if constexpr (B_ <= 4) {
    return quantize_raw<B_>(u, rdelta, r16) - QRAW_BIAS;
  } else {
    constexpr float lo = -(float)(1 << (B_ - 1));
    constexpr float hi = (float)((1 << (B_ - 1)) - 1);
    float s = mul_rn(u, rdelta);
    s = fminf(fmaxf(s, lo), hi);
    const int Z = __float2int_ru(mul_rn(s, 131072.f));
    return (uint32_t)((Z + (131070 + (131072 << (B_ - 1))) - 2 * (int)r16) >> 17);
  }
}

// Any b in 1..16 (64-bit fixed point).
__device__ __forceinline__ uint32_t quantize_code_rt(float u, float rdelta, uint32_t r16, int b) {
  if (b == 1) return quantize_code<1>(u, rdelta, r16);
  const float lo = -(float)(1 << (b - 1));
  const float hi = (float)((1 << (b - 1)) - 1);
  float s = mul_rn(u, rdelta);
  s = fminf(fmaxf(s, lo), hi);
  const long long A = __float2ll_ru(mul_rn(s, 131072.f)) >> 1;
  return (uint32_t)((A + (65535ll + (65536ll << (b - 1))) - (long long)r16) >> 16);
}

// Exact float value of the signed codebook index of a stored code (code < 2^16).
__device__ __forceinline__ float index_as_float(uint32_t code, int b) {
  // 0x4B000000 is 2^23: or-ing a small integer into its mantissa and subtracting 2^23 converts exactly.
  const float biased = __uint_as_float(0x4B000000u | code);
  if (b == 1) return code ? 1.0f : -1.0f;
  return __fsub_rn(biased, 8388608.f + (float)(1 << (b - 1)));
}

// The signed codebook indices of the 8 codes of one coordinate group (8 * BITS payload bits in `lo`), as exact
// floats, for the fixed widths.  The codes are moved into the mantissa of 2^23 by byte permutes (one integer
// instruction per code after a few shared masks), then one exact subtraction removes 2^23 and the offset.
template <int BITS>
__device__ __forceinline__ void decode8(uint64_t lo, float* k) {
  static_assert(BITS == 1 || BITS == 2 || BITS == 3 || BITS == 4 || BITS == 8, "fixed widths only");
  constexpr uint32_t MAGIC = 0x4B000000u;  // 2^23
  if constexpr (BITS == 3) {  // the paper's three-level setting: 3-bit fields do not line up with bytes, one shift and mask each
    const uint32_t w = (uint32_t)lo;
#pragma unroll
    for (int e = 0; e < 8; ++e) k[e] = __fsub_rn(__uint_as_float(MAGIC | ((w >> (3 * e)) & 7u)), 8388608.f + 4.f);
  } else if constexpr (BITS == 1) {
#pragma unroll
    for (int e = 0; e < 8; ++e) k[e] = ((uint32_t)lo >> e) & 1u ? 1.0f : -1.0f;
  } else {
    constexpr float C = 8388608.f + (float)(1 << (BITS - 1));
    if constexpr (BITS == 8) {
      const uint32_t w0 = (uint32_t)lo, w1 = (uint32_t)(lo >> 32);
#pragma unroll
      for (int e = 0; e < 8; ++e)
        k[e] = __fsub_rn(__uint_as_float(__byte_perm(e < 4 ? w0 : w1, MAGIC, 0x7440u + (e & 3))), C);
    } else if constexpr (BITS == 4) {
      const uint32_t w = (uint32_t)lo;
      const uint32_t ev = w & 0x0F0F0F0Fu, od = (w >> 4) & 0x0F0F0F0Fu;
#pragma unroll
      for (int e = 0; e < 8; ++e)
        k[e] = __fsub_rn(__uint_as_float(__byte_perm((e & 1) ? od : ev, MAGIC, 0x7440u + (e >> 1))), C);
    } else {  // 2 bits: code e sits in byte e/4 of (w >> 2 (e%4)) & 0x0303
      const uint32_t w = (uint32_t)lo;
      uint32_t x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) x[j] = (w >> (2 * j)) & 0x0303u;
#pragma unroll
      for (int e = 0; e < 8; ++e)
        k[e] = __fsub_rn(__uint_as_float(__byte_perm(x[e & 3], MAGIC, 0x7440u + (e >> 2))), C);
    }
  }
}

// acc + delta * k for a signed codebook index k of a BITS-wide code.  For one- and two-bit codes k is -2, -1, 0 or 1:
// the product is exact (as long as 2 delta is finite), so one fused multiply-add rounds exactly like the separate
// multiply and add of wider codes.
template <int BITS>
__device__ __forceinline__ float add_scaled_index(float acc, float delta, float k) {
  if constexpr (BITS == 1 || BITS == 2) return __fmaf_rn(delta, k, acc);
  else return add_rn(acc, mul_rn(delta, k));
}

__device__ __forceinline__ float soft_threshold(float w, float kappa) {
  const float a = fmaxf(__fsub_rn(fabsf(w), kappa), 0.f);
  return copysignf(a, w);
}

// The eight 16-bit lanes of a Philox block: lane e of coordinate group = bits of word e/2, low half first.
__device__ __forceinline__ uint32_t lane16(const U4& r, int e) {
  const uint32_t w = (e < 2) ? r.x : (e < 4) ? r.y : (e < 6) ? r.z : r.w;
  return (e & 1) ? (w >> 16) : (w & 0xFFFFu);
}

// One more coordinate outside the hull [lower, T]: two compares and a predicated float add, which keeps the
// count off the integer pipe (exact: a thread counts far fewer than 2^24 coordinates).
__device__ __forceinline__ void count_outside(float& cnt, float u, float T, float lower) {
  asm("{\n\t.reg .pred p;\n\t"
      "setp.gt.f32 p, %1, %2;\n\t"
      "setp.lt.or.f32 p, %1, %3, p;\n\t"
      "@p add.rn.f32 %0, %0, 0f3F800000;\n\t}"
      : "+f"(cnt)
      : "f"(u), "f"(T), "f"(lower));
}

// The 8 * BITS packed bits of one coordinate group (code e in bits [e BITS, (e+1) BITS)) from its eight values
// and its Philox block; `cnt` grows by the number of values outside the hull when COUNT is set.
template <int BITS, bool COUNT>
__device__ __forceinline__ uint64_t quantize_group8(const float* v, float rdelta, const U4& r, float T, float lower,
                                                    float& cnt) {
  static_assert(BITS == 1 || BITS == 2 || BITS == 3 || BITS == 4 || BITS == 8, "fixed widths only");
  uint32_t w0 = 0, w1 = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    if (COUNT) count_outside(cnt, v[e], T, lower);
    uint32_t c;
    if constexpr (BITS <= 4) c = quantize_raw<BITS>(v[e], rdelta, lane16(r, e));  // biased by QRAW_BIAS
    else c = quantize_code<BITS>(v[e], rdelta, lane16(r, e));
    // multiply-add form: the shift rides on the multiplier pipe, and biased values may carry into higher fields
    if (e * BITS < 32) w0 += c * (1u << ((e * BITS) & 31));
    else w1 += c * (1u << ((e * BITS) & 31));
  }
  if constexpr (BITS <= 4) {
    uint32_t bias = 0;  // sum of the biases at the eight field positions, modulo 2^32
#pragma unroll
    for (int e = 0; e < 8; ++e) bias += QRAW_BIAS << (e * BITS);
    w0 -= bias;
  }
  return (uint64_t)w0 | ((uint64_t)w1 << 32);
}

// ---- mbarrier / bulk-copy (TMA) wrappers ---------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Non-blocking look at a phase: true when the phase with this parity has completed.
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false when the phase did not complete within about two seconds.  One try suspends the
// thread for at most LPC_WAIT_HINT_NS nanoseconds before it looks again: with the system's default limit a waiter
// noticed a completed phase more than a microsecond late.
#ifndef LPC_WAIT_HINT_NS
#define LPC_WAIT_HINT_NS 100u
#endif
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint64_t limit_ns = 2000000000ull) {
  const uint32_t addr = smem_u32(bar);
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity), "r"(LPC_WAIT_HINT_NS)
        : "memory");
    if (ok) return true;
    if ((it & 255u) == 255u) {
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}
// Bounded spin on data that another CTA writes (tagged words): call once per unsuccessful look, `it` counting the looks
// and t0 starting at 0.  Returns true when the caller must stop looking: another thread raised `abort_flag`, or no
// progress for limit_ns, in which case this thread records DEV_TIMEOUT in `dev_status` and raises the flag itself, so
// that every other spin of the grid ends at its next look.
__device__ __forceinline__ bool spin_expired(uint32_t it, uint64_t& t0, unsigned int* abort_flag, unsigned int* dev_status,
                                             uint64_t limit_ns = 2000000000ull) {
  if ((it & 63u) != 63u) return false;
  unsigned int raised;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(raised) : "l"(abort_flag) : "memory");
  if (raised != 0u) return true;
  const uint64_t now = global_ns();
  if (t0 == 0) {
    t0 = now;
    return false;
  }
  if (now - t0 <= limit_ns) return false;
  atomicOr(dev_status, DEV_TIMEOUT);
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(abort_flag), "r"(1u) : "memory");
  return true;
}
// Same bounded wait with acquire semantics at cluster scope: for phases completed by stores of other CTAs of the
// cluster (st_async_cluster below).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, uint64_t limit_ns = 2000000000ull) {
  const uint32_t addr = smem_u32(bar);
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity), "r"(LPC_WAIT_HINT_NS)
        : "memory");
    if (ok) return true;
    if ((it & 255u) == 255u) {
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}
// A 32-bit store into the shared memory of CTA `cta` of the cluster, at the address `slot` has in this CTA, that
// counts 4 bytes on that CTA's mbarrier `bar` (same offset there) when it lands: data and signal in one message.
__device__ __forceinline__ void st_async_cluster(const void* slot, const uint64_t* bar, uint32_t cta, uint32_t value) {
  uint32_t rslot, rbar;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rslot) : "r"(smem_u32(slot)), "r"(cta));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_u32(bar)), "r"(cta));
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(rslot), "r"(value),
               "r"(rbar)
               : "memory");
}
// One-dimensional bulk copy global -> this CTA's shared memory, completion counted on `bar`.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ int64_t next_pow2_i64(int64_t n) {
  int64_t p = 1;
  while (p < n) p <<= 1;
  return p;
}

// ---- losses ----------------------------------------------------------------------------------------------
constexpr int LOSS_LOGISTIC = 0, LOSS_LEAST_SQUARES = 1;

__device__ __forceinline__ float loss_deriv(int loss, float m, float y) {
  if (loss == LOSS_LEAST_SQUARES) return __fsub_rn(m, y);
  const double t = __dmul_rn((double)y, (double)m);
  return __double2float_rn(__ddiv_rn(-(double)y, __dadd_rn(1.0, exp(t))));
}
__device__ __forceinline__ double loss_value(int loss, float m, float y) {
  if (loss == LOSS_LEAST_SQUARES) {
    const double r = (double)m - (double)y;
    return 0.5 * r * r;
  }
  const double t = (double)y * (double)m;
  return (t > 0.0) ? log1p(exp(-t)) : (-t + log1p(exp(t)));
}

}  // namespace lpc
