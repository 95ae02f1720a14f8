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

template <int BITS>  // 1, 2, 4, 8: fixed width; 0: b in 1..16 from the arguments; 32: floats
__global__ void __launch_bounds__(AT) unpack_average_prox_kernel(AggArgs a) {
  const int tile = blockIdx.x;
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
  for (int it = 0; it < AITER; ++it) {
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
        for (int e = 0; e < 8; ++e) acc[e] = add_rn(acc[e], mul_rn(di, kf[e]));
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
        yv[e] = soft_threshold(__fsub_rn(xv[e], mul_rn(a.inv4L, vv[e])), ky);
        zv[e] = soft_threshold(__fsub_rn(zv[e], mul_rn(a.alpha, hv[e])), kz);
        sv[e] = add_rn(sv[e], yv[e]);
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
// Sums of the codes of the N streams at 8 coordinates (K[e] += sum_i code_ie).  The fixed widths add whole words of
// codes as small integer lanes (4-bit codes in 8-bit lanes, 8-bit codes in 16-bit lanes) and spread the lanes out
// before they could overflow.
template <int BITS>
__device__ __forceinline__ void sum_codes8(const uint32_t* __restrict__ w, int64_t stride_words, int N, int64_t g, int b,
                                           int64_t pad_words, int* K) {
  if constexpr (BITS == 4) {
    // sixteen workers per round: all their words are requested before the first is used; 16 * 15 fits a byte
    for (int i0 = 0; i0 < N; i0 += 16) {
      uint32_t c[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) c[q] = (i0 + q < N) ? __ldcs(w + (int64_t)(i0 + q) * stride_words + g) : 0u;
      uint32_t ev = 0, od = 0;  // codes 0, 2, 4, 6 and 1, 3, 5, 7, one per byte
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        ev += c[q] & 0x0F0F0F0Fu;
        od += (c[q] >> 4) & 0x0F0F0F0Fu;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        K[2 * q] += (int)((ev >> (8 * q)) & 0xFFu);
        K[2 * q + 1] += (int)((od >> (8 * q)) & 0xFFu);
      }
    }
  } else if constexpr (BITS == 8) {
    for (int i0 = 0; i0 < N; i0 += 8) {  // eight workers per round, loads first; 8 * 255 fits 16 bits
      uint2 c[8];
#pragma unroll
      for (int q = 0; q < 8; ++q)
        c[q] = (i0 + q < N) ? __ldcs(reinterpret_cast<const uint2*>(w + (int64_t)(i0 + q) * stride_words + g * 2)) : make_uint2(0u, 0u);
      uint32_t a0 = 0, a1 = 0, a2 = 0, a3 = 0;  // codes (0, 2), (1, 3), (4, 6), (5, 7), one per half word
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        a0 += c[q].x & 0x00FF00FFu; a1 += (c[q].x >> 8) & 0x00FF00FFu;
        a2 += c[q].y & 0x00FF00FFu; a3 += (c[q].y >> 8) & 0x00FF00FFu;
      }
      K[0] += (int)(a0 & 0xFFFFu); K[2] += (int)(a0 >> 16); K[1] += (int)(a1 & 0xFFFFu); K[3] += (int)(a1 >> 16);
      K[4] += (int)(a2 & 0xFFFFu); K[6] += (int)(a2 >> 16); K[5] += (int)(a3 & 0xFFFFu); K[7] += (int)(a3 >> 16);
    }
  } else if constexpr (BITS == 2) {
#pragma unroll 4
    for (int i = 0; i < N; ++i) {
      const uint32_t c = reinterpret_cast<const uint16_t*>(w + (int64_t)i * stride_words)[g];
#pragma unroll
      for (int e = 0; e < 8; ++e) K[e] += (int)((c >> (2 * e)) & 3u);
    }
  } else {
#pragma unroll 2
    for (int i = 0; i < N; ++i) {
      uint64_t lo, hi;
      load_chunk<0>(w + (int64_t)i * stride_words, g, b, pad_words, lo, hi);
#pragma unroll
      for (int e = 0; e < 8; ++e) K[e] += (int)extract(lo, hi, e * b, b);
    }
  }
}

// The server of schemes (b) and (c) (Section 3.2).  A thread owns 8 consecutive coordinates per sweep: it adds the
// codes of the N streams as integers, then either stores the index sums K_j in offset binary with b_out =
// b + ceil(log2 N) bits (scheme (b) grants the sum that many more bits), or rounds the average K_j / N back to the
// b-bit grid with rule (1) of Section 2.2 and the server's own rounding stream (scheme (c), Eq. 4).  The 8 * b_out
// output bits of a thread are b_out whole bytes: one or two words stored directly when b_out is 4 or 8, else staged
// through shared memory and written out as words.
template <int BITS>  // input width: 2, 4, 8 fixed; 0: b in 2..16 from the arguments
__global__ void __launch_bounds__(AT) server_reduce_kernel(ServerArgs a) {
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
#pragma unroll 1
  for (int it = 0; it < AITER; ++it) {
    const int64_t sweep0 = tstart + (int64_t)it * AGROUP;
    if (sweep0 >= s.len) break;  // uniform for the block
    const int64_t j = sweep0 + tid * 8;
    const int nvalid = (j < s.len) ? (int)min((int64_t)8, s.len - j) : 0;
    int K[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) K[e] = -bias_in;
    if (nvalid > 0) sum_codes8<BITS>(w, a.stride_words, a.N, j >> 3, b, s.pad_words, K);
    uint64_t olo = 0, ohi = 0;
    if (nvalid > 0) {
      if (a.requantize) {
        const U4 r = stream_block(a.seed, TAG_REQUANT, 0u, a.k, s.block_base + (uint32_t)(j >> 3));
        if constexpr (BITS != 0) {
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
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            if (e < nvalid) {
              const float avg = pow2 ? mul_rn((float)K[e], invN) : __fdiv_rn((float)K[e], fN);
              const uint32_t code = quantize_code_rt(avg, 1.0f, lane16(r, e), b);
              const int pos = e * bo;
              if (pos < 64) {
                olo |= (uint64_t)code << pos;
                if (pos + bo > 64) ohi |= (uint64_t)code >> (64 - pos);
              } else {
                ohi |= (uint64_t)code << (pos - 64);
              }
            }
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (e < nvalid) {
            const uint32_t code = (uint32_t)(K[e] + (1 << (bo - 1)));
            const int pos = e * bo;
            if (pos < 64) {
              olo |= (uint64_t)code << pos;
              if (pos + bo > 64) ohi |= (uint64_t)code >> (64 - pos);
            } else {
              ohi |= (uint64_t)code << (pos - 64);
            }
          }
        }
      }
    }
    if (direct) {  // uniform for the launch
      const int64_t g = j >> 3;
      if (bo == 4) {
        if (g < so.pad_words) out[g] = (uint32_t)olo;
      } else {
        if (2 * g < so.pad_words) *reinterpret_cast<uint2*>(out + 2 * g) = make_uint2((uint32_t)olo, (uint32_t)(olo >> 32));
      }
    } else {
      if (it > 0) __syncthreads();
      for (int i = 0; i < bo; ++i) stage[tid * bo + i] = (uint8_t)((i < 8) ? (olo >> (8 * i)) : (ohi >> (8 * (i - 8))));
      __syncthreads();
      const int64_t w0 = (sweep0 >> 5) * bo;  // sweep0 is a multiple of 2048, so this is exact
      const uint32_t* stw = reinterpret_cast<const uint32_t*>(stage);
      for (int q = tid; q < (AGROUP / 32) * bo; q += AT)
        if (w0 + q < so.pad_words) out[w0 + q] = stw[q];
    }
  }
}

}  // namespace

cudaError_t launch_server_reduce(const ServerArgs& a, cudaStream_t st) {
  if (a.ntiles <= 0) return cudaSuccess;
  const dim3 grid((unsigned)a.ntiles), block(AT);
  switch (a.b) {
    case 2: server_reduce_kernel<2><<<grid, block, 0, st>>>(a); break;
    case 4: server_reduce_kernel<4><<<grid, block, 0, st>>>(a); break;
    case 8: server_reduce_kernel<8><<<grid, block, 0, st>>>(a); break;
    default: server_reduce_kernel<0><<<grid, block, 0, st>>>(a); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_unpack_average_prox(const AggArgs& a, cudaStream_t st) {
  if (a.ntiles <= 0) return cudaSuccess;
  const dim3 grid((unsigned)a.ntiles), block(AT);
  const size_t sh = (size_t)a.N * sizeof(float);
  switch (a.b) {
    case 1: unpack_average_prox_kernel<1><<<grid, block, sh, st>>>(a); break;
    case 2: unpack_average_prox_kernel<2><<<grid, block, sh, st>>>(a); break;
    case 4: unpack_average_prox_kernel<4><<<grid, block, sh, st>>>(a); break;
    case 8: unpack_average_prox_kernel<8><<<grid, block, sh, st>>>(a); break;
    case 32: unpack_average_prox_kernel<32><<<grid, block, sh, st>>>(a); break;
    default: unpack_average_prox_kernel<0><<<grid, block, sh, st>>>(a); break;
  }
  return cudaGetLastError();
}

}  // namespace lpc
