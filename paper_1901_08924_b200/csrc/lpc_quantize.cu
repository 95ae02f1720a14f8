// Quantization step of Algorithm 1 (step 7) for stand-alone worker vectors: the scale of Eq. 2
// (a reduction pass), then the stochastic quantizer Q_(delta,b) of Section 2.2 and bit packing
// (a second pass).  Vectors may be split into tensor segments that each get their own scale.
//
// Layout of the work: a CTA owns one tile of TILE consecutive coordinates of one segment of one
// worker; a thread owns groups of 8 consecutive coordinates (two 128-bit loads, one Philox block,
// 8*b packed bits).  All sums follow the balanced binary tree over the coordinate index, so the
// scale -- and with it every code -- does not depend on the tiling.
#include "lpc_device.cuh"
#include "lpc_kernels.h"

namespace lpc {
namespace {

constexpr int QT = 256;                   // threads per CTA
constexpr int QGROUP = QT * 8;            // coordinates per CTA sweep
constexpr int QITER = TILE / QGROUP;      // sweeps per tile
static_assert(QITER * QGROUP == TILE, "tile must be a whole number of sweeps");

// Eight consecutive values u[j..j+8) of (p - q), zero beyond len.  `vec` says 16-byte loads are legal.
__device__ __forceinline__ void load8(const float* __restrict__ p, const float* __restrict__ q, int64_t j,
                                      int64_t len, bool vec, float* v) {
  if (vec && j + 8 <= len) {
    const float4 a = *reinterpret_cast<const float4*>(p + j);
    const float4 c = *reinterpret_cast<const float4*>(p + j + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
    if (q) {
      const float4 e = *reinterpret_cast<const float4*>(q + j);
      const float4 f = *reinterpret_cast<const float4*>(q + j + 4);
      v[0] = __fsub_rn(v[0], e.x); v[1] = __fsub_rn(v[1], e.y); v[2] = __fsub_rn(v[2], e.z); v[3] = __fsub_rn(v[3], e.w);
      v[4] = __fsub_rn(v[4], f.x); v[5] = __fsub_rn(v[5], f.y); v[6] = __fsub_rn(v[6], f.z); v[7] = __fsub_rn(v[7], f.w);
    }
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int64_t i = j + e;
      v[e] = (i < len) ? (q ? __fsub_rn(p[i], q[i]) : p[i]) : 0.f;
    }
  }
}

__device__ __forceinline__ bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- pass 1: per-tile partial (max |u| as bit pattern, tree sums of u and u^2) ---------------------------
template <bool NEED_SUMS>
__device__ __forceinline__ void stats_tile(const QuantArgs& a, int tile, int worker, float* sh1, float* sh2, uint32_t* shm) {
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  const SegInfo s = a.segs[seg];
  const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
  const float* p = a.U + (int64_t)worker * a.ld + s.off;
  const float* q = a.U_sub ? a.U_sub + (int64_t)worker * a.ld + s.off : nullptr;
  const bool vec = aligned16(p) && (!q || aligned16(q));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  uint32_t mx = 0;
#pragma unroll
  for (int it = 0; it < QITER; ++it) {
    const int64_t j = tstart + (int64_t)it * QGROUP + tid * 8;
    float v[8];
    if (j < s.len) {
      load8(p, q, j, s.len, vec, v);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) mx = max(mx, __float_as_uint(fabsf(v[e])));
    if (NEED_SUMS) {
      float sq[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) sq[e] = mul_rn(v[e], v[e]);
      const float s1 = warp_tree_sum(tree8(v));
      const float s2 = warp_tree_sum(tree8(sq));
      if (lane == 0) { sh1[it * 8 + warp] = s1; sh2[it * 8 + warp] = s2; }
    }
  }
  mx = warp_max_u32(mx);
  if (lane == 0) shm[warp] = mx;
  __syncthreads();
  if (tid == 0) {
    uint32_t m = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) m = max(m, shm[w]);
    const int64_t o = (int64_t)worker * a.ntiles + tile;
    a.pmax[o] = m;
    if (NEED_SUMS) {
      a.ps1[o] = smem_tree_sum(sh1, QITER * 8);
      a.ps2[o] = smem_tree_sum(sh2, QITER * 8);
    }
  }
}

template <bool NEED_SUMS>
__global__ void __launch_bounds__(QT) stats_kernel(QuantArgs a) {
  __shared__ float sh1[QITER * 8], sh2[QITER * 8];
  __shared__ uint32_t shm[8];
  stats_tile<NEED_SUMS>(a, blockIdx.x, blockIdx.y, sh1, sh2, shm);
}

// Tree sum over `count` tile partials by one CTA of QT threads (leaf order = tile order).
__device__ float block_tree_sum(const float* __restrict__ v, int count, float* sh8) {
  int64_t P = 1;
  while (P < count) P <<= 1;
  const int chunk = (P >= QT) ? (int)(P / QT) : 1;
  const int lo = threadIdx.x * chunk;
  float stack[32];
  int top = 0;
  for (int i = 0; i < chunk; ++i) {
    float cur = (lo + i < count) ? __ldcg(v + lo + i) : 0.f;  // written by other CTAs: read where they wrote it
    int idx = i;
    while (idx & 1) { cur = add_rn(stack[--top], cur); idx >>= 1; }
    stack[top++] = cur;
  }
  const float w = warp_tree_sum(stack[0]);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh8[threadIdx.x >> 5] = w;
  __syncthreads();
  return tree8(sh8);
}

// ---- between the passes: one CTA per (segment, worker) finishes the reductions and applies Eq. 2 -------
// The scale record of (segment, worker) from its tile partials, by all threads of the CTA; valid in thread 0.
__device__ __forceinline__ ScaleRec finish_segment(const QuantArgs& a, int seg, int worker, float* sh8, uint32_t* shm) {
  const SegInfo s = a.segs[seg];
  const int64_t base = (int64_t)worker * a.ntiles + s.tile_first;
  uint32_t mx = 0;
  for (int t = threadIdx.x; t < s.tile_count; t += QT) mx = max(mx, __ldcg(a.pmax + base + t));
  mx = warp_max_u32(mx);
  if ((threadIdx.x & 31) == 0) shm[threadIdx.x >> 5] = mx;
  float S1 = 0.f, S2 = 0.f;
  if (a.clip_mode == CLIP_STD) {
    S1 = block_tree_sum(a.ps1 + base, s.tile_count, sh8);
    S2 = block_tree_sum(a.ps2 + base, s.tile_count, sh8);
  }
  __syncthreads();
  ScaleRec r;
  r.delta = r.rdelta = r.T = r.lower = 0.f;
  r.flags = r.pad0 = r.pad1 = r.pad2 = 0;
  if (threadIdx.x == 0) {
    uint32_t m = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) m = max(m, shm[w]);
    const Scale sc = make_scale(m, S1, S2, s.len, a.b, a.clip_mode, a.clip_value);
    r.delta = sc.delta; r.rdelta = sc.rdelta; r.T = sc.T; r.lower = sc.lower; r.flags = sc.flags;
  }
  return r;
}

__global__ void __launch_bounds__(QT) finish_kernel(QuantArgs a) {
  const int seg = blockIdx.x, worker = blockIdx.y;
  __shared__ float sh8[8];
  __shared__ uint32_t shm[8];
  const ScaleRec r = finish_segment(a, seg, worker, sh8, shm);
  if (threadIdx.x == 0) {
    const int64_t o = (int64_t)worker * a.nseg + seg;
    a.scales[o] = r;
    a.delta_out[o] = r.delta;
    a.clipped_out[o] = 0;
    if (r.flags & 2u) atomicOr(a.dev_status, DEV_NONFINITE);
  }
}

// ---- schemes (b), (c) of Section 3.2: delta_t = max_i delta_t^i.  delta^i = T^i / levels grows with the threshold
// T^i, so the record of the worker with the largest threshold is the unified scale; it replaces every worker's
// record of the segment.  Workers whose own vector is zero then send zeros on the shared grid; when every worker
// is degenerate nothing changes.  One warp per segment.
__global__ void __launch_bounds__(32) share_scale_kernel(QuantArgs a) {
  const int seg = blockIdx.x, lane = threadIdx.x;
  float bestT = -1.f;
  int best = -1;
  for (int i = lane; i < a.N; i += 32) {
    const ScaleRec r = a.scales[(int64_t)i * a.nseg + seg];
    if (!(r.flags & 1u) && r.T > bestT) { bestT = r.T; best = i; }  // the first worker among equal thresholds
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    const float oT = __shfl_xor_sync(0xFFFFFFFFu, bestT, m);
    const int ob = __shfl_xor_sync(0xFFFFFFFFu, best, m);
    if (ob >= 0 && (best < 0 || oT > bestT || (oT == bestT && ob < best))) { bestT = oT; best = ob; }
  }
  if (best < 0) return;
  const ScaleRec r = a.scales[(int64_t)best * a.nseg + seg];
  __syncwarp();
  for (int i = lane; i < a.N; i += 32) {
    a.scales[(int64_t)i * a.nseg + seg] = r;
    a.delta_out[(int64_t)i * a.nseg + seg] = r.delta;
  }
}

// ---- pass 2: quantize and pack -----------------------------------------------------------------------------
// BITS = 1, 2, 3, 4, 8: register/shuffle packing with direct coalesced stores.
// BITS = 0: any b in 1..16 read from the arguments; each thread's 8*b bits are b whole bytes, staged
//           through shared memory and written out as words.
// A CTA takes a run of QRUN consecutive tiles of one worker.  Runs that consist of whole tiles of one segment of
// 16-byte aligned vectors (all but a segment's last tiles) go through a software-pipelined loop: the loads of the
// next sweeps are in flight while the current ones are quantized, nothing is tested per group and every index is a
// small offset from the run's base.  Everything else goes tile by tile through the general code.
constexpr int QRUN = 8;

template <int BITS>
__device__ __forceinline__ void store_group(uint32_t* __restrict__ ot, int g, int lane, uint64_t lo) {
  if (BITS == 8) {
    *reinterpret_cast<uint2*>(ot + 2 * g) = make_uint2((uint32_t)lo, (uint32_t)(lo >> 32));
  } else if (BITS == 4) {
    ot[g] = (uint32_t)lo;
  } else if (BITS == 2) {
    const uint32_t next = __shfl_down_sync(0xFFFFFFFFu, (uint32_t)lo, 1);
    if ((lane & 1) == 0) ot[g >> 1] = (uint32_t)lo | (next << 16);
  } else if (BITS == 3) {
    // 24 bits per thread: four neighbouring lanes hold three words; lane i < 3 of them builds word i from its own bits
    // and its neighbour's
    const uint32_t mine = (uint32_t)lo, next = __shfl_down_sync(0xFFFFFFFFu, mine, 1);
    const int i = lane & 3;
    if (i < 3) ot[3 * (g >> 2) + i] = (mine >> (8 * i)) | (next << (24 - 8 * i));
  } else {
    const uint32_t mine = (uint32_t)lo;
    const uint32_t n1 = __shfl_down_sync(0xFFFFFFFFu, mine, 1);
    const uint32_t n2 = __shfl_down_sync(0xFFFFFFFFu, mine, 2);
    const uint32_t n3 = __shfl_down_sync(0xFFFFFFFFu, mine, 3);
    if ((lane & 3) == 0) ot[g >> 2] = mine | (n1 << 8) | (n2 << 16) | (n3 << 24);
  }
}

// `nsweeps` sweeps of QGROUP coordinates from pt/qt (this thread's first group); HAS_Q: u = p - q.
// A step covers SW sweeps (2 without a subtrahend, 1 with), i.e. four 16-byte loads per thread; the loads of step
// i + 1 are issued before step i is quantized.
template <int BITS, bool COUNT, bool HAS_Q>
__device__ __forceinline__ void quantize_run(const QuantArgs& a, const ScaleRec& sc, const float* __restrict__ pt,
                                             const float* __restrict__ qt, uint32_t block0, uint32_t* __restrict__ ot,
                                             int nsweeps, int worker, int tid, int lane, float& fclip) {
  constexpr int SW = HAS_Q ? 1 : 2;
  const int nsteps = nsweeps / SW;  // a tile has QITER = 4 sweeps, so this is exact
  float4 cur[4], nxt[4];
  auto load = [&](float4* dst, int step) {
#pragma unroll
    for (int w = 0; w < SW; ++w) {
      const int off = (step * SW + w) * QGROUP;
      dst[2 * w] = __ldcs(reinterpret_cast<const float4*>(pt + off));
      dst[2 * w + 1] = __ldcs(reinterpret_cast<const float4*>(pt + off + 4));
      if (HAS_Q) {
        dst[2] = __ldcs(reinterpret_cast<const float4*>(qt + off));
        dst[3] = __ldcs(reinterpret_cast<const float4*>(qt + off + 4));
      }
    }
  };
  auto work = [&](const float4* src, int step) {
#pragma unroll
    for (int w = 0; w < SW; ++w) {
      float v[8] = {src[2 * w].x, src[2 * w].y, src[2 * w].z, src[2 * w].w,
                    src[2 * w + 1].x, src[2 * w + 1].y, src[2 * w + 1].z, src[2 * w + 1].w};
      if (HAS_Q) {
        v[0] = __fsub_rn(v[0], src[2].x); v[1] = __fsub_rn(v[1], src[2].y); v[2] = __fsub_rn(v[2], src[2].z);
        v[3] = __fsub_rn(v[3], src[2].w); v[4] = __fsub_rn(v[4], src[3].x); v[5] = __fsub_rn(v[5], src[3].y);
        v[6] = __fsub_rn(v[6], src[3].z); v[7] = __fsub_rn(v[7], src[3].w);
      }
      const int g = (step * SW + w) * (QGROUP / 8) + tid;  // coordinate group inside the run
      const U4 r = stream_block(a.seed, TAG_ROUND, (uint32_t)worker, a.k, block0 + (uint32_t)g);
      const uint64_t lo = quantize_group8<BITS, COUNT>(v, sc.rdelta, r, sc.T, sc.lower, fclip);
      store_group<BITS>(ot, g, lane, lo);
    }
  };
  load(cur, 0);
#pragma unroll 1
  for (int step = 0; step < nsteps; step += 2) {  // nsteps is even: a tile is 2 or 4 steps
    load(nxt, step + 1);
    work(cur, step);
    if (step + 2 < nsteps) load(cur, step + 2);
    work(nxt, step + 1);
  }
}

template <int BITS, bool COUNT>
__device__ __forceinline__ void quantize_tile(const QuantArgs& a, int tile, int worker, uint8_t* stage, const ScaleRec& sc) {
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  const SegInfo s = a.segs[seg];
  const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
  const float* p = a.U + (int64_t)worker * a.ld + s.off;
  const float* q = a.U_sub ? a.U_sub + (int64_t)worker * a.ld + s.off : nullptr;
  const bool vec = aligned16(p) && (!q || aligned16(q));
  const int tid = threadIdx.x, lane = tid & 31;
  const int b = BITS ? BITS : a.b;
  const bool degenerate = (sc.flags & 1u) != 0;
  const uint32_t zero_code = (b == 1) ? 0u : (1u << (b - 1));
  uint32_t* out = a.codes + (int64_t)worker * a.stride_words + s.word_off;

  uint32_t nclip = 0;
  float fclip = 0.f;
#pragma unroll
  for (int it = 0; it < QITER; ++it) {
    const int64_t sweep0 = tstart + (int64_t)it * QGROUP;  // first coordinate of this sweep (segment-local)
    const int64_t j = sweep0 + tid * 8;
    uint64_t lo = 0, hi = 0;  // this thread's 8*b bits
    const int nvalid = (j < s.len) ? (int)min((int64_t)8, s.len - j) : 0;
    if (nvalid > 0) {
      float v[8];
      load8(p, q, j, s.len, vec, v);
      if (!degenerate) {
        const U4 r = stream_block(a.seed, TAG_ROUND, (uint32_t)worker, a.k, s.block_base + (uint32_t)(j >> 3));
        if constexpr (BITS != 0) {
          // all eight coordinates are computed without bounds tests (zero padding is inside the hull and is
          // never counted); codes past the end are masked off below
          lo = quantize_group8<BITS ? BITS : 1, COUNT>(v, sc.rdelta, r, sc.T, sc.lower, fclip);
          if (nvalid < 8) lo &= (1ull << (nvalid * BITS)) - 1ull;
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            if (e < nvalid) {
              const uint32_t code = quantize_code_rt(v[e], sc.rdelta, lane16(r, e), b);
              if (COUNT) nclip += (v[e] > sc.T || v[e] < sc.lower) ? 1u : 0u;
              const int pos = e * b;
              if (pos < 64) {
                lo |= (uint64_t)code << pos;
                if (pos + b > 64) hi |= (uint64_t)code >> (64 - pos);
              } else {
                hi |= (uint64_t)code << (pos - 64);
              }
            }
          }
        }
      } else {
        for (int e = 0; e < nvalid; ++e) {
          const int pos = e * b;
          if (pos < 64) {
            lo |= (uint64_t)zero_code << pos;
            if (pos + b > 64) hi |= (uint64_t)zero_code >> (64 - pos);
          } else {
            hi |= (uint64_t)zero_code << (pos - 64);
          }
        }
      }
    }
    // ---- store
    if (BITS == 8) {
      const int64_t w = (j >> 3) * 2;
      if (w < s.pad_words) *reinterpret_cast<uint2*>(out + w) = make_uint2((uint32_t)lo, (uint32_t)(lo >> 32));
    } else if (BITS == 4) {
      const int64_t w = j >> 3;
      if (w < s.pad_words) out[w] = (uint32_t)lo;
    } else if (BITS == 2) {
      const uint32_t mine = (uint32_t)lo;  // 16 bits
      const uint32_t next = __shfl_down_sync(0xFFFFFFFFu, mine, 1);
      const int64_t w = j >> 4;
      if ((lane & 1) == 0 && w < s.pad_words) out[w] = mine | (next << 16);
    } else if (BITS == 1) {
      const uint32_t mine = (uint32_t)lo;  // 8 bits
      const uint32_t n1 = __shfl_down_sync(0xFFFFFFFFu, mine, 1);
      const uint32_t n2 = __shfl_down_sync(0xFFFFFFFFu, mine, 2);
      const uint32_t n3 = __shfl_down_sync(0xFFFFFFFFu, mine, 3);
      const int64_t w = j >> 5;
      if ((lane & 3) == 0 && w < s.pad_words) out[w] = mine | (n1 << 8) | (n2 << 16) | (n3 << 24);
    } else if (BITS == 3) {
      const uint32_t mine = (uint32_t)lo, next = __shfl_down_sync(0xFFFFFFFFu, mine, 1);  // 24 bits each
      const int i = lane & 3;
      const int64_t w = 3 * (j >> 5) + i;
      if (i < 3 && w < s.pad_words) out[w] = (mine >> (8 * i)) | (next << (24 - 8 * i));
    } else {
      // generic: b bytes per thread at byte tid*b of the sweep's 256*b-byte block
      if (it > 0) __syncthreads();
      for (int i = 0; i < b; ++i)
        stage[tid * b + i] = (uint8_t)((i < 8) ? (lo >> (8 * i)) : (hi >> (8 * (i - 8))));
      __syncthreads();
      const int64_t w0 = (sweep0 >> 5) * b;  // sweep0 is a multiple of 2048, so this is exact
      const uint32_t* st = reinterpret_cast<const uint32_t*>(stage);
      for (int w = tid; w < (QGROUP / 32) * b; w += QT)
        if (w0 + w < s.pad_words) out[w0 + w] = st[w];
    }
  }
  nclip = __reduce_add_sync(0xFFFFFFFFu, nclip + (uint32_t)fclip);
  if (COUNT && lane == 0 && nclip) atomicAdd(&a.clipped_out[(int64_t)worker * a.nseg + seg], nclip);
}

template <int BITS, bool COUNT>
__global__ void __launch_bounds__(QT, 4) quantize_kernel(QuantArgs a) {
  const int worker = blockIdx.y;
  const int tile0 = blockIdx.x * QRUN;
  const int ntl = min(QRUN, a.ntiles - tile0);
  __shared__ __align__(16) uint8_t stage[BITS == 0 ? QT * 16 : 16];
  if constexpr (BITS != 0) {
    const int seg = a.tile_seg ? a.tile_seg[tile0] : 0;
    const int seg_last = a.tile_seg ? a.tile_seg[tile0 + ntl - 1] : 0;  // tiles are numbered segment by segment
    if (seg == seg_last) {
      const SegInfo s = a.segs[seg];
      const int64_t tstart = (int64_t)(tile0 - s.tile_first) * TILE;
      const float* p = a.U + (int64_t)worker * a.ld + s.off;
      const float* q = a.U_sub ? a.U_sub + (int64_t)worker * a.ld + s.off : nullptr;
      const ScaleRec sc = a.scales[(int64_t)worker * a.nseg + seg];
      if (aligned16(p) && (!q || aligned16(q)) && !(sc.flags & 1u) && tstart + (int64_t)ntl * TILE <= s.len) {
        const int tid = threadIdx.x, lane = tid & 31;
        const uint32_t block0 = s.block_base + (uint32_t)(tstart >> 3);
        uint32_t* ot = a.codes + (int64_t)worker * a.stride_words + s.word_off + (tstart >> 5) * BITS;
        float fclip = 0.f;
        if (q)
          quantize_run<BITS ? BITS : 1, COUNT, true>(a, sc, p + tstart + tid * 8, q + tstart + tid * 8, block0, ot,
                                                     ntl * QITER, worker, tid, lane, fclip);
        else
          quantize_run<BITS ? BITS : 1, COUNT, false>(a, sc, p + tstart + tid * 8, nullptr, block0, ot, ntl * QITER,
                                                      worker, tid, lane, fclip);
        const uint32_t nclip = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)fclip);
        if (COUNT && lane == 0 && nclip) atomicAdd(&a.clipped_out[(int64_t)worker * a.nseg + seg], nclip);
        return;
      }
    }
  }
  for (int t = 0; t < ntl; ++t) {
    if (BITS == 0 && t > 0) __syncthreads();  // the staging buffer is reused from tile to tile
    const int seg = a.tile_seg ? a.tile_seg[tile0 + t] : 0;
    quantize_tile<BITS, COUNT>(a, tile0 + t, worker, stage, a.scales[(int64_t)worker * a.nseg + seg]);
  }
}

// ---- one launch for vectors that stay in L2 between the two passes ------------------------------------------------
// The grid is resident as a whole (cooperative launch) and every CTA takes the (worker, tile) pairs item, item + grid,
// ...: first their statistics, then -- once all tiles of a pair's (worker, segment) have reported, which a counter per
// (worker, segment) says -- the scale from the tile partials (every CTA that needs it forms it itself: same partials,
// same tree, same bits) and the codes of its tiles, whose values come from L2 this time.  Two kernel boundaries and the
// separate scale kernel are gone, which is most of the cost of a short vector.  The counters only grow: call number
// `epoch` waits for (epoch + 1) * tile_count arrivals.  A wait that runs out records a timeout and goes on.
template <int BITS, bool COUNT, bool NEED_SUMS>
__global__ void __launch_bounds__(QT, 4) quantize_fused_kernel(QuantArgs a, unsigned int* done, unsigned int epoch, int cpw) {
  __shared__ float sh1[QITER * 8], sh2[QITER * 8], sh8[8];
  __shared__ uint32_t shm[8];
  __shared__ ScaleRec srec;
  __shared__ __align__(16) uint8_t stage[BITS == 0 ? QT * 16 : 16];
  const int tid = threadIdx.x, lane = tid & 31;
  // CTA (chunk, worker) takes the tiles [t0, t1) of its worker: cpw chunks of consecutive tiles per worker
  const int worker = blockIdx.x / cpw, chunk = blockIdx.x % cpw;
  const int t0 = (int)((int64_t)a.ntiles * chunk / cpw), t1 = (int)((int64_t)a.ntiles * (chunk + 1) / cpw);
  for (int tile = t0; tile < t1; ++tile) {
    const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
    if (tile != t0) __syncthreads();  // the reduction buffers are reused from tile to tile
    stats_tile<NEED_SUMS>(a, tile, worker, sh1, sh2, shm);
    if (tid == 0) {
      const int64_t o = (int64_t)worker * a.nseg + seg;
      if (tile == a.segs[seg].tile_first) a.clipped_out[o] = 0;
      __threadfence();  // the partials (and the cleared count) before the arrival
      atomicAdd(&done[o], 1u);
    }
  }
  // segments without a single coordinate have no tile: their records are written here
  for (int o = blockIdx.x; o < a.N * a.nseg; o += gridDim.x) {
    const int w = o / a.nseg, seg = o % a.nseg;
    if (a.segs[seg].tile_count != 0) continue;
    __syncthreads();
    const ScaleRec r = finish_segment(a, seg, w, sh8, shm);
    if (tid == 0) { a.scales[o] = r; a.delta_out[o] = r.delta; a.clipped_out[o] = 0; }
  }
  int tile = t0;
  while (tile < t1) {  // one pass per tensor segment that the chunk touches
    const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
    const SegInfo s = a.segs[seg];
    const int tend = min(t1, s.tile_first + s.tile_count);
    const int o = worker * a.nseg + seg;
    if (tid == 0) {
      const unsigned int want = (epoch + 1u) * (unsigned int)s.tile_count;
      uint64_t t0ns = 0;
      for (uint32_t it = 0;; ++it) {
        unsigned int seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(done + o) : "memory");
        if (seen >= want) break;
        if ((it & 63u) == 63u) {
          const uint64_t now = global_ns();
          if (t0ns == 0) t0ns = now;
          else if (now - t0ns > 2000000000ull) { atomicOr(a.dev_status, DEV_TIMEOUT); break; }
        }
      }
    }
    __syncthreads();
    const ScaleRec r = finish_segment(a, seg, worker, sh8, shm);
    if (tid == 0) {
      srec = r;
      if (tile == s.tile_first) {  // one CTA leaves the record and the scale for the caller
        a.scales[o] = r;
        a.delta_out[o] = r.delta;
        if (r.flags & 2u) atomicOr(a.dev_status, DEV_NONFINITE);
      }
    }
    __syncthreads();
    const ScaleRec sc = srec;
    // whole tiles of aligned vectors go through the pipelined loop, the rest tile by tile
    const float* p = a.U + (int64_t)worker * a.ld + s.off;
    const float* q = a.U_sub ? a.U_sub + (int64_t)worker * a.ld + s.off : nullptr;
    int whole = 0;
    if constexpr (BITS != 0) {
      if (aligned16(p) && (!q || aligned16(q)) && !(sc.flags & 1u)) {
        const int64_t full_tiles = s.len / TILE;  // tiles of the segment without a ragged end
        whole = (int)max((int64_t)0, min((int64_t)(tend - s.tile_first), full_tiles) - (tile - s.tile_first));
      }
      if (whole > 0) {
        const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
        const uint32_t block0 = s.block_base + (uint32_t)(tstart >> 3);
        uint32_t* ot = a.codes + (int64_t)worker * a.stride_words + s.word_off + (tstart >> 5) * BITS;
        float fclip = 0.f;
        if (q)
          quantize_run<BITS ? BITS : 1, COUNT, true>(a, sc, p + tstart + tid * 8, q + tstart + tid * 8, block0, ot, whole * QITER,
                                                     worker, tid, lane, fclip);
        else
          quantize_run<BITS ? BITS : 1, COUNT, false>(a, sc, p + tstart + tid * 8, nullptr, block0, ot, whole * QITER, worker,
                                                      tid, lane, fclip);
        const uint32_t nclip = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)fclip);
        if (COUNT && lane == 0 && nclip) atomicAdd(&a.clipped_out[o], nclip);
      }
    }
    for (int t = tile + whole; t < tend; ++t) {
      if (BITS == 0 && t > tile) __syncthreads();  // the staging buffer is reused from tile to tile
      quantize_tile<BITS, COUNT>(a, t, worker, stage, sc);
    }
    tile = tend;
    if (tile < t1) __syncthreads();  // srec and the reduction buffers are reused for the next segment
  }
}

// b = 32: the message is the vector itself (clamped to [-T, T] when a clip rule is set).
__device__ __forceinline__ void bypass_tile(const QuantArgs& a, int tile, int worker, const ScaleRec& sc) {
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  const SegInfo s = a.segs[seg];
  const int64_t tstart = (int64_t)(tile - s.tile_first) * TILE;
  const float* p = a.U + (int64_t)worker * a.ld + s.off;
  const float* q = a.U_sub ? a.U_sub + (int64_t)worker * a.ld + s.off : nullptr;
  const bool vec = aligned16(p) && (!q || aligned16(q));
  const int tid = threadIdx.x, lane = tid & 31;
  uint32_t* out = a.codes + (int64_t)worker * a.stride_words + s.word_off;
  uint32_t nclip = 0;
#pragma unroll
  for (int it = 0; it < QITER; ++it) {
    const int64_t j = tstart + (int64_t)it * QGROUP + tid * 8;
    if (j >= s.pad_words) continue;
    float v[8];
    if (j < s.len) {
      load8(p, q, j, s.len, vec, v);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = 0.f;
    }
    if (a.clip_mode != CLIP_NONE) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        if (j + e < s.len) {
          if (v[e] > sc.T) { v[e] = sc.T; ++nclip; }
          if (v[e] < -sc.T) { v[e] = -sc.T; ++nclip; }
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (j + e < s.pad_words) out[j + e] = (j + e < s.len) ? __float_as_uint(v[e]) : 0u;
  }
  nclip = __reduce_add_sync(0xFFFFFFFFu, nclip);
  if (lane == 0 && nclip) atomicAdd(&a.clipped_out[(int64_t)worker * a.nseg + seg], nclip);
}

__global__ void __launch_bounds__(QT) bypass_kernel(QuantArgs a) {
  const int tile = blockIdx.x, worker = blockIdx.y;
  const int seg = a.tile_seg ? a.tile_seg[tile] : 0;
  bypass_tile(a, tile, worker, a.scales[(int64_t)worker * a.nseg + seg]);
}

using FusedKernel = void (*)(QuantArgs, unsigned int*, unsigned int, int);
template <int BITS>
FusedKernel pick_fused(bool count, bool sums) {
  if (count) return sums ? quantize_fused_kernel<BITS, true, true> : quantize_fused_kernel<BITS, true, false>;
  return sums ? quantize_fused_kernel<BITS, false, true> : quantize_fused_kernel<BITS, false, false>;
}

}  // namespace

// The one-launch path (see quantize_fused_kernel): `done` holds N * nseg arrival counters that have seen `epoch` calls
// with this layout.  Returns cudaErrorCooperativeLaunchTooLarge when no CTA of the kernel fits on the device.
cudaError_t launch_quantize_fused(const QuantArgs& a, unsigned int* done, unsigned int epoch, int sm_count, cudaStream_t st) {
  if (a.N <= 0 || a.nseg <= 0) return cudaSuccess;
  FusedKernel k;
  const bool sums = a.clip_mode == CLIP_STD, count = a.count_clipped != 0;
  switch (a.b) {
    case 1: k = pick_fused<1>(count, sums); break;
    case 2: k = pick_fused<2>(count, sums); break;
    case 3: k = pick_fused<3>(count, sums); break;
    case 4: k = pick_fused<4>(count, sums); break;
    case 8: k = pick_fused<8>(count, sums); break;
    default: k = pick_fused<0>(count, sums); break;
  }
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, QT, 0);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
  const long long resident = (long long)per_sm * sm_count;
  if (resident < a.N) return cudaErrorCooperativeLaunchTooLarge;
  // chunks of consecutive tiles per worker: as many as fit the resident grid, at most one per tile
  long long cpw = resident / a.N;
  if (cpw > a.ntiles) cpw = a.ntiles;
  if (cpw < 1) cpw = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(cpw * a.N), 1, 1);
  cfg.blockDim = dim3(QT, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident or the launch fails: they wait on one another
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k, a, done, epoch, (int)cpw);
}

int quantize_run_tiles() { return QRUN; }

cudaError_t launch_quantize_pack(const QuantArgs& a, cudaStream_t st, LaunchHook hook, void* user) {
  if (a.N <= 0 || a.nseg <= 0) return cudaSuccess;
  const dim3 grid((unsigned)(a.ntiles > 0 ? a.ntiles : 1), (unsigned)a.N), block(QT);
  if (a.ntiles > 0) {
    if (hook) hook(user, 3 /* LPC_KERNEL_QUANT_STATS */, 1);
    if (a.clip_mode == CLIP_STD)
      stats_kernel<true><<<grid, block, 0, st>>>(a);
    else
      stats_kernel<false><<<grid, block, 0, st>>>(a);
    if (hook) hook(user, 3, 0);
  }
  if (hook) hook(user, 5 /* LPC_KERNEL_OTHER */, 1);
  finish_kernel<<<dim3((unsigned)a.nseg, (unsigned)a.N), block, 0, st>>>(a);  // also covers empty segments
  if (hook) hook(user, 5, 0);
  if (a.shared_scale) share_scale_kernel<<<(unsigned)a.nseg, 32, 0, st>>>(a);
  if (a.ntiles <= 0) return cudaGetLastError();
  struct Close {  // closes the timing scope of the second pass on every return path
    LaunchHook h; void* u;
    ~Close() { if (h) h(u, 4, 0); }
  } close_{hook, user};
  if (hook) hook(user, 4 /* LPC_KERNEL_QUANT_PACK */, 1);
  const dim3 grid_tiles = grid;  // one tile per CTA: the statistics pass and the full-precision bypass
  const dim3 grid_runs((unsigned)((a.ntiles + QRUN - 1) / QRUN), (unsigned)a.N);  // QRUN tiles per CTA
  if (a.count_clipped) {
    switch (a.b) {
      case 1: quantize_kernel<1, true><<<grid_runs, block, 0, st>>>(a); break;
      case 2: quantize_kernel<2, true><<<grid_runs, block, 0, st>>>(a); break;
      case 3: quantize_kernel<3, true><<<grid_runs, block, 0, st>>>(a); break;
      case 4: quantize_kernel<4, true><<<grid_runs, block, 0, st>>>(a); break;
      case 8: quantize_kernel<8, true><<<grid_runs, block, 0, st>>>(a); break;
      case 32: bypass_kernel<<<grid_tiles, block, 0, st>>>(a); break;
      default: quantize_kernel<0, true><<<grid_runs, block, 0, st>>>(a); break;
    }
  } else {
    switch (a.b) {
      case 1: quantize_kernel<1, false><<<grid_runs, block, 0, st>>>(a); break;
      case 2: quantize_kernel<2, false><<<grid_runs, block, 0, st>>>(a); break;
      case 3: quantize_kernel<3, false><<<grid_runs, block, 0, st>>>(a); break;
      case 4: quantize_kernel<4, false><<<grid_runs, block, 0, st>>>(a); break;
      case 8: quantize_kernel<8, false><<<grid_runs, block, 0, st>>>(a); break;
      case 32: bypass_kernel<<<grid_tiles, block, 0, st>>>(a); break;
      default: quantize_kernel<0, false><<<grid_runs, block, 0, st>>>(a); break;
    }
  }
  return cudaGetLastError();
}

}  // namespace lpc

namespace lpc {
namespace {
__global__ void stream_blocks_kernel(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block0,
                                     int64_t count, uint32_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) {
    const U4 r = stream_block(seed, tag, worker, k, block0 + (uint32_t)i);
    out[4 * i + 0] = r.x; out[4 * i + 1] = r.y; out[4 * i + 2] = r.z; out[4 * i + 3] = r.w;
  }
}
}  // namespace

cudaError_t launch_stream_blocks(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block0,
                                 int64_t count, uint32_t* out, cudaStream_t st) {
  stream_blocks_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(seed, tag, worker, k, block0, count, out);
  return cudaGetLastError();
}
}  // namespace lpc
