// Communication step 1 (Algorithm 1 step 4): the snapshot full gradient
//   mu = grad f(x~) = (1/n) sum_a l'(<X_a, x~>, y_a) X_a
// in ONE pass over X, together with the margins <X_a, x~> (kept for the inner steps) and f(x~).
// The same kernel without the gradient part evaluates the objective's smooth part f(x).
//
// Design: a persistent grid of one CTA per SM, eleven warps in three roles.
//   * Eight compute warps.  A tile of R consecutive rows (contiguous in memory, 64 KB for d >= 2048) arrives in a ring
//     of shared-memory stages by one bulk copy (TMA) tracked by an mbarrier per stage.  Each compute thread copies its
//     part of a tile (columns 4t..4t+3 of every 1024-column chunk, all R rows: R*KMAX = 16 float4) from shared memory
//     into registers ONCE and hands the stage back; from the registers come the margin products, reduced across the
//     warp by recursive halving into the 128-column leaves of every row's margin tree, and -- once l' of the rows is
//     known -- the column sums, which also stay in registers.
//   * Two row warps, one for the even and one for the odd tiles of the CTA.  A row warp finishes the margin trees of
//     its tile's rows (all rows side by side, one lane group each), forms l' (fp64 for the logistic loss), publishes
//     the coefficients, and only then evaluates the loss value for f: the longer half of the fp64 chain (log1p) runs
//     while the compute warps are already on the next tile, whose rows belong to the other row warp.
//   * One copy warp refills a stage as soon as every compute thread has read it.
// Hand-overs are named barriers (bar.arrive by the producer side, bar.sync by the consumer side), one pair per tile
// parity: "leaves of tile i stored and stage read" and "coefficients of tile i stored".
// The margin of a row is the balanced-tree fp32 sum of its products in column order, so it is
// bit-identical to the margin any other kernel of the library computes for the same row and point.
#include "lpc_device.cuh"
#include "lpc_kernels.h"
#include "lpc_snapshot.h"

namespace lpc {
namespace {

constexpr int ST = 256;            // compute threads
constexpr int SNT = ST + 96;       // plus two row warps and the copy warp
constexpr int CHUNK = ST * 4;      // columns covered by one sweep of the compute threads
constexpr int SNAP_FIXED = 2048;   // bytes of shared memory before the stages: barriers, leaves, coefficients

__host__ __device__ constexpr int rows_per_tile(int kmax) { return kmax >= 16 ? 1 : 16 / kmax; }

constexpr int BAR_LEAF = 1, BAR_COEF = 3;  // named barriers BAR_LEAF + parity, BAR_COEF + parity
__device__ __forceinline__ void nb_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void nb_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }

template <int KMAX, bool GRAD>
__global__ void __launch_bounds__(SNT, 1) snapshot_kernel(SnapArgs a) {
  constexpr int R = rows_per_tile(KMAX);
  constexpr int NV = R * KMAX;  // float4 values per compute thread and tile
  constexpr int LOGV = 4;
  constexpr int NL = 8 * KMAX;  // 128-column leaves per row of the padded width
  static_assert(NV == 16, "register layout");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int d = a.d;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);            // nstage <= 8
  volatile int* fail = reinterpret_cast<volatile int*>(smem_raw + 64);
  float* coef = reinterpret_cast<float*>(smem_raw + 128);            // [2][16]
  float* part = reinterpret_cast<float*>(smem_raw + 256);            // [2][R * NL = 128]
  float* stages = reinterpret_cast<float*>(smem_raw + SNAP_FIXED);   // nstage * R * d

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t stage_floats = (int64_t)R * d;
  const int nstage = a.nstage;
  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) mbar_init(&bars[s], 1);
    *fail = 0;
    mbar_fence_init();
  }
  __syncthreads();

  int P = 1;
  while (P < d) P <<= 1;
  const int nleaf = (P >= 128) ? P / 128 : 1;  // leaves of the margin tree

  const int64_t my_tiles = (a.ntiles > (int64_t)blockIdx.x) ? (a.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  auto tile_row0 = [&](int64_t i) { return ((int64_t)blockIdx.x + i * gridDim.x) * R; };

  if (warp == ST / 32 + 2) {
    // ---- copy warp -----------------------------------------------------------------------------------------------
    auto issue = [&](int64_t i) {  // lane 0 only
      const int64_t row0 = tile_row0(i);
      const int rows = (int)min((int64_t)R, a.n - row0);
      const uint32_t bytes = (uint32_t)((int64_t)rows * d * 4);
      const int s = (int)(i % nstage);
      mbar_expect_tx(&bars[s], bytes);
      bulk_load(stages + (int64_t)s * stage_floats, a.X + row0 * d, bytes, &bars[s]);
    };
    int64_t issued = 0;
    if (lane == 0)
      for (; issued < min((int64_t)nstage, my_tiles); ++issued) issue(issued);
#pragma unroll 1
    for (int64_t i = 0; i < my_tiles; ++i) {
      nb_sync(BAR_LEAF + (int)(i & 1), ST + 64);  // every compute thread has its part of tile i in registers
      if (lane == 0 && issued < my_tiles && *fail == 0) { issue(issued); ++issued; }
    }
    if (lane == 0 && *fail != 0) {
      // a wait ran out: copies already issued may still land in this CTA's shared memory; give them one more bounded
      // chance to finish before the CTA exits
      for (int64_t i = max((int64_t)0, issued - nstage); i < issued; ++i)
        mbar_wait(&bars[i % nstage], (uint32_t)((i / nstage) & 1));
    }
  } else if (warp >= ST / 32) {
    // ---- row warps: lane group r finishes the margin tree of row r of a tile and applies the loss ------------------
    constexpr int VPL = 4;          // leaves per lane (R * NL = 128 per tile)
    constexpr int LPR = NL / VPL;   // lanes per row
    const int par = warp - ST / 32;  // this warp's tiles: par, par + 2, ...
    const int r = lane / LPR, f = (lane % LPR) * VPL;
    const bool head = (lane % LPR) == 0;
    float y_next = 0.f;
    if (head && par < my_tiles && tile_row0(par) + r < a.n) y_next = a.y[tile_row0(par) + r];
    double fsum = 0.0;
#pragma unroll 1
    for (int64_t i = par; i < my_tiles; i += 2) {
      nb_sync(BAR_LEAF + par, ST + 64);
      const int64_t row0 = tile_row0(i);
      const int rows = (int)min((int64_t)R, a.n - row0);
      const float4 v = *reinterpret_cast<const float4*>(part + par * (R * NL) + r * NL + f);
      float m = (nleaf >= 4) ? tree4(v.x, v.y, v.z, v.w) : (nleaf == 2) ? add_rn(v.x, v.y) : v.x;
#pragma unroll
      for (int s = 1; s < LPR; s <<= 1)
        if (s * VPL < nleaf) m = add_rn(m, __shfl_xor_sync(0xFFFFFFFFu, m, s));
      const bool mine = head && r < rows;
      const float yv = y_next;
      // l' first: the compute warps wait for it.  Logistic loss with t = y m and e = exp(-|t|) <= 1:
      //   l' = -y / (1 + exp(t)) = -y / (1 + e) for t <= 0, -y e / (1 + e) for t > 0;   l = max(-t, 0) + log1p(e).
      double t = 0.0, e = 0.0;
      float c = 0.f;
      if (mine) {
        if (a.loss == LOSS_LEAST_SQUARES) {
          c = __fsub_rn(m, yv);
          // Measured: when the coefficients follow the leaves at once (this chain is one subtraction), the pass runs a
          // tenth slower (6.4 against 7.2 TB/s on 131,072 x 4,096 and 262,144 x 8,192) than with the fifth of a
          // microsecond that the logistic chain takes anyway; a shorter pause (50, 100 ns) does not help, a longer one
          // (300 ns and more) puts the row warp on the critical path.
          __nanosleep(150);
        } else {
          t = __dmul_rn((double)yv, (double)m);
          e = exp(-fabs(t));
          const double num = (t > 0.0) ? __dmul_rn(-(double)yv, e) : -(double)yv;
          c = __double2float_rn(__ddiv_rn(num, __dadd_rn(1.0, e)));
        }
      }
      if (head) coef[par * 16 + r] = c;
      __syncwarp();
      nb_arrive(BAR_COEF + par, ST + 32);
      if (mine) {
        if (a.margins_out) a.margins_out[row0 + r] = m;
        if (a.loss == LOSS_LEAST_SQUARES) {
          const double res = (double)m - (double)yv;
          fsum += 0.5 * res * res;
        } else {
          fsum += ((t > 0.0) ? 0.0 : -t) + log1p(e);
        }
      }
      const int64_t nrow = tile_row0(i + 2) + r;  // same slot of this warp's next tile
      if (head && i + 2 < my_tiles && nrow < a.n) y_next = a.y[nrow];
    }
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) fsum += __shfl_xor_sync(0xFFFFFFFFu, fsum, s);
    if (lane == 0) a.partial_f[blockIdx.x * 2 + par] = fsum;
  } else {
    // ---- compute warps -------------------------------------------------------------------------------------------
    float4 xq[KMAX];  // this thread's columns of the point x
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      const int col = k * CHUNK + tid * 4;
      xq[k] = (col < d) ? *reinterpret_cast<const float4*>(a.x + col) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float4 acc[KMAX];
#pragma unroll
    for (int k = 0; k < KMAX; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    bool failed = false;  // after one wait ran out this thread waits no more (the status word says so)
#pragma unroll 1
    for (int64_t i = 0; i < my_tiles; ++i) {
      const int par = (int)(i & 1);
      const int s = (int)(i % nstage);
      if (!failed && !mbar_wait(&bars[s], (uint32_t)((i / nstage) & 1))) {
        failed = true;
        *fail = 1;
        atomicOr(a.dev_status, DEV_TIMEOUT);
      }
      const int rows = (int)min((int64_t)R, a.n - tile_row0(i));
      const float* st = stages + (int64_t)s * stage_floats;
      // tile -> registers, products, per-warp leaves (128 columns each) of every row's margin tree
      float4 xv[NV];
      float pv[NV];
#pragma unroll
      for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
          const int col = k * CHUNK + tid * 4;
          const int q = r * KMAX + k;
          xv[q] = (col < d && r < rows) ? *reinterpret_cast<const float4*>(st + (int64_t)r * d + col)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
          pv[q] = tree4(mul_rn(xv[q].x, xq[k].x), mul_rn(xv[q].y, xq[k].y), mul_rn(xv[q].z, xq[k].z), mul_rn(xv[q].w, xq[k].w));
        }
      }
      WarpHalving<NV, 0>::run(pv, lane);
      if ((lane >> LOGV) == 0) {
        const int q = halving_index<LOGV>(lane);  // the value left in this lane
        part[par * (R * NL) + (q / KMAX) * NL + (q % KMAX) * 8 + warp] = pv[0];
      }
      __syncwarp();
      nb_arrive(BAR_LEAF + par, ST + 64);  // leaves stored, and this thread is done with the stage
      nb_sync(BAR_COEF + par, ST + 32);
      if constexpr (GRAD) {  // column sums  acc += l'_r * X_r, from registers
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const float c = coef[par * 16 + r];
#pragma unroll
          for (int k = 0; k < KMAX; ++k) {
            const int q = r * KMAX + k;
            acc[k].x = __fmaf_rn(c, xv[q].x, acc[k].x);
            acc[k].y = __fmaf_rn(c, xv[q].y, acc[k].y);
            acc[k].z = __fmaf_rn(c, xv[q].z, acc[k].z);
            acc[k].w = __fmaf_rn(c, xv[q].w, acc[k].w);
          }
        }
      }
    }
    if constexpr (GRAD) {
      float* out = a.partial_mu + (int64_t)blockIdx.x * (KMAX * CHUNK);
#pragma unroll
      for (int k = 0; k < KMAX; ++k) *reinterpret_cast<float4*>(out + k * CHUNK + tid * 4) = acc[k];
    }
  }
}

// mu_j = (sum over CTAs of the partial column sums) / n, summed in CTA order in fp64; f likewise.
__global__ void snapshot_reduce_kernel(const float* __restrict__ partial_mu, const double* __restrict__ partial_f,
                                       int nparts, int dpad, int d, int64_t n, float* __restrict__ mu,
                                       float* __restrict__ mu_copy, double* __restrict__ f_out) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (partial_mu && j < d) {
    double s = 0.0;
    for (int c0 = 0; c0 < nparts; c0 += 8) {  // eight loads in flight, the additions in CTA order
      float v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = (c0 + i < nparts) ? partial_mu[(int64_t)(c0 + i) * dpad + j] : 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (c0 + i < nparts) s += (double)v[i];
    }
    const float v = (float)(s / (double)n);
    mu[j] = v;
    if (mu_copy) mu_copy[j] = v;
  }
  if (j == 0) {
    double s = 0.0;
    for (int c0 = 0; c0 < 2 * nparts; c0 += 8) {  // one partial per row warp of every CTA
      double v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = (c0 + i < 2 * nparts) ? partial_f[c0 + i] : 0.0;
#pragma unroll
      for (int i = 0; i < 8; ++i) s += v[i];
    }
    *f_out = s / (double)n;
  }
}

// The regulariser's two norms for P(x), without their weights: out[0] = ||x||_1, out[1] = ||x||^2.  One CTA, fp64.
__global__ void l1_norm_kernel(const float* __restrict__ x, int d, double* __restrict__ out) {
  __shared__ double sh[32], sh2[32];
  double s = 0.0, q = 0.0;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    const double v = (double)x[j];
    s += fabs(v);
    q += v * v;
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    s += __shfl_xor_sync(0xFFFFFFFFu, s, m);
    q += __shfl_xor_sync(0xFFFFFFFFu, q, m);
  }
  if ((threadIdx.x & 31) == 0) { sh[threadIdx.x >> 5] = s; sh2[threadIdx.x >> 5] = q; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0, t2 = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { t += sh[w]; t2 += sh2[w]; }
    out[0] = t;
    out[1] = t2;
  }
}

template <int KMAX>
cudaError_t launch_k(const SnapArgs& a, int grid, size_t smem, cudaStream_t st) {
  cudaError_t e;
  if (a.partial_mu) {
    e = cudaFuncSetAttribute(snapshot_kernel<KMAX, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    snapshot_kernel<KMAX, true><<<grid, SNT, smem, st>>>(a);
  } else {
    e = cudaFuncSetAttribute(snapshot_kernel<KMAX, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    snapshot_kernel<KMAX, false><<<grid, SNT, smem, st>>>(a);
  }
  return cudaGetLastError();
}

}  // namespace

int snapshot_dpad(int d) {
  int k = (d + CHUNK - 1) / CHUNK;
  int kmax = 1;
  while (kmax < k) kmax <<= 1;
  return kmax * CHUNK;
}

void snapshot_plan(int d, int max_smem, int* R_out, int* nstage_out, size_t* smem_out) {
  const int kmax = snapshot_dpad(d) / CHUNK;
  const int R = rows_per_tile(kmax);  // fixed by the register layout: R * kmax = 16 float4 per thread
  const size_t stage = (((size_t)R * d * 4) + 127) & ~(size_t)127;
  int nstage = (int)(((size_t)max_smem - SNAP_FIXED) / stage);
  if (nstage > 8) nstage = 8;
  if (nstage < 1) nstage = 1;
  *R_out = R; *nstage_out = nstage; *smem_out = SNAP_FIXED + (size_t)nstage * (size_t)R * d * 4;
}

cudaError_t launch_snapshot(const SnapArgs& a, int grid, size_t smem, cudaStream_t st) {
  const int kmax = snapshot_dpad(a.d) / CHUNK;
  switch (kmax) {
    case 1: return launch_k<1>(a, grid, smem, st);
    case 2: return launch_k<2>(a, grid, smem, st);
    case 4: return launch_k<4>(a, grid, smem, st);
    case 8: return launch_k<8>(a, grid, smem, st);
    case 16: return launch_k<16>(a, grid, smem, st);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_snapshot_reduce(const float* partial_mu, const double* partial_f, int nparts, int dpad, int d,
                                   int64_t n, float* mu, float* mu_copy, double* f_out, cudaStream_t st) {
  const int threads = 128;
  const int blocks = (d + threads - 1) / threads;
  snapshot_reduce_kernel<<<blocks > 0 ? blocks : 1, threads, 0, st>>>(partial_mu, partial_f, nparts, dpad, d, n, mu,
                                                                      mu_copy, f_out);
  return cudaGetLastError();
}

cudaError_t launch_l1_norm(const float* x, int d, double* out, cudaStream_t st) {
  l1_norm_kernel<<<1, 1024, 0, st>>>(x, d, out);
  return cudaGetLastError();
}

}  // namespace lpc
