// Communication step 1 (Algorithm 1 step 4): the snapshot full gradient
//   mu = grad f(x~) = (1/n) sum_a l'(<X_a, x~>, y_a) X_a
// in ONE pass over X, together with the margins <X_a, x~> (kept for the inner steps) and f(x~).
// The same kernel without the gradient part evaluates the objective's smooth part f(x).
//
// Design: a persistent grid of one CTA per SM.  A CTA pulls tiles of R consecutive rows (contiguous
// in memory) into a ring of shared-memory stages with one bulk-copy (TMA) transaction per tile,
// tracked by an mbarrier per stage, so several tiles are in flight per SM while one is processed.
// Each thread copies its part of a tile (columns 4t..4t+3 of every 1024-column chunk, all R rows:
// R*KMAX = 16 float4) from shared memory into registers ONCE; the stage is handed back to the copy
// engine right after that.  From the registers come both the margin products and, once l' is known,
// the column sums, which also stay in registers.  The 16 per-thread partial products are reduced
// across the warp by recursive halving (16 shuffles instead of 16 x 5).
// The margin of a row is the balanced-tree fp32 sum of its products in column order, so it is
// bit-identical to the margin any other kernel of the library computes for the same row and point.
#include "lpc_device.cuh"
#include "lpc_kernels.h"
#include "lpc_snapshot.h"

namespace lpc {
namespace {

constexpr int ST = 256;       // threads
constexpr int CHUNK = ST * 4; // columns covered by one sweep of the CTA
constexpr int MAXLEAF = 128;  // 128-column leaves of the margin tree: d <= 16384

__host__ __device__ constexpr int rows_per_tile(int kmax) { return kmax >= 16 ? 1 : kmax >= 8 ? 2 : kmax >= 4 ? 4 : 8; }

template <int KMAX, bool GRAD>
__global__ void __launch_bounds__(ST, 1) snapshot_kernel(SnapArgs a) {
  constexpr int R = rows_per_tile(KMAX);
  constexpr int NV = R * KMAX;  // float4 values per thread and tile
  constexpr int LOGV = NV == 16 ? 4 : NV == 8 ? 3 : NV == 4 ? 2 : NV == 2 ? 1 : 0;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int d = a.d;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);                       // nstage
  float* part = reinterpret_cast<float*>(smem_raw + 64);                        // R * MAXLEAF
  float* coef = part + R * MAXLEAF;                                             // 8
  float* stages = coef + 8;                                                     // nstage * R * d
  __shared__ double fsh[8];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t stage_floats = (int64_t)R * d;

  // this thread's columns of the point x
  float4 xq[KMAX];
#pragma unroll
  for (int k = 0; k < KMAX; ++k) {
    const int col = k * CHUNK + tid * 4;
    xq[k] = (col < d) ? *reinterpret_cast<const float4*>(a.x + col) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (tid == 0) {
    for (int s = 0; s < a.nstage; ++s) mbar_init(&bars[s], 1);
    mbar_fence_init();
  }
  __syncthreads();

  int P = 1;
  while (P < d) P <<= 1;
  const int nleaf = (P >= 128) ? P / 128 : 1;  // leaves of the margin tree

  const int64_t my_tiles = (a.ntiles > (int64_t)blockIdx.x) ? (a.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  auto issue = [&](int64_t i) {  // thread 0 only
    const int64_t row0 = ((int64_t)blockIdx.x + i * gridDim.x) * R;
    const int rows = (int)min((int64_t)R, a.n - row0);
    const uint32_t bytes = (uint32_t)((int64_t)rows * d * 4);
    const int s = (int)(i % a.nstage);
    mbar_expect_tx(&bars[s], bytes);
    bulk_load(stages + (int64_t)s * stage_floats, a.X + row0 * d, bytes, &bars[s]);
  };
  if (tid == 0)
    for (int64_t i = 0; i < min((int64_t)a.nstage, my_tiles); ++i) issue(i);

  // lane 0 of warp r owns row r of a tile: its label is fetched one tile ahead
  float y_next = 0.f;
  if (lane == 0 && warp < R && my_tiles > 0) {
    const int64_t row = (int64_t)blockIdx.x * R + warp;
    if (row < a.n) y_next = a.y[row];
  }

  float4 acc[KMAX];
#pragma unroll
  for (int k = 0; k < KMAX; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  double fsum = 0.0;
  int64_t done = 0;  // tiles whose data has been consumed
  bool failed = false;

#pragma unroll 1
  for (int64_t i = 0; i < my_tiles; ++i) {
    const int s = (int)(i % a.nstage);
    const uint32_t parity = (uint32_t)((i / a.nstage) & 1);
    const int ok = mbar_wait(&bars[s], parity) ? 1 : 0;
    if (!__syncthreads_and(ok)) { failed = true; break; }
    const int64_t row0 = ((int64_t)blockIdx.x + i * gridDim.x) * R;
    const int rows = (int)min((int64_t)R, a.n - row0);
    const float* st = stages + (int64_t)s * stage_floats;

    // phase A: tile -> registers, products, per-warp leaves (128 columns each) of every row's margin tree
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
      // the value left in this lane belongs to q whose bits, most significant first, are the lane's low bits
      int q = 0;
#pragma unroll
      for (int sft = 0; sft < LOGV; ++sft) q |= ((lane >> sft) & 1) << (LOGV - 1 - sft);
      const int r = q / KMAX, k = q % KMAX;
      if (k * 8 + warp < nleaf) part[r * MAXLEAF + k * 8 + warp] = pv[0];
    }
    __syncthreads();  // leaves visible; every thread holds its part of the tile in registers
    ++done;
    if (tid == 0 && i + a.nstage < my_tiles) issue(i + a.nstage);  // the stage can be refilled already

    // phase B: warp r finishes row r's tree and applies the loss derivative
    if (warp < R) {
      float v4[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v4[e] = (lane * 4 + e < nleaf) ? part[warp * MAXLEAF + lane * 4 + e] : 0.f;
      const float m = warp_tree_sum(tree4(v4[0], v4[1], v4[2], v4[3]));
      if (lane == 0) {
        float c = 0.f;
        if (warp < rows) {
          if (a.margins_out) a.margins_out[row0 + warp] = m;
          c = loss_deriv(a.loss, m, y_next);
          fsum += loss_value(a.loss, m, y_next);
        }
        coef[warp] = c;
        const int64_t nrow = row0 + (int64_t)gridDim.x * R + warp;  // same slot of this CTA's next tile
        if (i + 1 < my_tiles && nrow < a.n) y_next = a.y[nrow];
      }
    }
    if (GRAD) {
      __syncthreads();
      // phase C: column sums  acc += l'_r * X_r, from registers
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float c = coef[r];
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

  if (failed) {
    if (tid == 0) {
      atomicOr(a.dev_status, DEV_TIMEOUT);
      // copies already issued may still land in this CTA's shared memory: give them one more bounded
      // chance to finish before the CTA exits
      const int64_t issued = min(my_tiles, done + a.nstage);
      for (int64_t i = done; i < issued; ++i) mbar_wait(&bars[i % a.nstage], (uint32_t)((i / a.nstage) & 1));
    }
    __syncthreads();
  }

  if (GRAD) {
    float* out = a.partial_mu + (int64_t)blockIdx.x * (KMAX * CHUNK);
#pragma unroll
    for (int k = 0; k < KMAX; ++k) *reinterpret_cast<float4*>(out + k * CHUNK + tid * 4) = acc[k];
  }
  // f partial of this CTA
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) fsum += __shfl_xor_sync(0xFFFFFFFFu, fsum, m);
  if (lane == 0) fsh[warp] = fsum;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < ST / 32; ++w) t += fsh[w];
    a.partial_f[blockIdx.x] = t;
  }
}

// mu_j = (sum over CTAs of the partial column sums) / n, summed in CTA order in fp64; f likewise.
__global__ void snapshot_reduce_kernel(const float* __restrict__ partial_mu, const double* __restrict__ partial_f,
                                       int nparts, int dpad, int d, int64_t n, float* __restrict__ mu,
                                       float* __restrict__ mu_copy, double* __restrict__ f_out) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (partial_mu && j < d) {
    double s = 0.0;
    for (int c = 0; c < nparts; ++c) s += (double)partial_mu[(int64_t)c * dpad + j];
    const float v = (float)(s / (double)n);
    mu[j] = v;
    if (mu_copy) mu_copy[j] = v;
  }
  if (j == 0) {
    double s = 0.0;
    for (int c = 0; c < nparts; ++c) s += partial_f[c];
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
    snapshot_kernel<KMAX, true><<<grid, ST, smem, st>>>(a);
  } else {
    e = cudaFuncSetAttribute(snapshot_kernel<KMAX, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    snapshot_kernel<KMAX, false><<<grid, ST, smem, st>>>(a);
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
  const int R = rows_per_tile(kmax);  // fixed by the register layout: R * kmax = 16 float4 per thread (8 for kmax = 1)
  const size_t fixed = 64 + ((size_t)R * MAXLEAF + 8) * 4;
  const size_t stage = (size_t)R * d * 4;
  int nstage = (int)(((size_t)max_smem - fixed) / stage);
  if (nstage > 8) nstage = 8;
  if (nstage < 1) nstage = 1;
  *R_out = R; *nstage_out = nstage; *smem_out = fixed + (size_t)nstage * stage;
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
