// Communication step 1 (Algorithm 1 step 4): the snapshot full gradient
//   mu = grad f(x~) = (1/n) sum_a l'(<X_a, x~>, y_a) X_a
// in ONE pass over X, together with the margins <X_a, x~> (kept for the inner steps) and f(x~).
// The same kernel without the gradient part evaluates the objective's smooth part f(x).
//
// Design: a persistent grid of one CTA per SM.  A CTA pulls tiles of R consecutive rows (contiguous
// in memory) into a ring of shared-memory stages with one bulk-copy (TMA) transaction per tile,
// tracked by an mbarrier per stage, so several tiles are in flight per SM while one is processed.
// A tile is read from shared memory twice: once for the margins and once, scaled by l', for the
// column sums, which stay in registers (thread t owns columns 4t..4t+3 of every 1024-column chunk).
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

template <int KMAX, bool GRAD>
__global__ void __launch_bounds__(ST, 1) snapshot_kernel(SnapArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int d = a.d;
  const int dpad = KMAX * CHUNK;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);                       // nstage
  float* part = reinterpret_cast<float*>(smem_raw + 64);                        // R * MAXLEAF
  float* coef = part + a.R * MAXLEAF;                                           // R (padded to 4)
  float* xs = coef + ((a.R + 3) & ~3);                                          // dpad
  float* stages = xs + dpad;                                                    // nstage * R * d
  __shared__ double fsh[8];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t stage_floats = (int64_t)a.R * d;

  for (int c = tid; c < dpad; c += ST) xs[c] = (c < d) ? a.x[c] : 0.f;
  if (tid == 0) {
    for (int s = 0; s < a.nstage; ++s) mbar_init(&bars[s], 1);
    mbar_fence_init();
  }
  __syncthreads();

  // leaves of the margin tree
  int P = 1;
  while (P < d) P <<= 1;
  const int nleaf = (P >= 128) ? P / 128 : 1;

  const int64_t my_tiles = (a.ntiles > (int64_t)blockIdx.x) ? (a.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  auto issue = [&](int64_t i) {  // thread 0 only
    const int64_t tile = (int64_t)blockIdx.x + i * gridDim.x;
    const int64_t row0 = tile * a.R;
    const int rows = (int)min((int64_t)a.R, a.n - row0);
    const uint32_t bytes = (uint32_t)((int64_t)rows * d * 4);
    const int s = (int)(i % a.nstage);
    mbar_expect_tx(&bars[s], bytes);
    bulk_load(stages + (int64_t)s * stage_floats, a.X + row0 * d, bytes, &bars[s]);
  };
  if (tid == 0)
    for (int64_t i = 0; i < min((int64_t)a.nstage, my_tiles); ++i) issue(i);

  float4 acc[KMAX];
#pragma unroll
  for (int k = 0; k < KMAX; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  double fsum = 0.0;
  int64_t done = 0;  // tiles whose data has been consumed
  bool failed = false;

  for (int64_t i = 0; i < my_tiles; ++i) {
    const int s = (int)(i % a.nstage);
    const uint32_t parity = (uint32_t)((i / a.nstage) & 1);
    const int ok = mbar_wait(&bars[s], parity) ? 1 : 0;
    if (!__syncthreads_and(ok)) { failed = true; break; }
    const int64_t tile = (int64_t)blockIdx.x + i * gridDim.x;
    const int64_t row0 = tile * a.R;
    const int rows = (int)min((int64_t)a.R, a.n - row0);
    const float* st = stages + (int64_t)s * stage_floats;

    // phase A: partial tree sums of the products, one leaf (128 columns) per warp and chunk
    for (int r = 0; r < rows; ++r) {
      const float* row = st + (int64_t)r * d;
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        const int col = k * CHUNK + tid * 4;
        float sv = 0.f;
        if (col < d) {  // d is a multiple of 4
          const float4 xv = *reinterpret_cast<const float4*>(row + col);
          const float4 wv = *reinterpret_cast<const float4*>(xs + col);
          sv = tree4(mul_rn(xv.x, wv.x), mul_rn(xv.y, wv.y), mul_rn(xv.z, wv.z), mul_rn(xv.w, wv.w));
        }
        if (k * CHUNK < d) sv = warp_tree_sum(sv);  // chunks past the row contribute zero leaves
        if (lane == 0 && k * 8 + warp < nleaf) part[r * MAXLEAF + k * 8 + warp] = sv;
      }
    }
    __syncthreads();
    // phase B: warp r finishes row r's tree, applies the loss derivative
    for (int r = warp; r < rows; r += ST / 32) {
      float v4[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v4[e] = (lane * 4 + e < nleaf) ? part[r * MAXLEAF + lane * 4 + e] : 0.f;
      const float m = warp_tree_sum(tree4(v4[0], v4[1], v4[2], v4[3]));
      if (lane == 0) {
        const float yy = a.y[row0 + r];
        if (a.margins_out) a.margins_out[row0 + r] = m;
        coef[r] = loss_deriv(a.loss, m, yy);
        fsum += loss_value(a.loss, m, yy);
      }
    }
    if (GRAD) {
      __syncthreads();
      // phase C: column sums  acc += l'_r * X_r
      for (int r = 0; r < rows; ++r) {
        const float* row = st + (int64_t)r * d;
        const float c = coef[r];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
          const int col = k * CHUNK + tid * 4;
          if (col < d) {
            const float4 xv = *reinterpret_cast<const float4*>(row + col);
            acc[k].x = __fmaf_rn(c, xv.x, acc[k].x);
            acc[k].y = __fmaf_rn(c, xv.y, acc[k].y);
            acc[k].z = __fmaf_rn(c, xv.z, acc[k].z);
            acc[k].w = __fmaf_rn(c, xv.w, acc[k].w);
          }
        }
      }
    }
    __syncthreads();  // every thread is done reading stage s
    ++done;
    if (tid == 0 && i + a.nstage < my_tiles) issue(i + a.nstage);
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
    float* out = a.partial_mu + (int64_t)blockIdx.x * dpad;
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      const int col = k * CHUNK + tid * 4;
      *reinterpret_cast<float4*>(out + col) = acc[k];
    }
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

// lambda-free L1 norm partials for P(x): one CTA, fp64.
__global__ void l1_norm_kernel(const float* __restrict__ x, int d, double* __restrict__ out) {
  __shared__ double sh[32];
  double s = 0.0;
  for (int j = threadIdx.x; j < d; j += blockDim.x) s += fabs((double)x[j]);
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, m);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    *out = t;
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
  const int dpad = snapshot_dpad(d);
  const size_t row_bytes = (size_t)d * 4;
  int R = 1;
  while (R < 8 && (size_t)(2 * R) * row_bytes <= 65536) R <<= 1;  // up to 64 KB per stage
  for (;;) {
    const size_t fixed = 64 + ((size_t)R * MAXLEAF + ((R + 3) & ~3) + dpad) * 4;
    const size_t stage = (size_t)R * row_bytes;
    int nstage = (int)(((size_t)max_smem - fixed) / stage);
    if (nstage > 6) nstage = 6;
    if (nstage >= 2 || R == 1) {
      if (nstage < 1) nstage = 1;
      *R_out = R; *nstage_out = nstage; *smem_out = fixed + (size_t)nstage * stage;
      return;
    }
    R >>= 1;
  }
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
