// Launch interface of the snapshot full-gradient / objective pass.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lpc {

struct SnapArgs {
  const float* X;      // n x d
  const float* y;      // n
  const float* x;      // point at which margins and gradient are taken (d)
  int64_t n;
  int d;
  int loss;
  int R;               // rows per tile
  int nstage;          // shared-memory stages
  int64_t ntiles;      // ceil(n / R)
  float* partial_mu;   // grid * dpad column sums, or NULL for the objective-only pass
  float* margins_out;  // n, nullable
  double* partial_f;   // 2 * grid: one partial sum of f per row warp of every CTA
  unsigned int* dev_status;
};

int snapshot_dpad(int d);  // columns padded to the per-thread register layout
void snapshot_plan(int d, int max_smem, int* R_out, int* nstage_out, size_t* smem_out);
cudaError_t launch_snapshot(const SnapArgs& a, int grid, size_t smem, cudaStream_t st);
cudaError_t launch_snapshot_reduce(const float* partial_mu, const double* partial_f, int nparts, int dpad, int d,
                                   int64_t n, float* mu, float* mu_copy, double* f_out, cudaStream_t st);
cudaError_t launch_l1_norm(const float* x, int d, double* out, cudaStream_t st);

}  // namespace lpc
