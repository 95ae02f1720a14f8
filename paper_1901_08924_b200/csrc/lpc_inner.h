// Launch interface of the fused worker kernel and the small ALPC helper kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lpc {

struct InnerArgs {
  const float* X;
  const float* y;
  int64_t n;
  int d;
  int loss;
  int N, B, b;
  int clip_mode;
  float clip_value;
  uint64_t seed;
  int sample_global;
  uint64_t k_base;         // iteration number = k_base + *k_dev (k_dev nullable)
  const uint64_t* k_dev;
  const float* x;          // point where the minibatch gradients are taken (d)
  const float* margins;    // cached <X_a, snapshot> (n)
  const float* mu;         // snapshot gradient, read by the J cluster only
  int has_J;               // 1: an extra cluster (index N) handles ALPC's shared batch J
  float* vhat;             // d, written by the J cluster
  uint32_t* codes;         // N * stride_words
  int64_t stride_words;
  int64_t pad_words;       // words of one worker's stream including zero padding (multiple of 4)
  float* delta;            // N
  uint32_t* clipped_part;  // N * inner_clipped_stride()
  int64_t* idx_tap;        // (N+1) * B, nullable
  float* coef_tap;         // (N+1) * B, nullable
  float* u_tap;            // N * d, nullable
  unsigned int* dev_status;
  int CS;                  // CTAs per cluster
  int SL;                  // coordinates per CTA slice
  int stream_stages;       // 0: the B rows are resident in shared memory; > 0: they stream through that many ring stages
};

// Arguments of the persistent inner loop (lpc_persist.cu): `count` steps k_base, k_base+1, ... in one launch.
struct PersistArgs {
  InnerArgs in;              // in.x = iterate at entry, in.k_dev unused, in.has_J = 0
  int count;
  float eta;
  float lambda_l1;
  // Exchange buffers of tagged 64-bit words (payload | tag << 32), two step-parity halves each; a word is valid
  // for step t of this launch when its tag equals tag_base + t + 1.  Tags only grow from launch to launch, so
  // stale words never match and the buffers need no clearing between launches.
  unsigned long long* pub;   // scale delta: 2 x 256 words, 128 bytes apart, word (worker * CS + rank)
  unsigned long long* ll;    // codes: 2 x N x (CS*SL/8) groups x wpg words
  unsigned long long* ll_vhat;  // Algorithm 2's second estimator: 2 x CS*SL words
  uint32_t tag_base;
  int wpg;                   // words per group of 8 coordinates: 1 (b <= 4), 2 (b <= 8), 4 (b <= 16), 8 (b = 32)
  unsigned int* abort_flag;  // zero at launch; set when a bounded wait ran out
  float* x_out;              // iterate after `count` steps (may alias in.x)
  float* v_tap;              // nullable: v of the last step
  int row_slots;             // shared-memory row slots of SL floats: B .. 2B (2B: all rows of a step are fetched a step ahead)
  // Algorithm 2 (alpc = 1): in.x is not read; y, z, ysum are read at entry and written at exit, xt is the
  // snapshot, vhat (d floats) receives the last step's second estimator, x_out the last coupled point
  int alpc;
  float tau1, tau2, alpha, inv4L;
  // strongly convex case (h with a (sigma/2)*||.||^2 term): factors on the two soft-threshold results, the snapshot
  // weight of the launch's first step and its growth per step; all 1 in the general convex case
  float cy, cz, w0, theta;
  float* y;
  float* z;
  float* ysum;
  const float* xt;
  float* vhat;
};
bool persist_plan(int d, int N, int B, int b, int alpc, int want_cs, int max_smem, int* CS_out, int* SL_out,
                  size_t* smem_out, int* row_slots_out);
int persist_coords_per_thread(int b, int SL);
// cooperative = false drops the launch attribute that makes the driver guarantee co-residency of the grid (the plan has
// checked that all clusters fit; the kernel's waits are bounded): for profilers that cannot replay cooperative launches.
cudaError_t launch_persist(const PersistArgs& pa, size_t smem, cudaStream_t st, bool cooperative = true);
// One small kernel whose bounded waits (an mbarrier phase; a tagged word when `word` is given) run out after limit_ns.
cudaError_t launch_wait_timeout(const unsigned long long* word, unsigned int* abort_flag, unsigned int* dev_status,
                                uint64_t limit_ns, cudaStream_t st);

int inner_max_b();
int inner_clipped_stride();
bool inner_plan(int d, int B, int want_cs, int max_smem, int* CS_out, int* SL_out, size_t* smem_out, int* stages_out);
cudaError_t launch_inner(const InnerArgs& a, size_t smem, cudaStream_t st);
cudaError_t launch_clipped_sum(const uint32_t* part, int N, uint32_t* out, cudaStream_t st);
cudaError_t launch_coupling(const float* z, const float* xt, const float* y, float tau1, float tau2, int d, float* x,
                            cudaStream_t st);
cudaError_t launch_mean_y(float* ysum, float inv_m, int d, float* x, cudaStream_t st);

}  // namespace lpc
