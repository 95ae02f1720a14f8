// Internal launch interface between the C ABI (lpc_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lpc {

constexpr int TILE = 8192;  // coordinates per CTA tile of the standalone quantizer / aggregator kernels

// One tensor segment of a (segmented) vector.
struct SegInfo {
  int64_t off;         // first element in the vector
  int64_t len;         // elements
  int64_t word_off;    // first word of its packed stream inside a worker's stream (multiple of 4)
  int64_t pad_words;   // words reserved for it (multiple of 4)
  uint32_t block_base; // first Philox block of its rounding stream
  int32_t tile_first;  // first tile index
  int32_t tile_count;
  int32_t pad_;
};

struct ScaleRec {  // result of the scale rule for one (worker, segment)
  float delta, rdelta, T, lower;
  uint32_t flags, pad0, pad1, pad2;
};

struct QuantArgs {
  const float* U;
  const float* U_sub;  // nullable
  int64_t ld;
  int N;
  int b;
  int clip_mode;
  float clip_value;
  uint64_t seed;
  uint64_t k;
  const SegInfo* segs;     // device, nseg entries
  const int32_t* tile_seg; // device, ntiles entries
  int nseg;
  int ntiles;
  // scratch
  uint32_t* pmax;  // N * ntiles
  float* ps1;      // N * ntiles
  float* ps2;      // N * ntiles
  ScaleRec* scales;  // N * nseg
  // outputs
  uint32_t* codes;
  int64_t stride_words;
  float* delta_out;       // N * nseg
  uint32_t* clipped_out;  // N * nseg, cleared by the finish kernel (never null: internal scratch when the caller gives none)
  int count_clipped;      // 0: skip counting the coordinates outside the hull (the counts stay zero)
  int shared_scale;       // 1: every worker quantizes with delta_t = max_i delta_t^i (schemes (b), (c) of Section 3.2)
  unsigned int* dev_status;
};

// hook(user, kind, begin) is called around each kernel of the sequence (kind = LPC_KERNEL_* of lpc.h) when non-null.
typedef void (*LaunchHook)(void* user, int kind, int begin);
// Tiles per CTA of the second pass, and whether the run of tiles that starts at tile0 consists of whole tiles of one
// segment (the condition, besides 16-byte aligned vectors and a non-degenerate scale, for its pipelined loop).
int quantize_run_tiles();
cudaError_t launch_quantize_pack(const QuantArgs& a, cudaStream_t st, LaunchHook hook = nullptr, void* user = nullptr);
// The same work in one cooperative launch, for vectors short enough to stay in L2 between the statistics and the codes
// (b in 1..16, own scales).  done: N * nseg arrival counters, zero before the first call with a layout; epoch: calls
// made with that layout since.
cudaError_t launch_quantize_fused(const QuantArgs& a, unsigned int* done, unsigned int epoch, int sm_count, cudaStream_t st);

struct AggArgs {
  const uint32_t* codes;
  int64_t stride_words;
  const float* delta;  // N * nseg
  int N;
  int b;
  int divisor;      // the decoded sum is divided by this count: N for Eq. 3; the worker count behind a server's sum stream
  const SegInfo* segs;
  const int32_t* tile_seg;
  int nseg;
  int ntiles;
  const float* mu;  // nullable
  float* x;         // in/out
  float eta;
  float lambda_l1;
  float* v_out;     // nullable
  uint64_t* k_counter;  // nullable: incremented by one when the kernel finishes (graph replay)
  // mode 1 (Algorithm 2, steps 12-13): x is read only (the coupled point x_{k+1}) and instead of the
  // proximal step on x the kernel updates  y = soft(x - inv4L*v, inv4L*lambda_l1),
  // z = soft(z - alpha*vhat, alpha*lambda_l1),  ysum += y.
  int mode;
  float* y;
  float* z;
  float* ysum;
  const float* vhat;
  float alpha;
  float inv4L;
  // strongly convex case of Algorithm 2, h = lambda_l1*||.||_1 + (sigma/2)*||.||^2: the soft-threshold results are
  // multiplied by cy = 1/(1 + sigma*inv4L) and cz = 1/(1 + alpha*sigma), and ysum += wy * y (the snapshot weight
  // (1 + alpha*sigma)^t of the step).  All three are 1 in the general convex case, where they change no bit.
  float cy, cz, wy;
  int split;  // CTAs per tile (1, 2 or 4): aggregate_split(ntiles, sm_count), set by the caller
};

// CTAs that share one tile of the aggregator: below two waves of resident CTAs (4 per SM) a tile's sweeps are spread
// over 2 or 4 CTAs so that short vectors still fill the machine.
int aggregate_split(int ntiles, int sm_count);
cudaError_t launch_unpack_average_prox(const AggArgs& a, cudaStream_t st);

// The server of the parameter-server schemes (Section 3.2): N code streams of b bits on one grid in, one stream out.
struct ServerArgs {
  const uint32_t* codes;   // N streams, stream i at codes + i * stride_words, segment layout `segs`
  int64_t stride_words;
  int N;
  int b;
  int b_out;               // scheme (b): b + ceil(log2 N), index sums; scheme (c): b, re-quantized average
  int requantize;
  uint64_t seed;
  uint64_t k;
  const SegInfo* segs;     // layout of the input streams (width b)
  const SegInfo* segs_out; // layout of the output stream (width b_out): same segments and tiles, other word offsets
  const int32_t* tile_seg;
  int nseg;
  int ntiles;
  uint32_t* out;
};
cudaError_t launch_server_reduce(const ServerArgs& a, cudaStream_t st);

// Histogram of the code values of every (worker, segment) message: hist[(worker * nseg + seg) * 2^b + code].
struct HistArgs {
  const uint32_t* codes;
  int64_t stride_words;
  int N;
  int b;                   // 1..8
  const SegInfo* segs;
  const int32_t* tile_seg;
  int nseg;
  int ntiles;
  unsigned long long* hist;  // N * nseg * 2^b counts, added to (the caller clears them)
};
cudaError_t launch_code_histogram(const HistArgs& a, cudaStream_t st);

}  // namespace lpc

namespace lpc {
cudaError_t launch_stream_blocks(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block0,
                                 int64_t count, uint32_t* out, cudaStream_t st);
}  // namespace lpc
