// lpc_quantize_pack_static: the quantize+pack call for callers that must not allocate device memory.
//
// lpc_quantize_pack keeps its working memory (per-tile partial maxima and sums, one scale record per
// worker, a one-entry segment table) in buffers that its context obtains from cudaMalloc.  Some callers
// cannot do that: code that runs inside a region where the allocator is off limits (a real-time loop
// that must not take the allocator's locks or trigger an implicit device synchronisation, a plug-in that
// is handed a fixed memory budget by its host application, a process whose memory pool is already
// carved up).  For them the same kernels run here with that working memory placed in one fixed array
// that is part of the library image.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/lpc.h"
#include "lpc_kernels.h"

namespace {

using namespace lpc;

// Layout of the fixed working memory (bytes from the start of the array):
//   [0, 64)                      one SegInfo (the vector as a single segment)
//   [64, 128)                    status word: the kernels need a place to flag non-finite input; nothing reads it back
//                                (there is no context to report through), the caller's signal is the NaN delta
//   [256, 256 + 32*MAX_N)        ScaleRec per worker
//   then three arrays of MAX_PARTS 32-bit entries: tile maxima, tile sums, tile sums of squares
constexpr int MAX_N = LPC_STATIC_MAX_WORKERS;
constexpr int MAX_PARTS = LPC_STATIC_MAX_TILES;  // workers x tiles of 8192 coordinates
constexpr size_t OFF_SEG = 0, OFF_STATUS = 64, OFF_SCALES = 256;
constexpr size_t OFF_PMAX = OFF_SCALES + sizeof(ScaleRec) * MAX_N;
constexpr size_t OFF_PS1 = OFF_PMAX + 4 * (size_t)MAX_PARTS;
constexpr size_t OFF_PS2 = OFF_PS1 + 4 * (size_t)MAX_PARTS;
constexpr size_t SCRATCH_BYTES = OFF_PS2 + 4 * (size_t)MAX_PARTS;

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SCRATCH_BYTES];

// Writes the segment record and clears the status word.  Device code may name the array directly.
__global__ void static_setup_kernel(SegInfo seg) {
  *reinterpret_cast<SegInfo*>(g_static_scratch + OFF_SEG) = seg;
  *reinterpret_cast<unsigned int*>(g_static_scratch + OFF_STATUS) = 0u;
}

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the address
// is asked for once per device, with that device current.
std::mutex g_mu;
unsigned char* g_dev_ptr[64] = {nullptr};

int scratch_address(unsigned char** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LPC_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_dev_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return LPC_ERR_CUDA;
    }
    g_dev_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_dev_ptr[dev];
  return LPC_OK;
}

}  // namespace

extern "C" int lpc_quantize_pack_static(const float* U, int64_t len, int64_t ld, int32_t N, int32_t b, int clip_mode,
                                        float clip_value, uint64_t seed, uint64_t k, uint32_t* codes_out,
                                        float* delta_out, uint32_t* clipped_out, void* stream) {
  if (!U || !codes_out || !delta_out || !clipped_out) return LPC_ERR_INVALID_ARG;
  if (len < 1 || ld < len || N < 1) return LPC_ERR_INVALID_ARG;
  if (!((b >= 1 && b <= 16) || b == 32)) return LPC_ERR_INVALID_ARG;
  if (clip_mode < LPC_CLIP_NONE || clip_mode > LPC_CLIP_STD) return LPC_ERR_INVALID_ARG;
  if (clip_mode == LPC_CLIP_LAMBDA && !(clip_value > 0.f && clip_value <= 1.f)) return LPC_ERR_INVALID_ARG;
  if (clip_mode == LPC_CLIP_STD && !(clip_value > 0.f)) return LPC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(codes_out) & 15u) != 0) return LPC_ERR_INVALID_ARG;
  const int64_t ntiles = (len + TILE - 1) / TILE;
  // the fixed working memory bounds the problem size: refuse anything larger, loudly
  if (N > MAX_N || ntiles * N > MAX_PARTS || (len + 7) / 8 > 0xFFFFFFFFll) return LPC_ERR_UNSUPPORTED;

  unsigned char* base = nullptr;
  const int rc = scratch_address(&base);
  if (rc != LPC_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

  SegInfo seg;
  seg.off = 0; seg.len = len; seg.word_off = 0;
  seg.pad_words = (((len * b + 31) / 32) + 3) & ~(int64_t)3;
  seg.block_base = 0; seg.tile_first = 0; seg.tile_count = (int32_t)ntiles; seg.pad_ = 0;
  static_setup_kernel<<<1, 1, 0, st>>>(seg);
  if (cudaGetLastError() != cudaSuccess) return LPC_ERR_CUDA;

  QuantArgs a;
  a.U = U; a.U_sub = nullptr; a.ld = ld; a.N = N; a.b = b; a.clip_mode = clip_mode; a.clip_value = clip_value;
  a.seed = seed; a.k = k;
  a.segs = reinterpret_cast<const SegInfo*>(base + OFF_SEG);
  a.tile_seg = nullptr; a.nseg = 1; a.ntiles = (int)ntiles;
  a.pmax = reinterpret_cast<uint32_t*>(base + OFF_PMAX);
  a.ps1 = reinterpret_cast<float*>(base + OFF_PS1);
  a.ps2 = reinterpret_cast<float*>(base + OFF_PS2);
  a.scales = reinterpret_cast<ScaleRec*>(base + OFF_SCALES);
  a.codes = codes_out; a.stride_words = seg.pad_words;
  a.delta_out = delta_out; a.clipped_out = clipped_out; a.count_clipped = 1; a.shared_scale = 0;
  a.dev_status = reinterpret_cast<unsigned int*>(base + OFF_STATUS);
  return launch_quantize_pack(a, st) == cudaSuccess ? LPC_OK : LPC_ERR_CUDA;
}
