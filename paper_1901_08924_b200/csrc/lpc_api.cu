// C ABI of the library (declared in include/lpc.h): argument checks, the context with its device
// scratch, launch orchestration, CUDA-graph replay of the inner loop, and the counted communication
// bits.  All arithmetic of the method runs in the kernels of the other files.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <queue>
#include <functional>
#include <cmath>
#include <vector>

#include "../../include/lpc.h"
#include "lpc_inner.h"
#include "lpc_kernels.h"
#include "lpc_snapshot.h"
#include "lpc_status.h"

namespace {

using namespace lpc;

struct SegPlan {
  int64_t len = -1;
  int b = 0;
  int nseg = 0;
  int ntiles = 0;
  int64_t stride_words = 0;
  std::vector<int64_t> offsets;     // nseg + 1
  std::vector<SegInfo> segs;        // host copy
  std::vector<int32_t> tile_seg;    // host copy
  SegInfo* d_segs = nullptr;
  int32_t* d_tile_seg = nullptr;    // nullptr when nseg == 1
  uint64_t msg_bits = 0;            // sum over segments of 32 + b*len_s
  uint64_t version = 0;             // changes whenever the tables are rebuilt
};

struct GraphKey {
  int kind = -1;  // 0 LPC, 1 ALPC
  int steps = 0;
  float p[5] = {0, 0, 0, 0, 0};
  int tap = 0, cs = 0, sample_global = 0;
  bool operator==(const GraphKey& o) const {
    return kind == o.kind && steps == o.steps && std::memcmp(p, o.p, sizeof(p)) == 0 && tap == o.tap && cs == o.cs &&
           sample_global == o.sample_global;
  }
};

}  // namespace

struct lpc_ctx {
  // problem
  const float* X = nullptr;
  const float* y = nullptr;
  int64_t n = 0;
  int d = 0, loss = 0;
  float lambda_l1 = 0.f;
  int N = 1, B = 1, b = 4, clip_mode = 0;
  float clip_value = 1.f;
  uint64_t seed = 0;
  cudaStream_t stream = nullptr;
  // options
  int sample_global = 0, tap_u = 0, want_cs = 0, use_graph = 1, use_persist = 1;
  // device state of the linear-model path
  float *x = nullptr, *xt = nullptr, *mu = nullptr, *margins = nullptr;
  float *yv = nullptr, *zv = nullptr, *ysum = nullptr, *vhat = nullptr, *v_tap = nullptr, *u_tap = nullptr;
  uint32_t* codes = nullptr;
  float* delta = nullptr;
  uint32_t *clipped_part = nullptr, *clipped = nullptr;
  int64_t* idx_tap = nullptr;
  float* coef_tap = nullptr;
  uint64_t* k_dev = nullptr;
  unsigned int* dev_status = nullptr;
  double* f_dev = nullptr;  // [0] = f, [1] = ||x||_1, [2] = ||x||^2
  // snapshot pass
  int snapR = 1, snapStages = 1, snapGrid = 1, dpad = 0;
  size_t snapSmem = 0;
  float* partial_mu = nullptr;
  double* partial_f = nullptr;
  // fused inner kernel
  bool inner_ok = false;
  int CS = 1, SL = 0;
  size_t innerSmem = 0;
  int innerStages = 0;  // 0: minibatch rows resident in shared memory; > 0: streamed through that many stages
  SegPlan inner_seg;  // one segment of length d for the aggregator
  // persistent inner loop
  bool persist_ok = false, apersist_ok = false;  // Algorithm 1 loop / Algorithm 2 loop
  int pCS = 1, pSL = 0, pSlots = 0, aCS = 1, aSL = 0, aSlots = 0;  // cluster size, slice, row slots of the two loops
  size_t persistSmem = 0, apersistSmem = 0;
  // exchange buffers of the one-launch loops: tagged 64-bit words (payload | tag << 32), two step-parity halves
  unsigned long long* flags = nullptr;    // scale words: 2 x 256, 128 bytes apart, + 1 abort word
  unsigned long long* ll = nullptr;       // code words: 2 x N x dpow2/8 groups x ll_wpg
  unsigned long long* ll_vhat = nullptr;  // second estimator of Algorithm 2: 2 x dpow2
  int ll_wpg = 1;                         // words per group of 8 coordinates
  uint32_t ll_tag = 0;                    // tags handed out so far; the buffers start zeroed and tag 0 is never used
  int64_t persist_launches = 0;
  // stand-alone quantizer
  SegPlan seg;
  SegPlan seg_out;       // layout of the server's output stream (schemes (b), (c))
  int shared_scale = 0;  // LPC_OPT_SHARED_SCALE
  float sigma = 0.f;     // strong convexity of h (lpc_set_strong_convexity); 0: general convex case
  float sc_w = 1.f;      // snapshot weight of the next ALPC step, (1 + alpha*sigma)^t in fp32
  float sc_wsum = 0.f;   // sum of the weights used so far in this epoch
  int divisor = 0;       // LPC_OPT_AVERAGE_DIVISOR; 0: the worker count N
  int last_split = 0;    // CTAs per tile of the last lpc_unpack_average_prox launch
  int64_t last_pipelined_runs = 0;  // runs of whole tiles per worker in the last lpc_quantize_pack launch
  uint32_t* q_pmax = nullptr;
  float *q_ps1 = nullptr, *q_ps2 = nullptr;
  size_t q_part_cap = 0;
  ScaleRec* q_scales = nullptr;
  uint32_t* q_clip = nullptr;
  size_t q_scale_cap = 0;
  // one-launch quantizer: arrival counters per (worker, segment), valid for one layout; calls made with it so far
  int loop_cooperative = 1;       // LPC_OPT_LOOP_COOPERATIVE
  int one_launch = 1;             // LPC_OPT_ONE_LAUNCH_QUANTIZE
  unsigned int* q_done = nullptr;
  uint64_t q_done_version = ~0ull;
  unsigned int q_epoch = 0;
  int last_one_launch = 0;
  // graph replay
  cudaGraphExec_t graph = nullptr;
  cudaStream_t cap_stream = nullptr;  // used only to capture the graph
  GraphKey graph_key;
  // per-kernel timing (LPC_OPT_PROFILE): event pairs recorded around launches, resolved on demand
  int profile = 0;
  std::vector<cudaEvent_t> ev_pool;   // 2 events per timed launch
  std::vector<int> ev_kind;
  size_t ev_used = 0;                 // timed launches recorded and not yet resolved
  double prof_ms[LPC_KERNEL_KINDS] = {0};
  int64_t prof_n[LPC_KERNEL_KINDS] = {0};
  // accounting
  uint64_t step1_bits = 0, step2_bits = 0;
  int sm_count = 148, max_smem = 227 * 1024;
  std::string err;
};

namespace {

int fail(lpc_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  return code;
}

#define CU(ctx, expr)                                                                      \
  do {                                                                                     \
    cudaError_t e_ = (expr);                                                               \
    if (e_ != cudaSuccess)                                                                 \
      return fail(ctx, LPC_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e_));  \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
int64_t roundup4(int64_t v) { return (v + 3) & ~(int64_t)3; }
bool valid_b(int b) { return (b >= 1 && b <= 16) || b == 32; }

__global__ void set_u64_kernel(uint64_t* p, uint64_t v) { *p = v; }

void free_plan(SegPlan& p) {
  if (p.d_segs) cudaFree(p.d_segs);
  if (p.d_tile_seg) cudaFree(p.d_tile_seg);
  p = SegPlan();
}

// Host-side layout of a segmented vector.  Returns an LPC status.
int layout(int64_t len, int b, const int64_t* seg_offsets, int nseg, std::vector<SegInfo>& segs,
           std::vector<int32_t>& tile_seg, int64_t* stride_words, uint64_t* msg_bits) {
  if (len < 0 || !valid_b(b) || nseg < 1) return LPC_ERR_INVALID_ARG;
  std::vector<int64_t> offs;
  if (seg_offsets) {
    offs.assign(seg_offsets, seg_offsets + nseg + 1);
    if (offs[0] != 0 || offs[nseg] != len) return LPC_ERR_INVALID_ARG;
    for (int s = 0; s < nseg; ++s)
      if (offs[s + 1] < offs[s]) return LPC_ERR_INVALID_ARG;
  } else {
    if (nseg != 1) return LPC_ERR_INVALID_ARG;
    offs = {0, len};
  }
  segs.resize(nseg);
  tile_seg.clear();
  int64_t word = 0, block = 0, tiles = 0;
  uint64_t bits = 0;
  for (int s = 0; s < nseg; ++s) {
    SegInfo& g = segs[s];
    g.off = offs[s];
    g.len = offs[s + 1] - offs[s];
    g.word_off = word;
    g.pad_words = roundup4((g.len * b + 31) / 32);
    if (block > 0xFFFFFFFFll) return LPC_ERR_UNSUPPORTED;
    g.block_base = (uint32_t)block;
    g.tile_first = (int32_t)tiles;
    const int64_t tc = (g.len + TILE - 1) / TILE;
    g.tile_count = (int32_t)tc;
    g.pad_ = 0;
    word += g.pad_words;
    block += (g.len + 7) / 8;
    tiles += tc;
    if (tiles > 0x7FFFFFFFll) return LPC_ERR_UNSUPPORTED;
    for (int64_t t = 0; t < tc; ++t) tile_seg.push_back(s);
    bits += 32ull + (uint64_t)b * (uint64_t)g.len;
  }
  if (block > 0x100000000ll) return LPC_ERR_UNSUPPORTED;
  *stride_words = word;
  if (msg_bits) *msg_bits = bits;
  return LPC_OK;
}

int make_plan(lpc_ctx* c, SegPlan& p, int64_t len, int b, const int64_t* seg_offsets, int nseg) {
  // reuse when the request matches the cached plan
  if (p.len == len && p.b == b && p.nseg == nseg) {
    bool same = true;
    if (seg_offsets)
      for (int s = 0; s <= nseg && same; ++s) same = (p.offsets[s] == seg_offsets[s]);
    if (same) return LPC_OK;
  }
  std::vector<SegInfo> segs;
  std::vector<int32_t> tile_seg;
  int64_t stride = 0;
  uint64_t bits = 0;
  const int rc = layout(len, b, seg_offsets, nseg, segs, tile_seg, &stride, &bits);
  if (rc != LPC_OK) return fail(c, rc, "invalid segment layout");
  CU(c, cudaStreamSynchronize(c->stream));  // the old tables may still be in use
  const uint64_t version = p.version + 1;
  free_plan(p);
  p.version = version;
  p.len = len; p.b = b; p.nseg = nseg; p.stride_words = stride; p.msg_bits = bits;
  p.ntiles = (int)tile_seg.size();
  p.offsets.resize(nseg + 1);
  for (int s = 0; s < nseg; ++s) p.offsets[s] = segs[s].off;
  p.offsets[nseg] = len;
  p.segs = segs;
  p.tile_seg = tile_seg;
  CU(c, cudaMalloc(&p.d_segs, sizeof(SegInfo) * nseg));
  CU(c, cudaMemcpyAsync(p.d_segs, p.segs.data(), sizeof(SegInfo) * nseg, cudaMemcpyHostToDevice, c->stream));
  if (nseg > 1 && p.ntiles > 0) {
    CU(c, cudaMalloc(&p.d_tile_seg, sizeof(int32_t) * p.ntiles));
    CU(c, cudaMemcpyAsync(p.d_tile_seg, p.tile_seg.data(), sizeof(int32_t) * p.ntiles, cudaMemcpyHostToDevice, c->stream));
  }
  CU(c, cudaStreamSynchronize(c->stream));  // the host vectors are pageable: finish the copies now
  return LPC_OK;
}

template <class T>
int dalloc(lpc_ctx* c, T** p, size_t count) {
  CU(c, cudaMalloc(reinterpret_cast<void**>(p), sizeof(T) * (count ? count : 1)));
  CU(c, cudaMemsetAsync(*p, 0, sizeof(T) * (count ? count : 1), c->stream));
  return LPC_OK;
}

#define TRY(expr)             \
  do {                        \
    const int rc_ = (expr);   \
    if (rc_ != LPC_OK) return rc_; \
  } while (0)

bool has_model(const lpc_ctx* c) { return c->X != nullptr; }

// ---- per-kernel timing ------------------------------------------------------------------------------
int prof_resolve(lpc_ctx* c) {
  if (c->ev_used == 0) return LPC_OK;
  CU(c, cudaStreamSynchronize(c->stream));
  for (size_t i = 0; i < c->ev_used; ++i) {
    float ms = 0.f;
    CU(c, cudaEventElapsedTime(&ms, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
    c->prof_ms[c->ev_kind[i]] += (double)ms;
    c->prof_n[c->ev_kind[i]] += 1;
  }
  c->ev_used = 0;
  return LPC_OK;
}

struct ProfScope {  // records an event before and after one launch when profiling is on
  lpc_ctx* c;
  cudaEvent_t stop = nullptr;
  ProfScope(lpc_ctx* ctx, int kind) : c(ctx) {
    if (!c->profile) return;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(c->stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) return;
    if (c->ev_used >= 32768) prof_resolve(c);
    if (c->ev_pool.size() < 2 * (c->ev_used + 1)) {
      cudaEvent_t a = nullptr, b = nullptr;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
      c->ev_pool.push_back(a);
      c->ev_pool.push_back(b);
      c->ev_kind.push_back(kind);
    }
    c->ev_kind[c->ev_used] = kind;
    cudaEventRecord(c->ev_pool[2 * c->ev_used], c->stream);
    stop = c->ev_pool[2 * c->ev_used + 1];
    c->ev_used += 1;
  }
  ~ProfScope() {
    if (stop) cudaEventRecord(stop, c->stream);
  }
};

void prof_hook(void* user, int kind, int begin) {
  // used by launch functions that issue several kernels: begin = 1 opens a scope, 0 closes it
  static thread_local ProfScope* open = nullptr;
  lpc_ctx* c = static_cast<lpc_ctx*>(user);
  if (begin) {
    open = new ProfScope(c, kind);
  } else if (open) {
    delete open;
    open = nullptr;
  }
}

InnerArgs inner_args(lpc_ctx* c, uint64_t k_base, const uint64_t* k_dev, int has_J) {
  InnerArgs a;
  a.X = c->X; a.y = c->y; a.n = c->n; a.d = c->d; a.loss = c->loss;
  a.N = c->N; a.B = c->B; a.b = c->b; a.clip_mode = c->clip_mode; a.clip_value = c->clip_value;
  a.seed = c->seed; a.sample_global = c->sample_global;
  a.k_base = k_base; a.k_dev = k_dev;
  a.x = c->x; a.margins = c->margins; a.mu = c->mu; a.has_J = has_J; a.vhat = c->vhat;
  a.codes = c->codes; a.stride_words = c->inner_seg.stride_words; a.pad_words = c->inner_seg.stride_words;
  a.delta = c->delta; a.clipped_part = c->clipped_part;
  a.idx_tap = c->idx_tap; a.coef_tap = c->coef_tap; a.u_tap = c->tap_u ? c->u_tap : nullptr;
  a.dev_status = c->dev_status; a.CS = c->CS; a.SL = c->SL; a.stream_stages = c->innerStages;
  return a;
}

// divisor: the count the decoded sum is divided by (Eq. 3: the worker count N).
AggArgs agg_args(lpc_ctx* c, const SegPlan& p, const uint32_t* codes, const float* delta, const float* mu, float* x,
                 float eta, float lambda_l1, float* v_out, int divisor) {
  AggArgs a;
  a.codes = codes; a.stride_words = p.stride_words; a.delta = delta; a.N = c->N; a.b = c->b;
  a.divisor = divisor;
  a.split = aggregate_split(p.ntiles, c->sm_count);
  a.segs = p.d_segs; a.tile_seg = p.d_tile_seg; a.nseg = p.nseg; a.ntiles = p.ntiles;
  a.mu = mu; a.x = x; a.eta = eta; a.lambda_l1 = lambda_l1; a.v_out = v_out; a.k_counter = nullptr;
  a.mode = 0; a.y = nullptr; a.z = nullptr; a.ysum = nullptr; a.vhat = nullptr; a.alpha = 0.f; a.inv4L = 0.f;
  a.cy = 1.f; a.cz = 1.f; a.wy = 1.f;
  return a;
}

int replan_inner(lpc_ctx* c) {
  size_t smem = 0;
  int cs = 1, sl = 0;
  int stages = 0;
  c->inner_ok = inner_plan(c->d, c->B, c->want_cs, c->max_smem, &cs, &sl, &smem, &stages);
  if (c->inner_ok) { c->CS = cs; c->SL = sl; c->innerSmem = smem; c->innerStages = stages; }
  int slots = 0;
  c->persist_ok = persist_plan(c->d, c->N, c->B, c->b, 0, c->want_cs, c->max_smem, &cs, &sl, &smem, &slots);
  if (c->persist_ok) { c->pCS = cs; c->pSL = sl; c->persistSmem = smem; c->pSlots = slots; }
  c->apersist_ok = persist_plan(c->d, c->N, c->B, c->b, 1, c->want_cs, c->max_smem, &cs, &sl, &smem, &slots);
  if (c->apersist_ok) { c->aCS = cs; c->aSL = sl; c->apersistSmem = smem; c->aSlots = slots; }
  return LPC_OK;
}

// One LPC inner step enqueued on the stream (Algorithm 1 steps 6-10).
int enqueue_lpc_step(lpc_ctx* c, float eta, uint64_t k_base, const uint64_t* k_dev, uint64_t* k_counter) {
  InnerArgs ia = inner_args(c, k_base, k_dev, 0);
  { ProfScope ps_(c, LPC_KERNEL_WORKER); CU(c, launch_inner(ia, c->innerSmem, c->stream)); }
  // the training loops always average over the context's N workers (Eq. 3); LPC_OPT_AVERAGE_DIVISOR does not apply
  AggArgs ag = agg_args(c, c->inner_seg, c->codes, c->delta, c->mu, c->x, eta, c->lambda_l1, c->tap_u ? c->v_tap : nullptr, c->N);
  ag.k_counter = k_counter;
  { ProfScope ps_(c, LPC_KERNEL_AGGREGATE); CU(c, launch_unpack_average_prox(ag, c->stream)); }
  return LPC_OK;
}

// One ALPC step enqueued on the stream (Algorithm 2 steps 6-13).
int enqueue_alpc_step(lpc_ctx* c, float tau1, float tau2, float alpha, float inv4L, uint64_t k_base,
                      const uint64_t* k_dev, uint64_t* k_counter) {
  { ProfScope ps_(c, LPC_KERNEL_OTHER); CU(c, launch_coupling(c->zv, c->xt, c->yv, tau1, tau2, c->d, c->x, c->stream)); }
  InnerArgs ia = inner_args(c, k_base, k_dev, 1);
  { ProfScope ps_(c, LPC_KERNEL_WORKER); CU(c, launch_inner(ia, c->innerSmem, c->stream)); }
  AggArgs ag = agg_args(c, c->inner_seg, c->codes, c->delta, c->mu, c->x, 0.f, c->lambda_l1, c->tap_u ? c->v_tap : nullptr, c->N);
  ag.k_counter = k_counter;
  ag.mode = 1; ag.y = c->yv; ag.z = c->zv; ag.ysum = c->ysum; ag.vhat = c->vhat; ag.alpha = alpha; ag.inv4L = inv4L;
  if (c->sigma > 0.f) {  // each product and sum below is one fp32 operation, as on the device
    volatile float t1 = c->sigma * inv4L, t2 = alpha * c->sigma;
    volatile float d1 = 1.0f + t1, d2 = 1.0f + t2;
    ag.cy = 1.0f / d1; ag.cz = 1.0f / d2; ag.wy = c->sc_w;
  }
  { ProfScope ps_(c, LPC_KERNEL_AGGREGATE); CU(c, launch_unpack_average_prox(ag, c->stream)); }
  if (c->sigma > 0.f) {  // the weight of the next step and the sum of those used (Algorithm 2's last step)
    volatile float t2 = alpha * c->sigma;
    volatile float theta = 1.0f + t2;
    volatile float ws = c->sc_wsum + c->sc_w, wn = c->sc_w * theta;
    c->sc_wsum = ws; c->sc_w = wn;
  }
  return LPC_OK;
}

constexpr int GRAPH_STEPS = 128;  // inner steps per captured graph

int run_steps(lpc_ctx* c, int kind, const float* p, uint64_t k0, int64_t count) {
  if (count < 0) return fail(c, LPC_ERR_INVALID_ARG, "count < 0");
  if (!has_model(c) || !c->inner_ok) return fail(c, LPC_ERR_UNSUPPORTED, "no linear model or d too large for the fused step");
  auto one = [&](uint64_t kb, const uint64_t* kd, uint64_t* kc) {
    return kind == 0 ? enqueue_lpc_step(c, p[0], kb, kd, kc) : enqueue_alpc_step(c, p[0], p[1], p[2], p[3], kb, kd, kc);
  };
  int64_t done = 0;
  const bool loop_ok = (kind == 0) ? c->persist_ok : c->apersist_ok;
  // the strongly convex ALPC step carries a weight that changes from step to step: plain per-step launches
  const bool weighted = (kind == 1 && c->sigma > 0.f);
  if (c->use_persist && loop_ok && count >= 2 && count <= 0x7FFFFFFF) {
    // the whole loop in one cooperative launch; on a launch refusal fall through to the per-step kernels
    PersistArgs pa;
    pa.in = inner_args(c, k0, nullptr, 0);
    pa.in.CS = kind == 0 ? c->pCS : c->aCS;
    pa.in.SL = kind == 0 ? c->pSL : c->aSL;
    pa.row_slots = kind == 0 ? c->pSlots : c->aSlots;
    pa.count = (int)count; pa.eta = kind == 0 ? p[0] : 0.f; pa.lambda_l1 = c->lambda_l1;
    pa.pub = c->flags; pa.abort_flag = reinterpret_cast<unsigned int*>(c->flags + 512 * 16); pa.x_out = c->x;
    pa.ll = c->ll; pa.ll_vhat = c->ll_vhat; pa.wpg = c->ll_wpg;
    if ((uint64_t)c->ll_tag + (uint64_t)count >= 0xFFFFFFF0ull) {  // tags would wrap: start over from cleared buffers
      int dp = 32;
      while (dp < c->d) dp <<= 1;
      CU(c, cudaMemsetAsync(c->flags, 0, (512 * 16 + 1) * sizeof(unsigned long long), c->stream));
      CU(c, cudaMemsetAsync(c->ll, 0, sizeof(unsigned long long) * 2 * (size_t)c->N * (size_t)(dp / 8) * c->ll_wpg, c->stream));
      CU(c, cudaMemsetAsync(c->ll_vhat, 0, sizeof(unsigned long long) * 2 * (size_t)dp, c->stream));
      c->ll_tag = 0;
    }
    pa.tag_base = c->ll_tag;
    pa.v_tap = c->tap_u ? c->v_tap : nullptr;
    pa.alpc = kind; pa.tau1 = p[0]; pa.tau2 = p[1]; pa.alpha = p[2]; pa.inv4L = p[3];
    pa.y = c->yv; pa.z = c->zv; pa.ysum = c->ysum; pa.xt = c->xt; pa.vhat = c->vhat;
    pa.cy = 1.f; pa.cz = 1.f; pa.w0 = 1.f; pa.theta = 1.f;
    if (weighted) {  // each product and sum is one fp32 operation, as on the device
      volatile float t1 = c->sigma * p[3], t2 = p[2] * c->sigma;
      volatile float d1 = 1.0f + t1, d2 = 1.0f + t2;
      pa.cy = 1.0f / d1; pa.cz = 1.0f / d2; pa.w0 = c->sc_w; pa.theta = d2;
    }
    CU(c, cudaMemsetAsync(pa.abort_flag, 0, sizeof(unsigned long long), c->stream));
    cudaError_t e;
    { ProfScope ps_(c, LPC_KERNEL_INNER_LOOP); e = launch_persist(pa, kind == 0 ? c->persistSmem : c->apersistSmem, c->stream, c->loop_cooperative != 0); }
    if (e == cudaSuccess) {
      done = count;
      if (weighted) {  // the weights the loop went through, and the one the next step starts from
        for (int64_t i = 0; i < count; ++i) {
          volatile float ws = c->sc_wsum + c->sc_w, wn = c->sc_w * pa.theta;
          c->sc_wsum = ws; c->sc_w = wn;
        }
      }
      c->persist_launches += 1;
      c->ll_tag += (uint32_t)count;
    } else {
      cudaGetLastError();  // clear the refusal and use the per-step path
      if (kind == 0) c->persist_ok = false; else c->apersist_ok = false;
    }
  }
  if (done < count && c->use_graph && !c->profile && !weighted && count >= GRAPH_STEPS) {
    GraphKey key;
    key.kind = kind; key.steps = GRAPH_STEPS; key.tap = c->tap_u; key.cs = c->CS; key.sample_global = c->sample_global;
    for (int i = 0; i < 4; ++i) key.p[i] = p[i];
    if (!c->graph || !(c->graph_key == key)) {
      if (c->graph) { cudaGraphExecDestroy(c->graph); c->graph = nullptr; }
      cudaGraph_t g = nullptr;
      // Capture on a stream of our own: the caller's stream may be the legacy default stream, which
      // cannot be captured.  Nothing runs during capture; the graph is launched on the caller's stream.
      if (!c->cap_stream) CU(c, cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking));
      cudaStream_t user = c->stream;
      CU(c, cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal));
      c->stream = c->cap_stream;
      int rc = LPC_OK;
      for (int i = 0; i < GRAPH_STEPS && rc == LPC_OK; ++i) rc = one(0, c->k_dev, c->k_dev);
      c->stream = user;
      cudaError_t e = cudaStreamEndCapture(c->cap_stream, &g);
      if (rc != LPC_OK) { if (g) cudaGraphDestroy(g); return rc; }
      CU(c, e);
      e = cudaGraphInstantiate(&c->graph, g, 0);
      cudaGraphDestroy(g);
      CU(c, e);
      c->graph_key = key;
    }
    set_u64_kernel<<<1, 1, 0, c->stream>>>(c->k_dev, k0);
    CU(c, cudaGetLastError());
    while (count - done >= GRAPH_STEPS) {
      CU(c, cudaGraphLaunch(c->graph, c->stream));
      done += GRAPH_STEPS;
    }
  }
  for (; done < count; ++done) TRY(one(k0 + (uint64_t)done, nullptr, nullptr));
  const uint64_t per_step = (32ull + (uint64_t)c->b * (uint64_t)c->d) * (uint64_t)c->N * (uint64_t)(c->N - 1);
  c->step2_bits += per_step * (uint64_t)count;
  return LPC_OK;
}

int buffer_of(lpc_ctx* c, int which, void** ptr, size_t* bytes) {
  const size_t d = (size_t)c->d, N = (size_t)c->N, B = (size_t)c->B;
  switch (which) {
    case LPC_BUF_X: *ptr = c->x; *bytes = d * 4; break;
    case LPC_BUF_XTILDE: *ptr = c->xt; *bytes = d * 4; break;
    case LPC_BUF_MU: *ptr = c->mu; *bytes = d * 4; break;
    case LPC_BUF_MARGINS: *ptr = c->margins; *bytes = (size_t)c->n * 4; break;
    case LPC_BUF_Y: *ptr = c->yv; *bytes = d * 4; break;
    case LPC_BUF_Z: *ptr = c->zv; *bytes = d * 4; break;
    case LPC_BUF_YSUM: *ptr = c->ysum; *bytes = d * 4; break;
    case LPC_BUF_CODES: *ptr = c->codes; *bytes = N * (size_t)c->inner_seg.stride_words * 4; break;
    case LPC_BUF_DELTA: *ptr = c->delta; *bytes = N * 4; break;
    case LPC_BUF_CLIPPED: *ptr = c->clipped; *bytes = N * 4; break;
    case LPC_BUF_BATCH_IDX: *ptr = c->idx_tap; *bytes = (N + 1) * B * 8; break;
    case LPC_BUF_COEF: *ptr = c->coef_tap; *bytes = (N + 1) * B * 4; break;
    case LPC_BUF_U: *ptr = c->u_tap; *bytes = N * d * 4; break;
    case LPC_BUF_V: *ptr = c->v_tap; *bytes = d * 4; break;
    case LPC_BUF_VHAT: *ptr = c->vhat; *bytes = d * 4; break;
    default: return LPC_ERR_INVALID_ARG;
  }
  return (*ptr) ? LPC_OK : LPC_ERR_UNSUPPORTED;
}

int snapshot_pass(lpc_ctx* c, const float* point, bool grad, float* margins_out) {
  SnapArgs a;
  a.X = c->X; a.y = c->y; a.x = point; a.n = c->n; a.d = c->d; a.loss = c->loss;
  a.R = c->snapR; a.nstage = c->snapStages; a.ntiles = (c->n + c->snapR - 1) / c->snapR;
  a.partial_mu = grad ? c->partial_mu : nullptr;
  a.margins_out = margins_out;
  a.partial_f = c->partial_f;
  a.dev_status = c->dev_status;
  const int grid = (int)std::min<int64_t>(c->snapGrid, std::max<int64_t>(a.ntiles, 1));
  { ProfScope ps_(c, LPC_KERNEL_SNAPSHOT); CU(c, launch_snapshot(a, grid, c->snapSmem, c->stream)); }
  CU(c, launch_snapshot_reduce(a.partial_mu, c->partial_f, grid, c->dpad, c->d, c->n, c->mu, nullptr, &c->f_dev[0], c->stream));
  return LPC_OK;
}

}  // namespace

extern "C" {

int lpc_packed_words(int64_t len, int32_t b, int64_t* words_out) {
  if (len < 0 || !valid_b(b) || !words_out) return LPC_ERR_INVALID_ARG;
  *words_out = (len * b + 31) / 32;
  return LPC_OK;
}

int lpc_packed_layout(int64_t len, int32_t b, const int64_t* seg_offsets, int32_t nseg, int64_t* word_offsets_out,
                      int64_t* stride_words_out) {
  std::vector<SegInfo> segs;
  std::vector<int32_t> tile_seg;
  int64_t stride = 0;
  const int rc = layout(len, b, seg_offsets, nseg, segs, tile_seg, &stride, nullptr);
  if (rc != LPC_OK) return rc;
  if (word_offsets_out) {
    for (int s = 0; s < nseg; ++s) word_offsets_out[s] = segs[s].word_off;
    word_offsets_out[nseg] = stride;
  }
  if (stride_words_out) *stride_words_out = stride;
  return LPC_OK;
}

int lpc_init(lpc_ctx** out, const float* X, const float* y, int64_t n, int32_t d, int loss, float lambda_l1, int32_t N,
             int32_t B, int32_t b, int clip_mode, float clip_value, uint64_t seed, void* stream) {
  if (!out) return LPC_ERR_INVALID_ARG;
  *out = nullptr;
  if (N < 1 || N > 1024 || !valid_b(b)) return LPC_ERR_INVALID_ARG;
  if (clip_mode < LPC_CLIP_NONE || clip_mode > LPC_CLIP_STD) return LPC_ERR_INVALID_ARG;
  if (clip_mode == LPC_CLIP_LAMBDA && !(clip_value > 0.f && clip_value <= 1.f)) return LPC_ERR_INVALID_ARG;
  if (clip_mode == LPC_CLIP_STD && !(clip_value > 0.f) ) return LPC_ERR_INVALID_ARG;
  if (!(lambda_l1 >= 0.f)) return LPC_ERR_INVALID_ARG;
  const bool model = (X != nullptr);
  if (model) {
    if (!y || n < 1 || d < 4 || (d & 3) || d > 16384) return LPC_ERR_INVALID_ARG;
    if (n % N != 0) return LPC_ERR_INVALID_ARG;
    if (B < 1 || B > inner_max_b()) return LPC_ERR_INVALID_ARG;
    if (loss != LPC_LOGISTIC && loss != LPC_LEAST_SQUARES) return LPC_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(y)) return LPC_ERR_INVALID_ARG;
  } else if (n != 0) {
    return LPC_ERR_INVALID_ARG;
  }
  lpc_ctx* c = new lpc_ctx();
  c->X = X; c->y = y; c->n = n; c->d = model ? d : 0; c->loss = loss; c->lambda_l1 = lambda_l1;
  c->N = N; c->B = model ? B : 1; c->b = b; c->clip_mode = clip_mode; c->clip_value = clip_value; c->seed = seed;
  c->stream = reinterpret_cast<cudaStream_t>(stream);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev);
  int optin = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) { delete c; return LPC_ERR_CUDA; }
  c->max_smem = optin - 1024;
  int rc = LPC_OK;
  auto A = [&](int r) { if (rc == LPC_OK) rc = r; };
  A(dalloc(c, &c->dev_status, 1));
  A(dalloc(c, &c->k_dev, 1));
  A(dalloc(c, &c->f_dev, 3));
  if (model && rc == LPC_OK) {
    const size_t dd = (size_t)d;
    A(dalloc(c, &c->x, dd)); A(dalloc(c, &c->xt, dd)); A(dalloc(c, &c->mu, dd)); A(dalloc(c, &c->margins, (size_t)n));
    A(dalloc(c, &c->yv, dd)); A(dalloc(c, &c->zv, dd)); A(dalloc(c, &c->ysum, dd)); A(dalloc(c, &c->vhat, dd));
    A(dalloc(c, &c->v_tap, dd));
    A(dalloc(c, &c->delta, (size_t)N));
    A(dalloc(c, &c->clipped, (size_t)N));
    A(dalloc(c, &c->clipped_part, (size_t)N * inner_clipped_stride()));
    A(dalloc(c, &c->flags, 512 * 16 + 1));
    {
      int dp = 32;
      while (dp < d) dp <<= 1;
      c->ll_wpg = (b <= 4) ? 1 : (b <= 8) ? 2 : (b <= 16) ? 4 : 8;
      A(dalloc(c, &c->ll, 2 * (size_t)N * (size_t)(dp / 8) * c->ll_wpg));
      A(dalloc(c, &c->ll_vhat, 2 * (size_t)dp));
    }
    A(dalloc(c, &c->idx_tap, (size_t)(N + 1) * B)); A(dalloc(c, &c->coef_tap, (size_t)(N + 1) * B));
    if (rc == LPC_OK) rc = make_plan(c, c->inner_seg, d, b, nullptr, 1);
    if (rc == LPC_OK) A(dalloc(c, &c->codes, (size_t)N * (size_t)c->inner_seg.stride_words));
    c->dpad = snapshot_dpad(d);
    snapshot_plan(d, c->max_smem, &c->snapR, &c->snapStages, &c->snapSmem);
    c->snapGrid = c->sm_count;
    A(dalloc(c, &c->partial_mu, (size_t)c->snapGrid * c->dpad));
    A(dalloc(c, &c->partial_f, 2 * (size_t)c->snapGrid));
    replan_inner(c);
  }
  if (rc != LPC_OK) { lpc_destroy(c); return rc; }
  *out = c;
  return LPC_OK;
}

int lpc_destroy(lpc_ctx* c) {
  if (!c) return LPC_OK;
  cudaStreamSynchronize(c->stream);
  if (c->graph) cudaGraphExecDestroy(c->graph);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  void* ptrs[] = {c->x, c->xt, c->mu, c->margins, c->yv, c->zv, c->ysum, c->vhat, c->v_tap, c->u_tap, c->codes,
                  c->delta, c->clipped_part, c->clipped, c->idx_tap, c->coef_tap, c->k_dev, c->dev_status, c->f_dev,
                  c->partial_mu, c->partial_f, c->flags, c->ll, c->ll_vhat, c->q_pmax, c->q_ps1, c->q_ps2, c->q_scales, c->q_clip, c->q_done};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  free_plan(c->inner_seg);
  free_plan(c->seg);
  free_plan(c->seg_out);
  delete c;
  return LPC_OK;
}

const char* lpc_last_error(const lpc_ctx* c) { return c ? c->err.c_str() : "null context"; }

int lpc_set_option(lpc_ctx* c, int option, int64_t value) {
  if (!c) return LPC_ERR_INVALID_ARG;
  switch (option) {
    case LPC_OPT_SAMPLE_GLOBAL: c->sample_global = value ? 1 : 0; return LPC_OK;
    case LPC_OPT_TAP_U:
      if (value && !c->u_tap && has_model(c)) TRY(dalloc(c, &c->u_tap, (size_t)c->N * (size_t)c->d));
      c->tap_u = value ? 1 : 0;
      return LPC_OK;
    case LPC_OPT_CLUSTER_SIZE:
      if (!(value == 0 || value == 1 || value == 2 || value == 4 || value == 8)) return fail(c, LPC_ERR_INVALID_ARG, "cluster size");
      c->want_cs = (int)value;
      if (has_model(c)) {
        replan_inner(c);
        if (!c->inner_ok) { c->want_cs = 0; replan_inner(c); return fail(c, LPC_ERR_UNSUPPORTED, "cluster size does not fit"); }
      }
      return LPC_OK;
    case LPC_OPT_USE_GRAPH: c->use_graph = value ? 1 : 0; return LPC_OK;
    case LPC_OPT_PERSISTENT: c->use_persist = value ? 1 : 0; return LPC_OK;
    case LPC_OPT_ONE_LAUNCH_QUANTIZE: c->one_launch = value ? 1 : 0; return LPC_OK;
    case LPC_OPT_LOOP_COOPERATIVE: c->loop_cooperative = value ? 1 : 0; return LPC_OK;
    case LPC_OPT_SHARED_SCALE:
      if (value && (c->b < 2 || c->b > 16)) return fail(c, LPC_ERR_UNSUPPORTED, "a unified scale needs an integer grid: b in 2..16");
      c->shared_scale = value ? 1 : 0;
      return LPC_OK;
    case LPC_OPT_AVERAGE_DIVISOR:
      if (value < 0 || value > (1 << 20)) return fail(c, LPC_ERR_INVALID_ARG, "divisor");
      c->divisor = (int)value;
      return LPC_OK;
    case LPC_OPT_PROFILE:
      TRY(prof_resolve(c));
      c->profile = value ? 1 : 0;
      return LPC_OK;
    default: return fail(c, LPC_ERR_INVALID_ARG, "unknown option");
  }
}

int lpc_sync_status(lpc_ctx* c) {
  if (!c) return LPC_ERR_INVALID_ARG;
  CU(c, cudaStreamSynchronize(c->stream));
  unsigned int st = 0;
  CU(c, cudaMemcpy(&st, c->dev_status, sizeof(st), cudaMemcpyDeviceToHost));
  if (st) CU(c, cudaMemset(c->dev_status, 0, sizeof(st)));
  if (st & DEV_TIMEOUT) return fail(c, LPC_ERR_TIMEOUT, "a bounded device-side wait ran out");
  if (st & DEV_NONFINITE) return fail(c, LPC_ERR_NONFINITE, "non-finite value reached the quantizer");
  return LPC_OK;
}

int lpc_get_buffer(lpc_ctx* c, int which, void* dst, size_t bytes) {
  if (!c || !dst) return LPC_ERR_INVALID_ARG;
  if (!has_model(c)) return fail(c, LPC_ERR_UNSUPPORTED, "quantizer-only context");
  void* p = nullptr;
  size_t cap = 0;
  if (which == LPC_BUF_CLIPPED) CU(c, launch_clipped_sum(c->clipped_part, c->N, c->clipped, c->stream));
  const int rc = buffer_of(c, which, &p, &cap);
  if (rc != LPC_OK) return fail(c, rc, "buffer not available");
  if (bytes > cap) return fail(c, LPC_ERR_INVALID_ARG, "bytes exceed the buffer");
  CU(c, cudaMemcpyAsync(dst, p, bytes, cudaMemcpyDeviceToDevice, c->stream));
  return LPC_OK;
}

int lpc_set_buffer(lpc_ctx* c, int which, const void* src, size_t bytes) {
  if (!c || !src) return LPC_ERR_INVALID_ARG;
  if (!has_model(c)) return fail(c, LPC_ERR_UNSUPPORTED, "quantizer-only context");
  void* p = nullptr;
  size_t cap = 0;
  const int rc = buffer_of(c, which, &p, &cap);
  if (rc != LPC_OK) return fail(c, rc, "buffer not available");
  if (bytes > cap) return fail(c, LPC_ERR_INVALID_ARG, "bytes exceed the buffer");
  CU(c, cudaMemcpyAsync(p, src, bytes, cudaMemcpyDeviceToDevice, c->stream));
  return LPC_OK;
}

int lpc_set_iterate(lpc_ctx* c, const float* x) { return c ? lpc_set_buffer(c, LPC_BUF_X, x, (size_t)c->d * 4) : LPC_ERR_INVALID_ARG; }
int lpc_get_iterate(lpc_ctx* c, float* x_out) { return c ? lpc_get_buffer(c, LPC_BUF_X, x_out, (size_t)c->d * 4) : LPC_ERR_INVALID_ARG; }

int lpc_snapshot_full_grad(lpc_ctx* c, float* mu_out, double* f_snapshot) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (!has_model(c)) return fail(c, LPC_ERR_UNSUPPORTED, "quantizer-only context");
  CU(c, cudaMemcpyAsync(c->xt, c->x, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
  TRY(snapshot_pass(c, c->xt, true, c->margins));
  if (mu_out) CU(c, cudaMemcpyAsync(mu_out, c->mu, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
  c->step1_bits += 32ull * (uint64_t)c->d * (uint64_t)c->N * (uint64_t)(c->N - 1);
  if (f_snapshot) {
    CU(c, cudaMemcpyAsync(f_snapshot, &c->f_dev[0], sizeof(double), cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
  }
  return LPC_OK;
}

int lpc_inner_step(lpc_ctx* c, float eta, uint64_t k) {
  if (!c) return LPC_ERR_INVALID_ARG;
  const float p[4] = {eta, 0, 0, 0};
  const int saved = c->use_graph;
  c->use_graph = 0;
  const int rc = run_steps(c, 0, p, k, 1);
  c->use_graph = saved;
  return rc;
}

int lpc_inner_steps(lpc_ctx* c, float eta, uint64_t k0, int64_t count) {
  if (!c) return LPC_ERR_INVALID_ARG;
  const float p[4] = {eta, 0, 0, 0};
  return run_steps(c, 0, p, k0, count);
}

int lpc_alpc_begin(lpc_ctx* c) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (!has_model(c)) return fail(c, LPC_ERR_UNSUPPORTED, "quantizer-only context");
  const size_t bytes = (size_t)c->d * 4;
  CU(c, cudaMemcpyAsync(c->yv, c->x, bytes, cudaMemcpyDeviceToDevice, c->stream));
  CU(c, cudaMemcpyAsync(c->zv, c->x, bytes, cudaMemcpyDeviceToDevice, c->stream));
  CU(c, cudaMemsetAsync(c->ysum, 0, bytes, c->stream));
  c->sc_w = 1.f; c->sc_wsum = 0.f;
  return LPC_OK;
}

int lpc_set_strong_convexity(lpc_ctx* c, float sigma) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (!(sigma >= 0.f) || !std::isfinite(sigma)) return fail(c, LPC_ERR_INVALID_ARG, "sigma must be finite and >= 0");
  c->sigma = sigma;
  c->sc_w = 1.f; c->sc_wsum = 0.f;
  return LPC_OK;
}

int lpc_alpc_double_sample_step(lpc_ctx* c, float tau1, float tau2, float alpha, float inv4L, uint64_t k) {
  if (!c) return LPC_ERR_INVALID_ARG;
  const float p[4] = {tau1, tau2, alpha, inv4L};
  const int saved = c->use_graph;
  c->use_graph = 0;
  const int rc = run_steps(c, 1, p, k, 1);
  c->use_graph = saved;
  return rc;
}

int lpc_alpc_double_sample_steps(lpc_ctx* c, float tau1, float tau2, float alpha, float inv4L, uint64_t k0, int64_t count) {
  if (!c) return LPC_ERR_INVALID_ARG;
  const float p[4] = {tau1, tau2, alpha, inv4L};
  return run_steps(c, 1, p, k0, count);
}

int lpc_alpc_end_epoch(lpc_ctx* c, int64_t m) {
  if (!c || m < 1) return LPC_ERR_INVALID_ARG;
  if (!has_model(c)) return fail(c, LPC_ERR_UNSUPPORTED, "quantizer-only context");
  float inv_m = 1.0f / (float)m;  // IEEE division on the host
  if (c->sigma > 0.f) {  // Algorithm 2: the weighted mean; the weights start over with the next epoch
    if (!(c->sc_wsum > 0.f)) return fail(c, LPC_ERR_INVALID_ARG, "no step since the last snapshot");
    inv_m = 1.0f / c->sc_wsum;
    c->sc_w = 1.f; c->sc_wsum = 0.f;
  }
  CU(c, launch_mean_y(c->ysum, inv_m, c->d, c->x, c->stream));
  return LPC_OK;
}

int lpc_objective(lpc_ctx* c, const float* x, double* P_out) {
  if (!c || !P_out) return LPC_ERR_INVALID_ARG;
  if (!has_model(c)) return fail(c, LPC_ERR_UNSUPPORTED, "quantizer-only context");
  const float* pt = x ? x : c->x;
  if (!aligned16(pt)) return fail(c, LPC_ERR_INVALID_ARG, "x must be 16-byte aligned");
  TRY(snapshot_pass(c, pt, false, nullptr));
  CU(c, launch_l1_norm(pt, c->d, &c->f_dev[1], c->stream));
  double h[3] = {0, 0, 0};
  CU(c, cudaMemcpyAsync(h, c->f_dev, sizeof(h), cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  *P_out = h[0] + (double)c->lambda_l1 * h[1] + 0.5 * (double)c->sigma * h[2];
  return LPC_OK;
}

int lpc_query(const lpc_ctx* c, int what, int64_t* out) {
  if (!c || !out) return LPC_ERR_INVALID_ARG;
  switch (what) {
    case LPC_INFO_STEP_CLUSTER_SIZE: *out = c->inner_ok ? c->CS : 0; return LPC_OK;
    case LPC_INFO_LOOP_CLUSTER_SIZE: *out = c->persist_ok ? c->pCS : 0; return LPC_OK;
    case LPC_INFO_ALPC_LOOP_CLUSTER_SIZE: *out = c->apersist_ok ? c->aCS : 0; return LPC_OK;
    case LPC_INFO_LOOP_ROW_SLOTS: *out = c->persist_ok ? c->pSlots : 0; return LPC_OK;
    case LPC_INFO_ALPC_LOOP_ROW_SLOTS: *out = c->apersist_ok ? c->aSlots : 0; return LPC_OK;
    case LPC_INFO_LOOP_COORDS_PER_THREAD: *out = c->persist_ok ? persist_coords_per_thread(c->b, c->pSL) : 0; return LPC_OK;
    case LPC_INFO_ALPC_LOOP_COORDS_PER_THREAD: *out = c->apersist_ok ? persist_coords_per_thread(c->b, c->aSL) : 0; return LPC_OK;
    case LPC_INFO_STEP_RING_STAGES: *out = c->inner_ok ? c->innerStages : 0; return LPC_OK;
    case LPC_INFO_LOOP_LAUNCHES: *out = c->persist_launches; return LPC_OK;
    case LPC_INFO_SNAPSHOT_ROWS_PER_TILE: *out = c->snapR; return LPC_OK;
    case LPC_INFO_SNAPSHOT_STAGES: *out = c->snapStages; return LPC_OK;
    case LPC_INFO_QUANT_ONE_LAUNCH: *out = c->last_one_launch; return LPC_OK;
    case LPC_INFO_AGGREGATE_SPLIT: *out = c->last_split; return LPC_OK;
    case LPC_INFO_QUANT_PIPELINED_RUNS: *out = c->last_pipelined_runs; return LPC_OK;
    default: return LPC_ERR_INVALID_ARG;
  }
}

int lpc_get_profile(lpc_ctx* c, double* ms_out, int64_t* launches_out, int32_t reset) {
  if (!c) return LPC_ERR_INVALID_ARG;
  TRY(prof_resolve(c));
  for (int i = 0; i < LPC_KERNEL_KINDS; ++i) {
    if (ms_out) ms_out[i] = c->prof_ms[i];
    if (launches_out) launches_out[i] = c->prof_n[i];
    if (reset) { c->prof_ms[i] = 0.0; c->prof_n[i] = 0; }
  }
  return LPC_OK;
}

int lpc_comm_bits(const lpc_ctx* c, uint64_t* step1_bits, uint64_t* step2_bits) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (step1_bits) *step1_bits = c->step1_bits;
  if (step2_bits) *step2_bits = c->step2_bits;
  return LPC_OK;
}

int lpc_quantize_pack(lpc_ctx* c, const float* U, const float* U_sub, int64_t len, int64_t ld, const int64_t* seg_offsets,
                      int32_t nseg, uint64_t k, uint32_t* codes_out, float* delta_out, uint32_t* clipped_out) {
  if (!c || !delta_out) return LPC_ERR_INVALID_ARG;
  if (len > 0 && (!U || !codes_out)) return fail(c, LPC_ERR_INVALID_ARG, "null vector or output");
  if (len < 0 || ld < len || nseg < 1) return fail(c, LPC_ERR_INVALID_ARG, "len / ld / nseg");  if (!aligned16(codes_out)) return fail(c, LPC_ERR_INVALID_ARG, "codes_out must be 16-byte aligned");
  TRY(make_plan(c, c->seg, len, c->b, seg_offsets, nseg));
  const SegPlan& p = c->seg;
  const size_t parts = (size_t)c->N * (size_t)std::max(p.ntiles, 1);
  if (parts > c->q_part_cap) {
    CU(c, cudaStreamSynchronize(c->stream));
    if (c->q_pmax) { cudaFree(c->q_pmax); cudaFree(c->q_ps1); cudaFree(c->q_ps2); c->q_pmax = nullptr; c->q_ps1 = c->q_ps2 = nullptr; }
    c->q_part_cap = 0;
    CU(c, cudaMalloc(&c->q_pmax, parts * 4)); CU(c, cudaMalloc(&c->q_ps1, parts * 4)); CU(c, cudaMalloc(&c->q_ps2, parts * 4));
    c->q_part_cap = parts;
  }
  const size_t recs = (size_t)c->N * (size_t)nseg;
  if (recs > c->q_scale_cap) {
    CU(c, cudaStreamSynchronize(c->stream));
    if (c->q_scales) { cudaFree(c->q_scales); cudaFree(c->q_clip); cudaFree(c->q_done); c->q_scales = nullptr; c->q_clip = nullptr; c->q_done = nullptr; }
    c->q_scale_cap = 0;
    CU(c, cudaMalloc(&c->q_scales, recs * sizeof(ScaleRec))); CU(c, cudaMalloc(&c->q_clip, recs * 4));
    CU(c, cudaMalloc(&c->q_done, recs * 4));
    c->q_scale_cap = recs;
    c->q_done_version = ~0ull;
  }
  QuantArgs a;
  a.U = U; a.U_sub = U_sub; a.ld = ld; a.N = c->N; a.b = c->b; a.clip_mode = c->clip_mode; a.clip_value = c->clip_value;
  a.seed = c->seed; a.k = k; a.segs = p.d_segs; a.tile_seg = p.d_tile_seg; a.nseg = p.nseg; a.ntiles = p.ntiles;
  a.pmax = c->q_pmax; a.ps1 = c->q_ps1; a.ps2 = c->q_ps2; a.scales = c->q_scales;
  a.codes = codes_out; a.stride_words = p.stride_words; a.delta_out = delta_out;
  a.clipped_out = clipped_out ? clipped_out : c->q_clip; a.count_clipped = clipped_out ? 1 : 0; a.dev_status = c->dev_status;
  a.shared_scale = c->shared_scale;
  {  // runs of the second pass that consist of whole tiles of one segment of 16-byte aligned vectors (per worker)
    const int run = quantize_run_tiles();
    const bool vec = aligned16(U) && (!U_sub || aligned16(U_sub)) && (ld % 4 == 0);
    int64_t runs = 0;
    const bool fixed_width = (c->b == 1 || c->b == 2 || c->b == 3 || c->b == 4 || c->b == 8);  // the other widths go tile by tile
    for (int t0 = 0; vec && fixed_width && t0 < p.ntiles; t0 += run) {
      const int t1 = std::min(t0 + run, p.ntiles) - 1;
      const SegInfo& g = p.segs[p.tile_seg[t0]];
      if (p.tile_seg[t0] == p.tile_seg[t1] && g.off % 4 == 0 && (int64_t)(t1 + 1 - g.tile_first) * TILE <= g.len) ++runs;
    }
    c->last_pipelined_runs = runs;
  }
  // one cooperative launch when the vectors stay in L2 between the statistics and the codes
  c->last_one_launch = 0;
  if (c->one_launch && !c->shared_scale && c->b != 32 && p.ntiles > 0 &&
      (int64_t)c->N * len * 4 * (U_sub ? 2 : 1) <= LPC_ONE_LAUNCH_BYTES) {
    int max_tiles = 1;
    for (const SegInfo& g : p.segs) max_tiles = std::max(max_tiles, g.tile_count);
    if (c->q_done_version != p.version || ((uint64_t)c->q_epoch + 2) * (uint64_t)max_tiles >= 0x7FFFFFFFull) {
      CU(c, cudaMemsetAsync(c->q_done, 0, recs * 4, c->stream));
      c->q_done_version = p.version;
      c->q_epoch = 0;
    }
    cudaError_t e;
    { ProfScope ps_(c, LPC_KERNEL_QUANT_FUSED); e = launch_quantize_fused(a, c->q_done, c->q_epoch, c->sm_count, c->stream); }
    if (e == cudaSuccess) {
      c->q_epoch += 1;
      c->last_one_launch = 1;
    } else {
      cudaGetLastError();  // the launch was refused: nothing ran, use the three launches
      c->one_launch = 0;
    }
  }
  if (c->last_one_launch) c->last_pipelined_runs = 0;
  else CU(c, launch_quantize_pack(a, c->stream, c->profile ? prof_hook : nullptr, c));
  if (!c->shared_scale) c->step2_bits += p.msg_bits * (uint64_t)c->N * (uint64_t)(c->N - 1);  // scheme (a); the server schemes count in lpc_server_reduce
  return LPC_OK;
}

namespace {
int ceil_log2_int(int N) {
  int r = 0;
  while ((1 << r) < N) ++r;
  return r;
}
}  // namespace

int lpc_sum_bits(int32_t b, int32_t N, int32_t* bits_out) {
  if (!bits_out || b < 2 || b > 16 || N < 1) return LPC_ERR_INVALID_ARG;
  *bits_out = b + ceil_log2_int(N);
  return LPC_OK;
}

int lpc_scheme_bits(int scheme, int64_t d, int32_t b, int32_t N, uint64_t* bits_out) {
  if (!bits_out || d < 0 || b < 1 || N < 1) return LPC_ERR_INVALID_ARG;
  const uint64_t bd = (uint64_t)b * (uint64_t)d;
  switch (scheme) {
    case LPC_SCHEME_BROADCAST: *bits_out = (32u + bd) * (uint64_t)N * (uint64_t)(N - 1); return LPC_OK;
    case LPC_SCHEME_SERVER_SUM: *bits_out = (uint64_t)N * (64u + 2u * bd + (uint64_t)d * (uint64_t)ceil_log2_int(N)); return LPC_OK;
    case LPC_SCHEME_SERVER_REQUANTIZE: *bits_out = (uint64_t)N * (64u + 2u * bd); return LPC_OK;
    default: return LPC_ERR_INVALID_ARG;
  }
}

namespace {
// n * H in bits for a histogram.
double entropy_of(const unsigned long long* h, int bins) {
  unsigned long long n = 0;
  for (int c = 0; c < bins; ++c) n += h[c];
  double bits = 0.0;
  for (int c = 0; c < bins; ++c)
    if (h[c]) bits -= (double)h[c] * std::log2((double)h[c] / (double)n);
  return bits;
}
// Length of the message under Huffman's code for its own histogram: the sum of the weights of all merged nodes.
uint64_t huffman_of(const unsigned long long* h, int bins) {
  std::vector<unsigned long long> w;
  for (int c = 0; c < bins; ++c)
    if (h[c]) w.push_back(h[c]);
  if (w.empty()) return 0;
  if (w.size() == 1) return w[0];  // a code word cannot be empty: one bit per coordinate
  std::priority_queue<unsigned long long, std::vector<unsigned long long>, std::greater<unsigned long long>> q(w.begin(), w.end());
  uint64_t total = 0;
  while (q.size() > 1) {
    const unsigned long long x = q.top(); q.pop();
    const unsigned long long y = q.top(); q.pop();
    total += x + y;
    q.push(x + y);
  }
  return total;
}
}  // namespace

int lpc_message_entropy(lpc_ctx* c, const uint32_t* codes, int64_t len, const int64_t* seg_offsets, int32_t nseg,
                        unsigned long long* hist_dev, double* entropy_bits_out, uint64_t* huffman_bits_out) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (!hist_dev || (len > 0 && !codes)) return fail(c, LPC_ERR_INVALID_ARG, "null stream or histogram");
  if (len < 0 || nseg < 1) return fail(c, LPC_ERR_INVALID_ARG, "len / nseg");
  if (c->b < 1 || c->b > 8) return fail(c, LPC_ERR_UNSUPPORTED, "code histograms cover b in 1..8");
  if (!aligned16(codes)) return fail(c, LPC_ERR_INVALID_ARG, "codes must be 16-byte aligned");
  TRY(make_plan(c, c->seg, len, c->b, seg_offsets, nseg));
  const int bins = 1 << c->b;
  const size_t count = (size_t)c->N * (size_t)nseg * (size_t)bins;
  CU(c, cudaMemsetAsync(hist_dev, 0, count * sizeof(unsigned long long), c->stream));
  HistArgs a;
  a.codes = codes; a.stride_words = c->seg.stride_words; a.N = c->N; a.b = c->b; a.segs = c->seg.d_segs;
  a.tile_seg = c->seg.d_tile_seg; a.nseg = nseg; a.ntiles = c->seg.ntiles; a.hist = hist_dev;
  { ProfScope ps_(c, LPC_KERNEL_OTHER); CU(c, launch_code_histogram(a, c->stream)); }
  if (!entropy_bits_out && !huffman_bits_out) return LPC_OK;  // histogram only: stays asynchronous
  std::vector<unsigned long long> h(count);
  CU(c, cudaMemcpyAsync(h.data(), hist_dev, count * sizeof(unsigned long long), cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  for (size_t m = 0; m < (size_t)c->N * (size_t)nseg; ++m) {
    if (entropy_bits_out) entropy_bits_out[m] = entropy_of(h.data() + m * bins, bins);
    if (huffman_bits_out) huffman_bits_out[m] = huffman_of(h.data() + m * bins, bins);
  }
  return LPC_OK;
}

int lpc_server_reduce(lpc_ctx* c, const uint32_t* codes, int64_t len, const int64_t* seg_offsets, int32_t nseg, int scheme,
                      uint64_t k, uint32_t* codes_out) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (len > 0 && (!codes || !codes_out)) return fail(c, LPC_ERR_INVALID_ARG, "null streams");
  if (len < 0 || nseg < 1) return fail(c, LPC_ERR_INVALID_ARG, "len / nseg");
  if (scheme != LPC_SCHEME_SERVER_SUM && scheme != LPC_SCHEME_SERVER_REQUANTIZE) return fail(c, LPC_ERR_INVALID_ARG, "scheme");
  if (c->b < 2 || c->b > 16) return fail(c, LPC_ERR_UNSUPPORTED, "the server schemes need an integer grid: b in 2..16");
  const int b_out = (scheme == LPC_SCHEME_SERVER_SUM) ? c->b + ceil_log2_int(c->N) : c->b;
  if (b_out > 16) return fail(c, LPC_ERR_UNSUPPORTED, "b + ceil(log2 N) exceeds 16 bits");
  if (!aligned16(codes) || !aligned16(codes_out)) return fail(c, LPC_ERR_INVALID_ARG, "streams must be 16-byte aligned");
  TRY(make_plan(c, c->seg, len, c->b, seg_offsets, nseg));
  TRY(make_plan(c, c->seg_out, len, b_out, seg_offsets, nseg));
  ServerArgs a;
  a.codes = codes; a.stride_words = c->seg.stride_words; a.N = c->N; a.b = c->b; a.b_out = b_out;
  a.requantize = (scheme == LPC_SCHEME_SERVER_REQUANTIZE) ? 1 : 0; a.seed = c->seed; a.k = k;
  a.segs = c->seg.d_segs; a.segs_out = c->seg_out.d_segs; a.tile_seg = c->seg.d_tile_seg; a.nseg = nseg; a.ntiles = c->seg.ntiles;
  a.out = codes_out;
  { ProfScope ps_(c, LPC_KERNEL_AGGREGATE); CU(c, launch_server_reduce(a, c->stream)); }
  // Table 1: every worker sends its message (b bits per coordinate and the scale) and receives the server's (b_out bits
  // per coordinate and the scale), per tensor segment
  c->step2_bits += (uint64_t)c->N * (c->seg.msg_bits + c->seg_out.msg_bits);
  return LPC_OK;
}

int lpc_unpack_average_prox(lpc_ctx* c, const uint32_t* codes, const float* delta, int64_t len, const int64_t* seg_offsets,
                            int32_t nseg, const float* mu, float* x_inout, float eta, float lambda_l1, float* v_out) {
  if (!c || !codes || !delta || !x_inout) return LPC_ERR_INVALID_ARG;
  if (len < 0 || nseg < 1) return fail(c, LPC_ERR_INVALID_ARG, "len / nseg");
  if (!aligned16(codes)) return fail(c, LPC_ERR_INVALID_ARG, "codes must be 16-byte aligned");
  TRY(make_plan(c, c->seg, len, c->b, seg_offsets, nseg));
  AggArgs a = agg_args(c, c->seg, codes, delta, mu, x_inout, eta, lambda_l1, v_out, c->divisor > 0 ? c->divisor : c->N);
  c->last_split = a.split;
  { ProfScope ps_(c, LPC_KERNEL_AGGREGATE); CU(c, launch_unpack_average_prox(a, c->stream)); }
  return LPC_OK;
}

int lpc_debug_wait_timeout(lpc_ctx* c, uint64_t limit_ns) {
  if (!c) return LPC_ERR_INVALID_ARG;
  if (limit_ns < 1000ull || limit_ns > 100000000ull) return fail(c, LPC_ERR_INVALID_ARG, "limit must be 1 us .. 100 ms");
  unsigned int* abort_flag = c->flags ? reinterpret_cast<unsigned int*>(c->flags + 512 * 16) : nullptr;
  if (abort_flag) CU(c, cudaMemsetAsync(abort_flag, 0, sizeof(unsigned long long), c->stream));
  CU(c, launch_wait_timeout(c->flags, abort_flag, c->dev_status, limit_ns, c->stream));
  return LPC_OK;
}

int lpc_debug_stream_blocks(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block0, int64_t count,
                            uint32_t* out, void* stream) {
  if (count < 0 || (count > 0 && !out)) return LPC_ERR_INVALID_ARG;
  if (count == 0) return LPC_OK;
  const cudaError_t e = launch_stream_blocks(seed, tag, worker, k, block0, count, out, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? LPC_OK : LPC_ERR_CUDA;
}

int lpc_svrg_run_host(const float* X_host, const float* y_host, int64_t n, int32_t d, int loss, float lambda_l1, int32_t N,
                      int32_t B, int32_t b, int clip_mode, float clip_value, uint64_t seed, int32_t S, int64_t m, float eta,
                      float* x_host_inout, double* objective_out, uint64_t* step2_bits_out) {
  if (!X_host || !y_host || !x_host_inout || n < 1 || d < 4 || S < 0 || m < 0) return LPC_ERR_INVALID_ARG;
  float *dX = nullptr, *dy = nullptr, *dx = nullptr;
  cudaStream_t st = nullptr;
  lpc_ctx* c = nullptr;
  int rc = LPC_OK;
  auto cu = [&](cudaError_t e) { if (e != cudaSuccess && rc == LPC_OK) rc = LPC_ERR_CUDA; return e == cudaSuccess; };
  if (cu(cudaStreamCreate(&st)) && cu(cudaMalloc(&dX, (size_t)n * d * 4)) && cu(cudaMalloc(&dy, (size_t)n * 4)) &&
      cu(cudaMalloc(&dx, (size_t)d * 4))) {
    cu(cudaMemcpyAsync(dX, X_host, (size_t)n * d * 4, cudaMemcpyHostToDevice, st));
    cu(cudaMemcpyAsync(dy, y_host, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    cu(cudaMemcpyAsync(dx, x_host_inout, (size_t)d * 4, cudaMemcpyHostToDevice, st));
    if (rc == LPC_OK) rc = lpc_init(&c, dX, dy, n, d, loss, lambda_l1, N, B, b, clip_mode, clip_value, seed, st);
    if (rc == LPC_OK) rc = lpc_set_iterate(c, dx);
    for (int s = 0; s < S && rc == LPC_OK; ++s) {
      rc = lpc_snapshot_full_grad(c, nullptr, nullptr);
      if (rc == LPC_OK) rc = lpc_inner_steps(c, eta, (uint64_t)s * (uint64_t)m, m);
    }
    if (rc == LPC_OK) rc = lpc_get_iterate(c, dx);
    if (rc == LPC_OK) cu(cudaMemcpyAsync(x_host_inout, dx, (size_t)d * 4, cudaMemcpyDeviceToHost, st));
    if (rc == LPC_OK && objective_out) rc = lpc_objective(c, nullptr, objective_out);
    if (rc == LPC_OK) rc = lpc_sync_status(c);
    if (rc == LPC_OK && step2_bits_out) lpc_comm_bits(c, nullptr, step2_bits_out);
  }
  if (c) lpc_destroy(c);
  if (st) cudaStreamSynchronize(st);
  if (dX) cudaFree(dX);
  if (dy) cudaFree(dy);
  if (dx) cudaFree(dx);
  if (st) cudaStreamDestroy(st);
  return rc;
}

}  // extern "C"

#ifdef LPC_TRACE
namespace lpc { cudaError_t read_stream_trace(unsigned long long* host_out); }
extern "C" int lpc_debug_stream_trace(unsigned long long* host_out) {
  return lpc::read_stream_trace(host_out) == cudaSuccess ? LPC_OK : LPC_ERR_CUDA;
}
#endif
