// The fused worker side of one inner iteration (Algorithm 1 steps 6-7, Algorithm 2 steps 7-8 and 11):
// minibatch sampling, the SVRG difference u^i, the scale of Eq. 2, the stochastic quantizer and bit
// packing in one kernel.  u^i lives in registers from the moment it is formed until its codes are
// stored; it is never written to memory (unless the inspection tap is on).
//
// Design: one thread-block cluster per worker.  The CS CTAs of a cluster split the coordinate range
// [0, P) (P = d rounded up to a power of two) into contiguous slices of SL = P/CS coordinates.  A CTA
// pulls its slice of the B sampled rows into shared memory with bulk copies (TMA) signalled on one
// mbarrier, computes the slice's part of every margin <X_a, x>, and exchanges the parts through
// distributed shared memory; after one cluster barrier every CTA knows the B margins and forms the
// coefficients l'(m_a(x)) - l'(m_a(x~)) (the snapshot margins are cached).  u is then accumulated from
// the rows still resident in shared memory, its max / sum / sum of squares are exchanged the same
// way, and after a second cluster barrier every CTA derives the same scale and quantizes its slice.
// In ALPC-SVRG one more cluster handles the shared batch J and stores v^ = u_J + mu in full
// precision.  No load with cluster multicast is used; each CTA fetches its own slice.
//
// Large minibatches (STREAM = true: more rows than shared memory holds, up to 1024 per worker) stream the
// rows instead, in batch order, through a ring of small stages filled by bulk copies, with no block barrier
// in the loop.  The warps are specialised: eight take the margin partial sums (one warp per row of a group, over
// the whole slice, reduced by shuffles alone) and send them to every CTA of the cluster as asynchronous stores that
// count on the receiver's mbarrier of that group; two turn the complete margins into coefficients; eight own the
// coordinates of u and add the rows -- still in shared memory -- into u, then hand the stage back; one refills
// the stages.  Every hand-over is an mbarrier phase, so waiting warps sleep in hardware and take no issue slots or
// shared-memory bandwidth from the working ones.  Each row is read from HBM once.
#include <cooperative_groups.h>

#include "lpc_device.cuh"
#include "lpc_inner.h"

namespace cg = cooperative_groups;

namespace lpc {
namespace {

constexpr int IT = 256;           // threads per CTA
constexpr int IGROUP = IT * 8;    // coordinates per pass
constexpr int MAXP = 4;           // passes per CTA: SL <= 8192
constexpr int MAXB = 64;          // minibatch rows
constexpr int MAXCS = 8;
// streaming path
constexpr int SG = 4;             // rows per ring stage
constexpr int SSLOTS = 16;        // exchange slots (a peer's margins run at most 2 * SMAXR - 2 groups ahead of this CTA's u)
constexpr int SMAXR = 8;          // ring stages at most
constexpr int SMAXB = 1024;       // rows per worker at most
constexpr int SDW = 8;            // warps that take margin partial sums: SDW / SG groups in flight on that side
constexpr int SUW = 8;            // warps that own the coordinates of u
constexpr int SCW = 2;            // warps that form coefficients (they alternate groups)
constexpr int SPW = 1;            // warp that refills the ring
constexpr int SMETAW = 1;         // warp that gathers labels and snapshot margins of the sampled rows, 32 rows per pass
constexpr int SNT = (SDW + SUW + SCW + SPW + SMETAW) * 32;  // threads of the streaming kernel

struct Smem {
  uint64_t bar;
  uint64_t xbar;                  // scale statistics of every CTA of the cluster have arrived (bytes of their stores)
  int64_t idx[MAXB];
  float yv[MAXB];
  float msnap[MAXB];
  float coef[MAXB];
  float wpart[MAXB * MAXP * 8];   // per-row warp partials of the margin products
  float mpart[MAXB * MAXCS];      // per-row slice partials of every CTA of the cluster (written by peers)
  float s1part[MAXCS], s2part[MAXCS];
  uint32_t maxpart[MAXCS];
  float ws1[MAXP * 8], ws2[MAXP * 8];
  uint32_t wmax[8];
  uint32_t wclip[8];
  Scale scale;
  int load_ok;
  __align__(16) uint8_t stage[IT * 16];
  // streaming path: every hand-over is an mbarrier phase, so a waiting warp sleeps in hardware instead of polling
  uint64_t sbar[SMAXR];           // stage filled (bulk-copy bytes)
  uint64_t ebar[SMAXR];           // stage read (one arrival per warp that adds rows into u and per margin warp of the group's side)
  uint64_t pbar[SSLOTS];          // margin partial sums of a group have arrived from every CTA (bytes of their stores)
  uint64_t cbar[SSLOTS];          // coefficients of a group are in `coefs`
  uint64_t mbar_meta[SMAXB / 32]; // labels and snapshot-side derivatives of 32 sampled rows are in place (used once each)
  __align__(16) float parts[SSLOTS][SG * MAXCS * 4];  // quarter-slice partial sums of the groups in flight (written by all CTAs of the cluster)
  __align__(16) float coefs[SSLOTS][SG];
  int stream_fail;                // a bounded wait ran out somewhere in this CTA
  int issued;                     // groups whose bulk copies have been issued
};

// Phase timestamps of every CTA of the kernel (entry, first copies issued, block-wide prologue done, cluster started, u
// complete, scale known, codes stored), for latency studies; compiled in only with -DLPC_TRACE.
#ifdef LPC_TRACE
constexpr int TRACE_CTAS = 1024;
__device__ unsigned long long g_stream_cta[TRACE_CTAS * 8];
#define LPC_PHASE_MARK(i)                                                         \
  do {                                                                            \
    const unsigned int cta_ = blockIdx.y * gridDim.x + blockIdx.x;                \
    if (threadIdx.x == 0 && cta_ < TRACE_CTAS) g_stream_cta[cta_ * 8 + (i)] = global_ns(); \
  } while (0)
#define LPC_WARP_MARK(i) /* by lane 0 of the calling warp */                       \
  do {                                                                            \
    const unsigned int cta_ = blockIdx.y * gridDim.x + blockIdx.x;                \
    if ((threadIdx.x & 31) == 0 && cta_ < TRACE_CTAS) g_stream_cta[cta_ * 8 + (i)] = global_ns(); \
  } while (0)
#else
#define LPC_PHASE_MARK(i) do { } while (0)
#define LPC_WARP_MARK(i) do { } while (0)
#endif

// BITS: 1, 2, 4, 8 fixed-width packing; 0: b from the arguments (1..16 or 32).
// STREAM: rows pass through a ring of stages (large minibatches; one pass, SL <= IGROUP) instead of all being resident.
template <int BITS, bool STREAM>
__global__ void __launch_bounds__(STREAM ? SNT : IT) inner_kernel(InnerArgs a) {
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  unsigned char* dyn = smem_raw + ((sizeof(Smem) + 15) & ~(size_t)15);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  LPC_PHASE_MARK(0);
  constexpr int NT = STREAM ? SNT : IT;  // the streaming path runs more warps, specialised by role
  const int rank = (int)cluster.block_rank();
  const int CS = a.CS, SL = a.SL, B = a.B, d = a.d;
  // sampled rows, their labels and cached snapshot margins; the row data (resident: B x SL; streaming: the ring)
  int64_t* s_idx = sm.idx;
  float* s_yv = sm.yv;
  float* s_ms = sm.msnap;
  float* rows = reinterpret_cast<float*>(dyn);
  if constexpr (STREAM) {
    const int Bp = (B + 3) & ~3;
    s_idx = reinterpret_cast<int64_t*>(dyn);
    s_yv = reinterpret_cast<float*>(s_idx + Bp);
    s_ms = s_yv + Bp;
    rows = s_ms + Bp;
  }
  const int worker = blockIdx.y;
  const bool is_J = (worker == a.N);
  const uint64_t k = a.k_base + (a.k_dev ? *a.k_dev : 0ull);
  const int b = BITS ? BITS : a.b;
  const int passes = (SL + IGROUP - 1) / IGROUP;
  const int c0 = rank * SL;                         // first coordinate of this CTA's slice
  const int width = max(0, min(SL, d - c0));        // coordinates of the slice that exist

  // ---- sampling (Algorithm 1 step 6): slot a uses word 0 of block a of the batch stream -----------------
  auto sample_slot = [&](int slot) -> int64_t {
    int64_t lo, span;
    uint32_t tag, wk;
    if (is_J) { lo = 0; span = a.n; tag = TAG_BATCH_J; wk = 0; }
    else if (a.sample_global) { lo = 0; span = a.n; tag = TAG_BATCH; wk = (uint32_t)worker; }
    else { span = a.n / a.N; lo = (int64_t)worker * span; tag = TAG_BATCH; wk = (uint32_t)worker; }
    const U4 r = stream_block(a.seed, tag, wk, k, (uint32_t)slot);
    return lo + (int64_t)(((uint64_t)r.x * (uint64_t)span) >> 32);
  };
  if constexpr (STREAM) {
    // The refill warp starts the first fills of the ring before anything else of the step: it sets up the stages'
    // barriers itself, samples the rows of the first stages (one per lane) and issues their copies; the other warps
    // sample the whole batch and set up the remaining barriers meanwhile.
    static_assert(SMAXR * SG <= 32 && SMAXR <= 32, "the first fills are issued by one warp, one row per lane");
    if (warp == SDW + SUW + SCW) {
      const int R0 = a.stream_stages, first = min(R0, (B + SG - 1) / SG);
      if (lane < SMAXR) mbar_init(&sm.sbar[lane], 1);
      mbar_fence_init();
      __syncwarp();
      const int g = lane / SG, j = lane % SG, cnt = min(SG, B - g * SG);
      if (width > 0 && g < first) {
        const uint32_t bytes = (uint32_t)width * 4u;
        if (j == 0) mbar_expect_tx(&sm.sbar[g], bytes * (uint32_t)cnt);
        if (j < cnt)
          bulk_load(rows + ((size_t)g * SG + j) * SL, a.X + sample_slot(g * SG + j) * (int64_t)d + c0, bytes, &sm.sbar[g]);
      }
      if (lane == 0) sm.issued = (width > 0) ? first : 0;
      LPC_WARP_MARK(2);
    }
  }
  for (int slot = tid; slot < B; slot += NT) {
    const int64_t row = sample_slot(slot);
    s_idx[slot] = row;
    if constexpr (!STREAM) {
      s_yv[slot] = a.y[row];
      s_ms[slot] = a.margins[row];
    }
  }
  if constexpr (STREAM) {
    // the barriers of the streaming path are set up side by side, one or two per thread
    static_assert(SMAXR + SSLOTS + SMAXB / 32 <= 64, "two warps set up the barriers");
    if (tid < SMAXR) {
      mbar_init(&sm.ebar[tid], SUW + SDW / 2);
    } else if (tid < SMAXR + SSLOTS) {
      mbar_init(&sm.pbar[tid - SMAXR], 1);
      mbar_init(&sm.cbar[tid - SMAXR], 1);
    } else if (tid < SMAXR + SSLOTS + (B + 31) / 32) {
      mbar_init(&sm.mbar_meta[tid - SMAXR - SSLOTS], 1);
    }
    if (tid == 0) {
      mbar_init(&sm.bar, 1);
      mbar_init(&sm.xbar, 1);
      sm.stream_fail = 0;
    }
    if (tid < 64) mbar_fence_init();
  } else if (tid == 0) {
    mbar_init(&sm.bar, 1);
    mbar_init(&sm.xbar, 1);
    mbar_fence_init();
  }
  // Every CTA of the cluster announces that it is running (its barriers exist); peers wait for this before their
  // first store into this CTA's shared memory.
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  __syncthreads();
  if (!STREAM && tid == 0 && width > 0) {
    const uint32_t bytes = (uint32_t)width * 4u;
    mbar_expect_tx(&sm.bar, bytes * (uint32_t)B);
    for (int r = 0; r < B; ++r) bulk_load(rows + (size_t)r * SL, a.X + s_idx[r] * (int64_t)d + c0, bytes, &sm.bar);
  }

  // ---- this thread's coordinates and the iterate at them ---------------------------------------------------
  float xr[MAXP][8];
#pragma unroll
  for (int p = 0; p < MAXP; ++p) {
    const int off = p * IGROUP + tid * 8;  // offset inside the slice
#pragma unroll
    for (int e = 0; e < 8; ++e) xr[p][e] = 0.f;
    if (p < passes && off < width) {  // width is a multiple of 4
      const float4 v0 = *reinterpret_cast<const float4*>(a.x + c0 + off);
      xr[p][0] = v0.x; xr[p][1] = v0.y; xr[p][2] = v0.z; xr[p][3] = v0.w;
      if (off + 4 < width) {
        const float4 v1 = *reinterpret_cast<const float4*>(a.x + c0 + off + 4);
        xr[p][4] = v1.x; xr[p][5] = v1.y; xr[p][6] = v1.z; xr[p][7] = v1.w;
      }
    }
  }

  bool ok = true;
  if (!STREAM && width > 0) ok = mbar_wait(&sm.bar, 0);
  if (!ok) {
    atomicOr(a.dev_status, DEV_TIMEOUT);
    ok = mbar_wait(&sm.bar, 0);  // one more bounded chance for the copies in flight before going on
  }

  // A row value of the slice (zero outside the existing columns).
  auto row8 = [&](int r, int off, float* v) {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = 0.f;
    if (off < width) {
      const float4 v0 = *reinterpret_cast<const float4*>(rows + (size_t)r * SL + off);
      v[0] = v0.x; v[1] = v0.y; v[2] = v0.z; v[3] = v0.w;
      if (off + 4 < width) {
        const float4 v1 = *reinterpret_cast<const float4*>(rows + (size_t)r * SL + off + 4);
        v[4] = v1.x; v[5] = v1.y; v[6] = v1.z; v[7] = v1.w;
      }
    }
  };

  const float invB = __fdiv_rn(1.0f, (float)B);
  float u[MAXP][8];
  if constexpr (STREAM) {
    // ---- streaming: groups of SG rows in batch order through a ring of R stages, no block barrier inside.
    // The first SDW warps take the margin partial sums (one warp per row, over the whole slice) and send them to
    // the cluster; the last SCW warps turn the partial sums of all CTAs into coefficients and refill the stages;
    // the SUW warps in between own the coordinates of u and add the rows, then hand the stage back. ----------------------
#pragma unroll
    for (int p = 0; p < MAXP; ++p) {
#pragma unroll
      for (int e = 0; e < 8; ++e) u[p][e] = 0.f;
    }
    const int R = a.stream_stages;
    const int ngroups = (B + SG - 1) / SG;
    const uint32_t row_bytes = (uint32_t)width * 4u;
    // One warp: the rows of group g into stage g % R.  Lane 0 arms the stage's barrier with the byte count, lane j
    // issues the copy of row j: a bulk copy occupies its issuing thread for a noticeable time, so the rows of a
    // group are issued side by side.
    auto issue = [&](int g, int lane_in_group) {
      const int s = g % R;
      const int cnt = min(SG, B - g * SG);
      if (lane_in_group == 0) {
        mbar_expect_tx(&sm.sbar[s], row_bytes * (uint32_t)cnt);
        sm.issued = g + 1;
      }
      if (lane_in_group < cnt)
        bulk_load(rows + ((size_t)s * SG + lane_in_group) * SL, a.X + s_idx[g * SG + lane_in_group] * (int64_t)d + c0,
                  row_bytes, &sm.sbar[s]);
    };
    static_assert(SG * MAXCS == 32, "one lane per (row, CTA) pair when the coefficients are formed");
    LPC_PHASE_MARK(1);
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // all peers have started
    LPC_PHASE_MARK(3);
    bool gave_up = false;  // after one wait ran out this thread waits no more (the status word says so)
    auto wait_on = [&](uint64_t* bar, uint32_t parity, bool from_cluster) {
      if (gave_up) return;
      if (!from_cluster && mbar_test(bar, parity)) return;
      const bool ok = from_cluster ? mbar_wait_cluster(bar, parity) : mbar_wait(bar, parity);
      if (!ok) {
        atomicOr(a.dev_status, DEV_TIMEOUT);
        sm.stream_fail = 1;
        gave_up = true;
      }
    };
    auto wait_stage = [&](int g) {
      if (width > 0) wait_on(&sm.sbar[g % R], (uint32_t)((g / R) & 1), false);
    };
    // Shared-memory reads are laid out so that a warp's 16-byte loads touch consecutive addresses (no bank
    // conflicts): the ring is read twice per row and written once, and that traffic is what bounds a group.
    constexpr int NBK = IGROUP / 128;    // blocks of 128 coordinates per slice: 16; a lane takes 4 coordinates of each
    constexpr int AT = SUW * 32;         // threads that own the coordinates of u
    constexpr int UC = IGROUP / 4 / AT;  // 4-coordinate pieces per such thread: 2, IGROUP / UC apart
    float ua[UC][4];
#pragma unroll
    for (int q = 0; q < UC; ++q)
#pragma unroll
      for (int e = 0; e < 4; ++e) ua[q][e] = 0.f;
    const bool full = (width == IGROUP);  // the usual case: every column of the slice exists, nothing to test per load
    auto row4 = [&](int r, int off) {  // four row values of the slice (zero outside the existing columns)
      return (off < width) ? *reinterpret_cast<const float4*>(rows + (size_t)r * SL + off) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    if (warp < SDW) {
      // -- margins: the SMW = 4 warps of a side share a group, warp w of them taking the blocks 4 w .. 4 w + 3 (a quarter
      // of the slice) of all rows of the group; the two sides alternate groups.  Lane l holds x for the coordinates
      // 128 q + 4 l .. + 3 of its blocks q.  The leaves of the tree in coordinate order: four products per lane
      // (tree4), then the tree over the 32 lanes of a block, then the tree over the four blocks; the quarter sums go to
      // every CTA of the cluster as stores that count on that CTA's barrier of the group, and are combined there.
      // Sixteen independent 16-byte loads and one reduction per group keep a warp's dependent chains short.
      constexpr int SMW = 4, QB = NBK / SMW;  // warps per side; blocks per warp
      static_assert(SDW == 2 * SMW && QB * SG == 16, "one 16-value recursive-halving reduction per group");
      const int wq = warp % SMW;
      float4 xs[QB];
#pragma unroll
      for (int q = 0; q < QB; ++q) {
        const int off = (wq * QB + q) * 128 + lane * 4;  // width is a multiple of 4
        xs[q] = (off < width) ? *reinterpret_cast<const float4*>(a.x + c0 + off) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      // after the reduction lane l holds the sum of row halving_index<2>(l & 3); lane l sends it to CTA l >> 2
      const int myrow = ((lane & 1) << 1) | ((lane >> 1) & 1);
#pragma unroll 1
      for (int g = warp / SMW; g < ngroups; g += SDW / SMW) {
        const int cnt = min(SG, B - g * SG);
        wait_stage(g);
        // two rows at a time (eight loads in flight): the sixteen partial sums of the group are all that stays
        float sv[SG * QB];
#pragma unroll
        for (int h = 0; h < SG; h += 2) {
          float4 v[2][QB];
          if (full) {
            const float* src = rows + (size_t)((g % R) * SG + h) * SL + wq * QB * 128 + lane * 4;
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
              for (int q = 0; q < QB; ++q) v[j][q] = *reinterpret_cast<const float4*>(src + j * SL + q * 128);
          } else {
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
              for (int q = 0; q < QB; ++q) v[j][q] = row4((g % R) * SG + h + j, (wq * QB + q) * 128 + lane * 4);
          }
#pragma unroll
          for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int q = 0; q < QB; ++q)
              sv[(h + j) * QB + q] = tree4(mul_rn(v[j][q].x, xs[q].x), mul_rn(v[j][q].y, xs[q].y), mul_rn(v[j][q].z, xs[q].z),
                                           mul_rn(v[j][q].w, xs[q].w));
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ebar[g % R]);  // this warp has read its quarter of the stage
        WarpHalving<SG * QB, 0>::run(sv, lane);  // lane holds the 32-lane tree sum of (row, block) halving_index<4>(lane)
        float part = sv[0];
        part = add_rn(part, __shfl_xor_sync(0xFFFFFFFFu, part, 8));  // blocks 2k, 2k+1 of the row
        part = add_rn(part, __shfl_xor_sync(0xFFFFFFFFu, part, 4));
        if ((lane >> 2) < CS && myrow < cnt)
          st_async_cluster(&sm.parts[g % SSLOTS][(myrow * MAXCS + rank) * SMW + wq], &sm.pbar[g % SSLOTS],
                           (uint32_t)(lane >> 2), __float_as_uint(part));
      }
    } else if (warp < SDW + SUW) {
      // -- u: thread t of these warps owns the coordinates 4 t .. 4 t + 3 of each half of the slice.  The rows of a
      // group go from the stage into registers as soon as the stage is filled, one group ahead of the group whose
      // coefficients are awaited, and the stage is handed back at once: a stage is then occupied for the time of
      // its copies and two shared-memory reads, not for the round trip of the margins through the cluster.
      const int t = tid - SDW * 32;
      float4 va[SG][UC], vb[SG][UC];
      auto take = [&](int g, float4 (&v)[SG][UC]) {  // rows past a ragged end are read and not used
        const int s = g % R;
        wait_stage(g);
        if (full) {
          const float* src = rows + (size_t)(s * SG) * SL + t * 4;
#pragma unroll
          for (int j = 0; j < SG; ++j)
#pragma unroll
            for (int q = 0; q < UC; ++q) v[j][q] = *reinterpret_cast<const float4*>(src + j * SL + q * (IGROUP / UC));
        } else {
#pragma unroll
          for (int j = 0; j < SG; ++j)
#pragma unroll
            for (int q = 0; q < UC; ++q) v[j][q] = row4(s * SG + j, q * (IGROUP / UC) + t * 4);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ebar[s]);  // release: the loads above are performed before the arrival counts
      };
      auto add = [&](int g, const float4 (&v)[SG][UC]) {
        const int cnt = min(SG, B - g * SG);
        wait_on(&sm.cbar[g % SSLOTS], (uint32_t)((g / SSLOTS) & 1), false);
        const float4 c4 = *reinterpret_cast<const float4*>(sm.coefs[g % SSLOTS]);
        const float cj[SG] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
        for (int j = 0; j < SG; ++j) {
          if (j < cnt) {
#pragma unroll
            for (int q = 0; q < UC; ++q) {
              ua[q][0] = add_rn(ua[q][0], mul_rn(cj[j], v[j][q].x));
              ua[q][1] = add_rn(ua[q][1], mul_rn(cj[j], v[j][q].y));
              ua[q][2] = add_rn(ua[q][2], mul_rn(cj[j], v[j][q].z));
              ua[q][3] = add_rn(ua[q][3], mul_rn(cj[j], v[j][q].w));
            }
          }
        }
      };
      take(0, va);
#pragma unroll 1
      for (int g = 0; g < ngroups; g += 2) {
        if (g + 1 < ngroups) take(g + 1, vb);
        add(g, va);
        if (g + 1 < ngroups) {
          if (g + 2 < ngroups) take(g + 2, va);
          add(g + 1, vb);
        }
      }
    } else if (warp < SDW + SUW + SCW) {
      // -- coefficients (warp c of this side takes the groups c, c + SCW, ...): lane j collects the partial sums of
      // row j of a group from all CTAs of the cluster and leaves the coefficient l'(m) - l'(m~) for the update side.
      // Running in warps of their own, the fp64 loss derivative delays neither the margins nor the updates.
#pragma unroll 1
      for (int g = warp - (SDW + SUW); g < ngroups; g += SCW) {
        const int cnt = min(SG, B - g * SG);
        const int sl = g % SSLOTS;
        if (lane == 0) mbar_expect_tx(&sm.pbar[sl], (uint32_t)(CS * cnt * 16));  // this phase: one arrival and the bytes of 4 quarter sums per row and CTA
        __syncwarp();
        wait_on(&sm.mbar_meta[(g * SG) / 32], 0u, false);
        wait_on(&sm.pbar[sl], (uint32_t)((g / SSLOTS) & 1), true);
        // lane (j, q) = (lane / MAXCS, lane % MAXCS): the tree over the four quarter sums of CTA q's slice for row j, then
        // the tree over the CTAs by shuffles; lane (j, 0) ends with the margin of row j
        {
          const int j = lane / MAXCS, q = lane % MAXCS;
          float mq = 0.f;
          if (q < CS) {
            const float4 pq = *reinterpret_cast<const float4*>(&sm.parts[sl][(j * MAXCS + q) * 4]);
            mq = tree4(pq.x, pq.y, pq.z, pq.w);
          }
          // CS is a power of two: the tree over q = 0 .. CS-1
          if (CS > 1) mq = add_rn(mq, __shfl_xor_sync(0xFFFFFFFFu, mq, 1));
          if (CS > 2) mq = add_rn(mq, __shfl_xor_sync(0xFFFFFFFFu, mq, 2));
          if (CS > 4) mq = add_rn(mq, __shfl_xor_sync(0xFFFFFFFFu, mq, 4));
          if (q == 0) {
            float c = 0.f;
            if (j < cnt) {
              const int slot = g * SG + j;
              c = __fsub_rn(loss_deriv(a.loss, mq, s_yv[slot]), s_ms[slot]);
              if (rank == 0) {
                if (a.idx_tap) a.idx_tap[(int64_t)worker * B + slot] = s_idx[slot];
                if (a.coef_tap) a.coef_tap[(int64_t)worker * B + slot] = c;
              }
            }
            sm.coefs[sl][j] = c;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.cbar[sl]);
      }
    } else if (warp < SDW + SUW + SCW + SPW) {
      // -- refills: a stage goes back to the bulk copies the moment the update side has handed it over
#pragma unroll 1
      for (int g = R; g < ngroups; ++g) {
        const int h = g - R;
        wait_on(&sm.ebar[h % R], (uint32_t)((h / R) & 1), false);
        if (gave_up) break;
        if (width > 0 && lane < SG) issue(g, lane);
        __syncwarp();
      }
    } else {
      // -- labels and the snapshot side of the coefficients, l'(m~_a), 32 sampled rows per pass, ahead of their use
#pragma unroll 1
      for (int base = 0; base < B; base += 32) {
        const int slot = base + lane;
        if (slot < B) {
          const int64_t row = s_idx[slot];
          const float yv = a.y[row];
          s_yv[slot] = yv;
          s_ms[slot] = loss_deriv(a.loss, a.margins[row], yv);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.mbar_meta[base / 32]);
      }
    }
    __syncthreads();  // both sides are done with the ring: it now carries u to the usual owner of each coordinate
    if (sm.stream_fail) {  // a wait ran out: give the copies still in flight a bounded chance to land before the ring is reused
      if (tid == 0 && width > 0)
        for (int g = max(0, sm.issued - R); g < sm.issued; ++g) mbar_wait(&sm.sbar[g % R], (uint32_t)((g / R) & 1), 100000000ull);
      __syncthreads();
    }
    if (warp >= SDW && warp < SDW + SUW) {
      const int t = tid - SDW * 32;
#pragma unroll
      for (int q = 0; q < UC; ++q) {
        const int off = q * (IGROUP / UC) + t * 4;
        if (off < SL)  // the ring holds at least one slice
          *reinterpret_cast<float4*>(rows + off) = make_float4(ua[q][0], ua[q][1], ua[q][2], ua[q][3]);
      }
    }
    __syncthreads();
    if (tid < IT && tid * 8 < SL) {
      const float4 v0 = *reinterpret_cast<const float4*>(rows + tid * 8);
      const float4 v1 = *reinterpret_cast<const float4*>(rows + tid * 8 + 4);
      u[0][0] = v0.x; u[0][1] = v0.y; u[0][2] = v0.z; u[0][3] = v0.w;
      u[0][4] = v1.x; u[0][5] = v1.y; u[0][6] = v1.z; u[0][7] = v1.w;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) u[0][e] = mul_rn(u[0][e], invB);
  } else {
  // ---- margins <X_a, x>: balanced tree over the column index ---------------------------------------------------
  for (int r = 0; r < B; ++r) {
#pragma unroll
    for (int p = 0; p < MAXP; ++p) {
      if (p < passes) {
        float v[8], pr[8];
        row8(r, p * IGROUP + tid * 8, v);
#pragma unroll
        for (int e = 0; e < 8; ++e) pr[e] = mul_rn(v[e], xr[p][e]);
        const float s = warp_tree_sum(tree8(pr));
        if (lane == 0) sm.wpart[(r * MAXP + p) * 8 + warp] = s;
      }
    }
  }
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // all peers have started
  __syncthreads();
  if (tid < B) {
    int np = 1;
    while (np < passes) np <<= 1;
    float part;
    if (np == 1) {
      part = smem_tree_sum(&sm.wpart[tid * MAXP * 8], 8);
    } else {
      float tmp[MAXP];
      for (int p = 0; p < np; ++p) tmp[p] = (p < passes) ? smem_tree_sum(&sm.wpart[(tid * MAXP + p) * 8], 8) : 0.f;
      part = (np == 2) ? add_rn(tmp[0], tmp[1]) : tree4(tmp[0], tmp[1], tmp[2], tmp[3]);
    }
    for (int q = 0; q < CS; ++q) {
      float* peer = cluster.map_shared_rank(sm.mpart, q);
      peer[tid * MAXCS + rank] = part;
    }
  }
  cluster.sync();
  if (tid < B) {
    const float m = smem_tree_sum(&sm.mpart[tid * MAXCS], CS);
    const float g_cur = loss_deriv(a.loss, m, s_yv[tid]);
    const float g_snap = loss_deriv(a.loss, s_ms[tid], s_yv[tid]);
    const float c = __fsub_rn(g_cur, g_snap);
    sm.coef[tid] = c;
    if (rank == 0) {
      if (a.idx_tap) a.idx_tap[(int64_t)worker * B + tid] = s_idx[tid];
      if (a.coef_tap) a.coef_tap[(int64_t)worker * B + tid] = c;
    }
  }
  __syncthreads();

  // ---- u = (1/B) sum_a c_a X_a, summed in batch order (Algorithm 1 step 6) ------------------------------------
#pragma unroll
  for (int p = 0; p < MAXP; ++p) {
#pragma unroll
    for (int e = 0; e < 8; ++e) u[p][e] = 0.f;
    if (p < passes) {
      for (int r = 0; r < B; ++r) {
        float v[8];
        row8(r, p * IGROUP + tid * 8, v);
        const float c = sm.coef[r];
#pragma unroll
        for (int e = 0; e < 8; ++e) u[p][e] = add_rn(u[p][e], mul_rn(c, v[e]));
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) u[p][e] = mul_rn(u[p][e], invB);
    }
  }

  }

  if (is_J) {  // double sampling: v^ = u_J + mu in full precision, nothing quantized
#pragma unroll
    for (int p = 0; p < MAXP; ++p) {
      const int off = p * IGROUP + tid * 8;
      if (p < passes) {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (off + e < width) a.vhat[c0 + off + e] = add_rn(u[p][e], a.mu[c0 + off + e]);
      }
    }
    return;  // the whole cluster leaves together: no further cluster barrier on this path
  }
  if (a.u_tap) {
#pragma unroll
    for (int p = 0; p < MAXP; ++p) {
      const int off = p * IGROUP + tid * 8;
      if (p < passes) {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (off + e < width) a.u_tap[(int64_t)worker * d + c0 + off + e] = u[p][e];
      }
    }
  }

  // rounding bits of the first pass: they depend on the counters only, so they are drawn before the scale is known
  U4 r_first = U4{0, 0, 0, 0};
  if (b != 32) r_first = stream_block(a.seed, TAG_ROUND, (uint32_t)worker, k, (uint32_t)((c0 + tid * 8) >> 3));

  // ---- scale (Eq. 2): max |u| and, for the c*std rule, tree sums of u and u^2 ----------------------------------
  LPC_PHASE_MARK(5);
  uint32_t mx = 0;
#pragma unroll
  for (int p = 0; p < MAXP; ++p) {
    if (p < passes) {
#pragma unroll
      for (int e = 0; e < 8; ++e) mx = max(mx, __float_as_uint(fabsf(u[p][e])));
      if (a.clip_mode == CLIP_STD) {
        float sq[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) sq[e] = mul_rn(u[p][e], u[p][e]);
        const float s1 = warp_tree_sum(tree8(u[p]));
        const float s2 = warp_tree_sum(tree8(sq));
        if (lane == 0 && warp < IT / 32) { sm.ws1[p * 8 + warp] = s1; sm.ws2[p * 8 + warp] = s2; }
      }
    }
  }
  mx = warp_max_u32(mx);
  if (lane == 0 && warp < IT / 32) sm.wmax[warp] = mx;
  __syncthreads();
  if (tid == 0) {
    uint32_t m = 0;
    for (int w = 0; w < 8; ++w) m = max(m, sm.wmax[w]);
    float s1 = 0.f, s2 = 0.f;
    if (a.clip_mode == CLIP_STD) {
      int np = 1;
      while (np < passes) np <<= 1;
      for (int i = passes * 8; i < np * 8; ++i) { sm.ws1[i] = 0.f; sm.ws2[i] = 0.f; }
      s1 = smem_tree_sum(sm.ws1, np * 8);
      s2 = smem_tree_sum(sm.ws2, np * 8);
    }
    // the three statistics go to every CTA of the cluster as stores that count on the receiver's barrier: the one
    // thread that needs them waits for their bytes, and no cluster-wide barrier is paid
    mbar_expect_tx(&sm.xbar, (uint32_t)(CS * 12));
    for (int q = 0; q < CS; ++q) {
      st_async_cluster(&sm.maxpart[rank], &sm.xbar, (uint32_t)q, m);
      st_async_cluster(&sm.s1part[rank], &sm.xbar, (uint32_t)q, __float_as_uint(s1));
      st_async_cluster(&sm.s2part[rank], &sm.xbar, (uint32_t)q, __float_as_uint(s2));
    }
    if (!mbar_wait_cluster(&sm.xbar, 0)) atomicOr(a.dev_status, DEV_TIMEOUT);
  }
  if (tid == 0) {
    uint32_t m = 0;
    for (int q = 0; q < CS; ++q) m = max(m, sm.maxpart[q]);
    float S1 = 0.f, S2 = 0.f;
    if (a.clip_mode == CLIP_STD) { S1 = smem_tree_sum(sm.s1part, CS); S2 = smem_tree_sum(sm.s2part, CS); }
    sm.scale = make_scale(m, S1, S2, d, b, a.clip_mode, a.clip_value);
    if (rank == 0) {
      a.delta[worker] = sm.scale.delta;
      if (sm.scale.flags & 2u) atomicOr(a.dev_status, DEV_NONFINITE);
    }
  }
  __syncthreads();
  LPC_PHASE_MARK(6);
  const Scale sc = sm.scale;
  const bool degenerate = (sc.flags & 1u) != 0;
  const uint32_t zero_code = (b == 1) ? 0u : (1u << (b - 1));
  uint32_t* out = a.codes + (int64_t)worker * a.stride_words;

  // ---- quantize (Section 2.2) and pack ---------------------------------------------------------------------------
  uint32_t nclip = 0;
#pragma unroll
  for (int p = 0; p < MAXP; ++p) {
    if (p >= passes) break;
    const int off = p * IGROUP + tid * 8;
    const int c = c0 + off;  // global coordinate, multiple of 8
    const bool mine = off < SL;
    if (b == 32) {
      if (mine) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float v = u[p][e];
          if (a.clip_mode != CLIP_NONE && c + e < d) {
            if (v > sc.T) { v = sc.T; ++nclip; }
            if (v < -sc.T) { v = -sc.T; ++nclip; }
          }
          if (c + e < a.pad_words) out[c + e] = (c + e < d) ? __float_as_uint(v) : 0u;
        }
      }
      continue;
    }
    uint64_t lo = 0, hi = 0;
    if (mine && c < d) {
      U4 r = U4{0, 0, 0, 0};
      if (!degenerate) r = (p == 0) ? r_first : stream_block(a.seed, TAG_ROUND, (uint32_t)worker, k, (uint32_t)(c >> 3));
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        if (c + e < d) {
          uint32_t code = zero_code;
          if (!degenerate) {
            code = BITS ? quantize_code<BITS ? BITS : 2>(u[p][e], sc.rdelta, lane16(r, e))
                        : quantize_code_rt(u[p][e], sc.rdelta, lane16(r, e), b);
            nclip += (u[p][e] > sc.T || u[p][e] < sc.lower) ? 1u : 0u;
          }
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
    if (BITS == 8) {
      const int64_t w = (int64_t)(c >> 3) * 2;
      if (mine && w < a.pad_words) *reinterpret_cast<uint2*>(out + w) = make_uint2((uint32_t)lo, (uint32_t)(lo >> 32));
    } else if (BITS == 4) {
      const int64_t w = c >> 3;
      if (mine && w < a.pad_words) out[w] = (uint32_t)lo;
    } else if (BITS == 2) {
      const uint32_t own = (uint32_t)lo;
      const uint32_t next = __shfl_down_sync(0xFFFFFFFFu, own, 1);
      const int64_t w = c >> 4;
      if (mine && (lane & 1) == 0 && w < a.pad_words) out[w] = own | (next << 16);
    } else if (BITS == 1) {
      const uint32_t own = (uint32_t)lo;
      const uint32_t n1 = __shfl_down_sync(0xFFFFFFFFu, own, 1);
      const uint32_t n2 = __shfl_down_sync(0xFFFFFFFFu, own, 2);
      const uint32_t n3 = __shfl_down_sync(0xFFFFFFFFu, own, 3);
      const int64_t w = c >> 5;
      if (mine && (lane & 3) == 0 && w < a.pad_words) out[w] = own | (n1 << 8) | (n2 << 16) | (n3 << 24);
    } else {
      if (p > 0) __syncthreads();
      for (int i = 0; i < b; ++i)
        if (tid < IT) sm.stage[tid * b + i] = (uint8_t)((i < 8) ? (lo >> (8 * i)) : (hi >> (8 * (i - 8))));
      __syncthreads();
      const int span = min(IGROUP, SL - p * IGROUP);           // coordinates of this pass (multiple of 32)
      const int64_t w0 = (int64_t)((c0 + p * IGROUP) >> 5) * b;  // exact: the pass starts on a multiple of 32
      const uint32_t* st = reinterpret_cast<const uint32_t*>(sm.stage);
      for (int w = tid; w < (span / 32) * b && tid < IT; w += IT)
        if (w0 + w < a.pad_words) out[w0 + w] = st[w];
    }
  }
  nclip = __reduce_add_sync(0xFFFFFFFFu, nclip);
  if (lane == 0 && warp < IT / 32) sm.wclip[warp] = nclip;
  __syncthreads();
  if (tid == 0) {
    uint32_t t = 0;
    for (int w = 0; w < 8; ++w) t += sm.wclip[w];
    a.clipped_part[worker * MAXCS + rank] = t;
  }
  LPC_PHASE_MARK(7);
}

template <int BITS, bool STREAM>
cudaError_t launch_t(const InnerArgs& a, size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(inner_kernel<BITS, STREAM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)a.CS, (unsigned)(a.N + (a.has_J ? 1 : 0)), 1);
  cfg.blockDim = dim3(STREAM ? SNT : IT, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)a.CS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, inner_kernel<BITS, STREAM>, a);
}

__global__ void clipped_sum_kernel(const uint32_t* __restrict__ part, int N, uint32_t* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) {
    uint32_t t = 0;
    for (int q = 0; q < MAXCS; ++q) t += part[i * MAXCS + q];
    out[i] = t;
  }
}

// x = tau1*z + tau2*x~ + (1 - tau1 - tau2)*y  (Algorithm 2 step 6), evaluated as ((tau1*z)+(tau2*x~))+(tau3*y).
__global__ void coupling_kernel(const float* __restrict__ z, const float* __restrict__ xt, const float* __restrict__ y,
                                float tau1, float tau2, int d, float* __restrict__ x) {
  const float tau3 = __fsub_rn(__fsub_rn(1.0f, tau1), tau2);
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < d) x[j] = add_rn(add_rn(mul_rn(tau1, z[j]), mul_rn(tau2, xt[j])), mul_rn(tau3, y[j]));
}

// x~ candidate = ysum / m (Algorithm 3 step 5) becomes the iterate; ysum is cleared.
__global__ void mean_y_kernel(float* __restrict__ ysum, float inv_m, int d, float* __restrict__ x) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < d) {
    x[j] = mul_rn(ysum[j], inv_m);
    ysum[j] = 0.f;
  }
}

}  // namespace

int inner_max_b() { return SMAXB; }
int inner_clipped_stride() { return MAXCS; }

// Picks the cluster size and slice width, and whether the rows stay resident in shared memory (stages = 0) or
// stream through a ring of `stages` stages of SG rows.  Returns false when d is too large for the fused kernel.
bool inner_plan(int d, int B, int want_cs, int max_smem, int* CS_out, int* SL_out, size_t* smem_out, int* stages_out) {
  int P = 1;
  while (P < d) P <<= 1;
  if (P < 32) P = 32;
  const size_t fixed = (sizeof(Smem) + 15) & ~(size_t)15;
  if (B <= MAXB) {
    for (int cs = 1; cs <= MAXCS; cs <<= 1) {
      if (want_cs > 0 && cs != want_cs) continue;
      const int SL = P / cs;
      if (SL < 32) break;
      if (SL > IGROUP * MAXP) continue;
      const size_t smem = fixed + (size_t)B * SL * 4;
      if (smem > (size_t)max_smem) continue;
      // automatic choice: the first (smallest) cluster whose slice is covered in one pass
      if (want_cs > 0 || SL <= IGROUP || cs == MAXCS) {
        *CS_out = cs; *SL_out = SL; *smem_out = smem; *stages_out = 0;
        return true;
      }
    }
  }
  if (B > SMAXB) return false;
  // streaming: one pass per CTA (SL <= IGROUP), as many ring stages as shared memory holds
  const size_t meta = (size_t)((B + 3) & ~3) * 16;
  for (int cs = 1; cs <= MAXCS; cs <<= 1) {
    if (want_cs > 0 && cs != want_cs) continue;
    const int SL = P / cs;
    if (SL < 32) break;
    if (SL > IGROUP) continue;
    const size_t stage = (size_t)SG * SL * 4;
    if (fixed + meta + 3 * stage > (size_t)max_smem) continue;
    int R = (int)(((size_t)max_smem - fixed - meta) / stage);
    if (R > SMAXR) R = SMAXR;
    *CS_out = cs; *SL_out = SL; *smem_out = fixed + meta + (size_t)R * stage; *stages_out = R;
    return true;
  }
  return false;
}

template <bool STREAM>
cudaError_t launch_s(const InnerArgs& a, size_t smem, cudaStream_t st) {
  switch (a.b) {
    case 1: return launch_t<1, STREAM>(a, smem, st);
    case 2: return launch_t<2, STREAM>(a, smem, st);
    case 4: return launch_t<4, STREAM>(a, smem, st);
    case 8: return launch_t<8, STREAM>(a, smem, st);
    default: return launch_t<0, STREAM>(a, smem, st);
  }
}

cudaError_t launch_inner(const InnerArgs& a, size_t smem, cudaStream_t st) {
  return a.stream_stages > 0 ? launch_s<true>(a, smem, st) : launch_s<false>(a, smem, st);
}

#ifdef LPC_TRACE
cudaError_t read_stream_trace(unsigned long long* host_out) {  // TRACE_CTAS x 8 marks
  return cudaMemcpyFromSymbol(host_out, g_stream_cta, sizeof(g_stream_cta));
}
#endif

cudaError_t launch_clipped_sum(const uint32_t* part, int N, uint32_t* out, cudaStream_t st) {
  clipped_sum_kernel<<<(N + 127) / 128, 128, 0, st>>>(part, N, out);
  return cudaGetLastError();
}

cudaError_t launch_coupling(const float* z, const float* xt, const float* y, float tau1, float tau2, int d, float* x,
                            cudaStream_t st) {
  coupling_kernel<<<(d + 255) / 256, 256, 0, st>>>(z, xt, y, tau1, tau2, d, x);
  return cudaGetLastError();
}

cudaError_t launch_mean_y(float* ysum, float inv_m, int d, float* x, cudaStream_t st) {
  mean_y_kernel<<<(d + 255) / 256, 256, 0, st>>>(ysum, inv_m, d, x);
  return cudaGetLastError();
}

}  // namespace lpc
