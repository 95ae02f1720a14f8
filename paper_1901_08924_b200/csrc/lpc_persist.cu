// The whole inner loop of Algorithm 1 (steps 5-11) in ONE cooperative launch.
//
// An inner iteration moves only N*B rows of X, so it is bound by latency, not bandwidth: the chain
// "all workers' codes of step t -> x_{t+1} -> margins -> u -> scale -> codes of step t+1" is strictly
// serial.  Launching kernels per step pays a launch + drain for every link of that chain.  Here the
// grid stays resident for `count` steps (one cluster per worker, one CTA per SM, launched
// cooperatively so that co-residency is guaranteed) and the only grid-wide dependency per step is the
// arrival of the other workers' messages:
//   - every CTA keeps its slice of x and of mu in REGISTERS across steps;
//   - the rows of step t+1 do not depend on step t (sampling is counter-based), so they are sampled
//     and fetched by bulk copies (TMA) into the other half of a double buffer while step t computes;
//     labels and cached snapshot margins of those rows travel in registers of the thread that owns the
//     minibatch slot;
//   - the codes travel between CTAs as self-validating 64-bit words: 32 bits of payload (the codes of 8
//     coordinates, or part of them) and a 32-bit tag that names the step (unique across launches).  Aligned
//     64-bit stores are single-copy atomic, so a reader that sees the tag it expects also sees the payload:
//     no fence, no flag and no block barrier sit between "codes stored" and "codes read".  The scale delta of
//     a worker travels the same way (delta | tag), one word per CTA, and so does the full-precision second
//     estimator of Algorithm 2 (value | tag per coordinate).  At the top of a step every thread loads, for
//     ITS 8 coordinates, the words of all workers (all loads in flight together), repeats until every tag
//     matches, then averages, adds mu and applies the proximal step in registers.  The exchange buffers are
//     double-buffered by step parity, because a fast CTA may store step t+1 while a slow one still reads
//     step t (it cannot get further ahead: storing step t+2 needs every reader's step t+1).
//   - only the last step also writes the packed codes, delta and the second estimator in their documented
//     layouts, for the caller.
// Every wait is bounded; when one runs out the thread records a timeout in the status word, raises a global
// abort flag that makes every other wait return at once, and the loop finishes without hanging (all CTAs
// still execute the same cluster barriers).
//
// The loop body is re-fetched from the instruction cache hierarchy every step, so its size shows up in the
// step latency: the number of 2048-coordinate passes per CTA is a template parameter (no dead second pass)
// and loops are unrolled only as far as instruction-level parallelism needs.
//
// The arithmetic (sampling, margins as balanced-tree sums, u summed in batch order, Eq. 2, the
// quantizer, Eq. 3, the proximal step) is operation for operation that of the per-step kernels.
#include <cooperative_groups.h>

#include "lpc_device.cuh"
#include "lpc_inner.h"

namespace cg = cooperative_groups;

namespace lpc {
namespace {

constexpr int PT = 256;
constexpr int PGROUP = PT * 8;
constexpr int PMAXP = 2;   // passes per CTA: SL <= 4096
constexpr int PMAXB = 64;
constexpr int PMAXCS = 8;
constexpr int PMAXFLAGS = 256;
constexpr int PMAXN = 64;      // workers in the one-launch loop (a lane carries the scales of PMAXN / 32 of them)
constexpr int PUB_STRIDE = 16;  // publication words sit 128 bytes apart: one cache line each

struct PSmem {
  uint64_t bar[2];
  __align__(16) float coef[PMAXB];
  float wpart[PMAXB * PMAXP * 8];
  // cluster exchange slots, written by the peers through distributed shared memory as tagged words, two
  // step-parity halves: margin partial sums (slot b * PMAXCS + rank) and statistics (max, S1, S2 per rank)
  unsigned long long mx[2][PMAXB * PMAXCS];
  unsigned long long sx[2][3 * PMAXCS];
  float ws1[PMAXP * 8], ws2[PMAXP * 8];
  uint32_t wmax[8];
  uint32_t wclip[8];
  Scale scale;
  __align__(16) uint8_t stage[PT * 16];
};

// Tagged 64-bit words (payload | tag << 32): relaxed, device scope, one indivisible access each.
__device__ __forceinline__ unsigned long long ld_word(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_word(unsigned long long* p, uint32_t payload, uint32_t tag) {
  const unsigned long long v = (unsigned long long)payload | ((unsigned long long)tag << 32);
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t word_tag(unsigned long long w) { return (uint32_t)(w >> 32); }
// Two neighbouring tagged words (16-byte aligned) by one vector access: each 64-bit element is still one indivisible
// access that carries its own tag, the pair need not be.
__device__ __forceinline__ void ld_word2(const unsigned long long* p, unsigned long long& w0, unsigned long long& w1) {
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_word2(unsigned long long* p, uint32_t payload0, uint32_t payload1, uint32_t tag) {
  const unsigned long long v0 = (unsigned long long)payload0 | ((unsigned long long)tag << 32);
  const unsigned long long v1 = (unsigned long long)payload1 | ((unsigned long long)tag << 32);
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(v0), "l"(v1) : "memory");
}
// The same kind of word in shared memory: stored into CTA `cta` of the cluster at the address that `slot` has in
// this CTA, read back from this CTA's own shared memory.
__device__ __forceinline__ void st_cluster_word(const unsigned long long* slot, uint32_t cta, uint32_t payload, uint32_t tag) {
  const unsigned long long v = (unsigned long long)payload | ((unsigned long long)tag << 32);
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(slot)), "r"(cta));
  asm volatile("st.relaxed.cluster.shared::cluster.u64 [%0], %1;" ::"r"(remote), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_shared_word(const unsigned long long* slot) {
  unsigned long long v;
  asm volatile("ld.relaxed.cluster.shared::cta.u64 %0, [%1];" : "=l"(v) : "r"(smem_u32(slot)) : "memory");
  return v;
}

__device__ __forceinline__ uint32_t extract_bits(uint64_t lo, uint64_t hi, int pos, int b) {
  uint64_t v;
  if (pos < 64) {
    v = lo >> pos;
    if (pos + b > 64) v |= hi << (64 - pos);
  } else {
    v = hi >> (pos - 64);
  }
  return (uint32_t)v & ((1u << b) - 1u);
}

// Bulky scalar routines that one thread (or B threads) run once per step: kept out of line so that the loop
// body every warp walks through stays small.
__device__ __noinline__ Scale scale_out_of_line(uint32_t max_bits, float S1, float S2, int64_t len, int b, int clip_mode,
                                               float clip_value) {
  return make_scale(max_bits, S1, S2, len, b, clip_mode, clip_value);
}
__device__ __noinline__ float deriv_out_of_line(int loss, float m, float y) { return loss_deriv(loss, m, y); }
__device__ __noinline__ int64_t sample_row_out_of_line(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t slot,
                                                       int64_t lo, int64_t span) {
  const U4 r = stream_block(seed, tag, worker, k, slot);
  return lo + (int64_t)(((uint64_t)r.x * (uint64_t)span) >> 32);
}
__device__ __noinline__ bool spin_expired_out_of_line(uint32_t it, uint64_t& t0, unsigned int* abort_flag, unsigned int* dev_status) {
  return spin_expired(it, t0, abort_flag, dev_status);
}
__device__ __forceinline__ float tree_small(const float* v, int n) {  // n in {1, 2, 4, 8}
  if (n == 1) return v[0];
  if (n == 2) return add_rn(v[0], v[1]);
  if (n == 4) return tree4(v[0], v[1], v[2], v[3]);
  return tree8(v);
}

// Phase timestamps of one CTA for latency studies; compiled in only with -DLPC_TRACE.
#ifdef LPC_TRACE
__device__ unsigned long long g_trace[64 * 16];
#define LPC_TRACE_MARK(i)                                                                   \
  do {                                                                                      \
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0 && t >= 8 && t < 72)         \
      g_trace[(t - 8) * 16 + (i)] = global_ns();                                            \
  } while (0)
#else
#define LPC_TRACE_MARK(i) do { } while (0)
#endif

// A thread's EPT consecutive row values of a slice from shared memory (zero outside the existing columns).
// EPT = 8: a thread's two 16-byte halves are 32 bytes from its neighbour's, so a plain "lower halves, then upper halves"
// pair of loads would hit every bank twice.  Threads with `swz` set (bit 2 of the lane) read their upper half first
// instead: each load then covers 32 distinct banks per quarter warp.  Such a thread gets its values with the halves
// exchanged, v[e] = value of coordinate e ^ 4, and the callers keep their operands in the same order.
template <int EPT>
__device__ __forceinline__ void row_vals(const float* rowp, int off, int width, bool swz, float* v) {
#pragma unroll
  for (int e = 0; e < EPT; ++e) v[e] = 0.f;
  if constexpr (EPT == 8) {  // width is a multiple of 4 and off a multiple of EPT
    const int o0 = off + (swz ? 4 : 0), o1 = off + (swz ? 0 : 4);
    if (o0 < width) {
      const float4 t = *reinterpret_cast<const float4*>(rowp + o0);
      v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    if (o1 < width) {
      const float4 t = *reinterpret_cast<const float4*>(rowp + o1);
      v[4] = t.x; v[5] = t.y; v[6] = t.z; v[7] = t.w;
    }
  } else if (off < width) {
    if constexpr (EPT == 2) {
      const float2 t = *reinterpret_cast<const float2*>(rowp + off);
      v[0] = t.x; v[1] = t.y;
    } else {
      const float4 t = *reinterpret_cast<const float4*>(rowp + off);
      v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
  }
}
// Balanced-tree sum of a thread's EPT consecutive values (the lowest levels of the tree over the coordinate index).
template <int EPT>
__device__ __forceinline__ float tree_ept(const float* v) {
  if constexpr (EPT == 8) return tree8(v);
  else if constexpr (EPT == 4) return tree4(v[0], v[1], v[2], v[3]);
  else return add_rn(v[0], v[1]);
}

// BITS: 1, 2, 4, 8 fixed width; 0: b from the arguments (1..16 or 32).
// NP: passes of PT * EPT coordinates that a CTA makes over its slice (1 or 2).
// EPT: consecutive coordinates a thread owns per pass (8, 4 or 2): slices of 1024 or 512 coordinates still give every
//      thread of the CTA work, which shortens each serial phase of a step; a group of 8 coordinates (one Philox block,
//      one tagged code word for b <= 4) is then shared by 8 / EPT neighbouring lanes.  BITS = 0 and NP = 2 use EPT = 8.
// ALPC: Algorithm 2's step (coupling, double sampling on one more cluster, y/z updates) instead of Algorithm 1's.
template <int BITS, int NP, int EPT, bool ALPC>
__global__ void __launch_bounds__(PT, 1) persist_kernel(PersistArgs pa) {
  static_assert(EPT == 8 || ((EPT == 4 || EPT == 2) && BITS != 0 && NP == 1), "narrow threads: fixed widths, one pass");
  constexpr int PSPAN = PT * EPT;               // coordinates per pass
  constexpr int LPG = 8 / EPT;                  // lanes that share a group of 8 coordinates
  constexpr int TB = EPT * (BITS ? BITS : 1);   // code bits a thread produces per pass (fixed widths)
  const InnerArgs& a = pa.in;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  PSmem& sm = *reinterpret_cast<PSmem*>(smem_raw);
  const int CS = a.CS, SL = a.SL, B = a.B, d = a.d, N = a.N;
  float* rows = reinterpret_cast<float*>(smem_raw + ((sizeof(PSmem) + 15) & ~(size_t)15));  // RS row slots of SL floats

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool swz = (EPT == 8) && ((lane >> 2) & 1);  // this thread reads the halves of its row values exchanged (row_vals)
  const int rank = (int)cluster.block_rank();
  const int worker = blockIdx.y;
  const bool is_J = ALPC && (worker == N);  // the extra cluster that handles the shared batch J
  // Row slots: step t keeps its B rows in slots (t*B + a) % RS.  RS = 2B: all rows of step t+1 are fetched while step
  // t computes.  B <= RS < 2B (the slices of two steps do not fit): the first RS - B rows of step t+1 go into the free
  // slots at the top of step t, the others into the slots that step t gives back once its u is formed.
  const int RS = pa.row_slots;
  const int PA = RS - B;                    // rows of the next step fetched at the top of a step
  const int b = BITS ? BITS : a.b;
  const int c0 = rank * SL;
  const int width = max(0, min(SL, d - c0));
  const float invN = __fdiv_rn(1.0f, (float)N);
  const float invB = __fdiv_rn(1.0f, (float)B);
  const float kappa = mul_rn(pa.eta, pa.lambda_l1);
  const uint32_t zero_code = (b == 1) ? 0u : (1u << (b - 1));
  const uint32_t row_bytes = (uint32_t)width * 4u;

  if (tid == 0) {
    mbar_init(&sm.bar[0], 1);
    mbar_init(&sm.bar[1], 1);
    mbar_fence_init();
  }
  // no exchange slot may look valid before a peer has written it: tags start at 1
  for (int i = tid; i < 2 * PMAXB * PMAXCS; i += PT) (&sm.mx[0][0])[i] = 0ull;
  for (int i = tid; i < 2 * 3 * PMAXCS; i += PT) (&sm.sx[0][0])[i] = 0ull;
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  __syncthreads();

  // Thread a < B owns minibatch slot a.  fetch_rows(t, sb, lo, hi) samples step t's row for the slots lo <= a < hi,
  // starts the bulk copy of this CTA's slice of it into row slot (sb + a) % RS and loads its label and cached
  // snapshot margin into registers (a step ahead, so these loads never stall the step that issues them).  The
  // barrier of step t (bar[t & 1]) gets its one arrival from the call that covers the last slot.
  const int64_t samp_span = (a.sample_global || is_J) ? a.n : a.n / N;  // rows this cluster samples from
  const int64_t samp_lo = (a.sample_global || is_J) ? 0 : (int64_t)worker * samp_span;
  int64_t row_next = 0, row_cur = 0;
  float y_next = 0.f, y_cur = 0.f, ms_next = 0.f, ms_cur = 0.f;
  auto sample_rows = [&](int t, int lo, int hi) {
    if (tid >= lo && tid < hi)
      row_next = sample_row_out_of_line(a.seed, is_J ? TAG_BATCH_J : TAG_BATCH, is_J ? 0u : (uint32_t)worker,
                                        a.k_base + (uint64_t)t, (uint32_t)tid, samp_lo, samp_span);
  };
  auto copy_rows = [&](int t, int sb, int lo, int hi) {  // after sample_rows(t, lo, hi)
    if (hi <= lo) return;
    uint64_t* bar = &sm.bar[t & 1];
    if (tid == 0 && width > 0) {
      const uint32_t bytes = row_bytes * (uint32_t)(hi - lo);
      if (hi == B) mbar_expect_tx(bar, bytes);  // arrives as well: the phase can now complete
      else asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
    }
    if (tid >= lo && tid < hi) {
      int slot = sb + tid;
      if (slot >= RS) slot -= RS;
      if (width > 0) bulk_load(rows + (size_t)slot * SL, a.X + row_next * (int64_t)d + c0, row_bytes, bar);
      y_next = a.y[row_next];
      ms_next = a.margins[row_next];
    }
  };
  auto fetch_rows = [&](int t, int sb, int lo, int hi) {
    sample_rows(t, lo, hi);
    copy_rows(t, sb, lo, hi);
  };

  // this thread's slice of the iterate and of the snapshot gradient stay in registers for the whole loop
  float xr[NP][EPT], mur[NP][EPT];
#pragma unroll
  for (int p = 0; p < NP; ++p) {
    const int off = p * PSPAN + tid * EPT;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const bool in = off + e < width;
      xr[p][e] = in ? a.x[c0 + off + e] : 0.f;
      mur[p][e] = in ? a.mu[c0 + off + e] : 0.f;
    }
  }
  // Algorithm 2 keeps y, z, the running sum of y and the snapshot in registers too; xr is then the coupled point
  float yr[ALPC ? NP : 1][EPT], zr[ALPC ? NP : 1][EPT], sr[ALPC ? NP : 1][EPT], xtr[ALPC ? NP : 1][EPT];
  if constexpr (ALPC) {
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int off = p * PSPAN + tid * EPT;
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const bool in = off + e < width;
        yr[p][e] = in ? pa.y[c0 + off + e] : 0.f;
        zr[p][e] = in ? pa.z[c0 + off + e] : 0.f;
        sr[p][e] = in ? pa.ysum[c0 + off + e] : 0.f;
        xtr[p][e] = in ? pa.xt[c0 + off + e] : 0.f;
      }
    }
  }
  const float tau3 = __fsub_rn(__fsub_rn(1.0f, pa.tau1), pa.tau2);
  const float kappa_y = mul_rn(pa.inv4L, pa.lambda_l1), kappa_z = mul_rn(pa.alpha, pa.lambda_l1);
  if (pa.count > 0) fetch_rows(0, 0, 0, B);
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

  // Every spin in this kernel ends: after about two seconds without progress the thread records a timeout and
  // raises the abort flag, which ends all other spins at their next look at it.
  auto wait_expired = [&](uint32_t it, uint64_t& t0) -> bool {
    if ((it & 63u) != 63u) return false;  // the rare path is out of line: the loop body is fetched anew every step, its size counts
    return spin_expired_out_of_line(it, t0, pa.abort_flag, a.dev_status);
  };

  // Applies step target-1's update to this thread's coordinates:
  //   x <- prox_{eta h}(x - eta (mean_i delta_i k_i + mu))      (Algorithm 2: the y and z updates).
  // The tagged words that hold the thread's codes are loaded for CH workers at a time, all in flight together (one L2
  // round trip), and re-loaded until every tag names step target-1.  The workers' scales are the same for every
  // thread: lane l of a warp loads those of workers l, l + 32, ... and the warp hands them round by shuffles.
  constexpr int WMAX = (BITS == 0) ? 8 : (BITS == 8 ? 2 : 1);  // tagged words per group of 8 coordinates
  constexpr int NW = (BITS == 0) ? 8 : (TB >= 32 ? TB / 32 : 1);  // of which a thread reads / writes this many
  // (A layout with the workers' words of a coordinate group side by side, read two workers per 16-byte load, halves the
  // loads of the update but scatters every worker's stores over lines that the other workers write too: 5.53 against
  // 4.93 us per step on the least-squares workload, 12.5 against 9.9 on the Algorithm 2 workload; dropped.)
  // workers per round of loads: 16 words in flight per thread.  (32 per round for the 32 workers of the Algorithm 2
  // workload moved the second round's time into the first: 40 loads per thread queue up on the way from L2.)
  constexpr int CH = (BITS == 0) ? 4 : 16 / (NP * NW) > 0 ? 16 / (NP * NW) : 1;
  const int wpg = (BITS == 0) ? pa.wpg : WMAX;
  const int sub = (LPG > 1) ? (tid & (LPG - 1)) : 0;          // this thread's place in its group of 8 coordinates
  const int wfirst = (BITS == 0) ? 0 : (sub * TB) >> 5;        // first word of the group that holds its codes
  const int wshift = (BITS == 0) ? 0 : (sub * TB) & 31;        // and their position in it
  const size_t groups = (size_t)(CS * SL) >> 3;
  float wcur = pa.w0;  // snapshot weight of the step whose update comes next
  // `between` runs once, while the first round's loads are in flight.
  auto apply_update = [&](unsigned int target, auto between) {
    const int rpar = (pa.count - (int)target) & 1;  // parity half that holds step target-1
    const uint32_t tag = pa.tag_base + target;
    const unsigned long long good = (unsigned long long)tag << 32;  // stands in for words this thread does not need
    const unsigned long long* dwords = pa.pub + ((size_t)rpar * PMAXFLAGS + rank) * PUB_STRIDE;
    const unsigned long long* ll_in = pa.ll + (size_t)rpar * N * groups * wpg;
    int cc[NP];
    bool act[NP];
    float acc[NP][EPT];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int off = p * PSPAN + tid * EPT;
      cc[p] = c0 + off;
      act[p] = off < SL && cc[p] < d;
#pragma unroll
      for (int e = 0; e < EPT; ++e) acc[p][e] = 0.f;
    }
    unsigned long long cw[CH][NP][NW], vw[ALPC ? NP * EPT : 1], dw;
    // No load is predicated and no round is special (branches and a peeled first round would double the size of this
    // code, and the loop body is fetched anew every step): a thread without coordinates in a pass reads the words of
    // coordinate 0, a round that reaches past the last worker repeats the last one with the scale 0, and lane l of a
    // warp fetches the scale of the round's worker l % CH for the whole warp.
    size_t gq[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) gq[p] = (act[p] ? (size_t)(cc[p] >> 3) : 0) * wpg + wfirst;
    const size_t wstride = groups * wpg;
    auto issue_vhat = [&]() {
      if constexpr (ALPC) {
#pragma unroll
        for (int p = 0; p < NP; ++p)
#pragma unroll
          for (int e = 0; e < EPT; e += 2)  // pairs of neighbouring words by one 16-byte access
            ld_word2(pa.ll_vhat + (size_t)rpar * groups * 8 + (act[p] ? cc[p] : c0) + e, vw[p * EPT + e], vw[p * EPT + e + 1]);
      }
    };
    if constexpr (ALPC) issue_vhat();
#pragma unroll 1
    for (int i0 = 0; i0 < N; i0 += CH) {
      uint64_t t0 = 0;
      const int mine = i0 + (lane & (CH - 1));  // the worker whose scale this lane fetches
#pragma unroll 1
      for (uint32_t it = 0;; ++it) {
        dw = ld_word(dwords + (size_t)min(mine, N - 1) * CS * PUB_STRIDE);
#pragma unroll
        for (int j = 0; j < CH; ++j) {
          const unsigned long long* q = ll_in + (size_t)min(i0 + j, N - 1) * wstride;
#pragma unroll
          for (int p = 0; p < NP; ++p) {
            if constexpr (BITS == 8 && NW == 2) {  // the two words of a group of eight 8-bit codes: one 16-byte load
              ld_word2(q + gq[p], cw[j][p][0], cw[j][p][1]);
            } else {
#pragma unroll
              for (int w = 0; w < NW; ++w) cw[j][p][w] = (w < wpg) ? ld_word(q + gq[p] + w) : good;
            }
          }
        }
        if (i0 == 0 && it == 0) between();
        bool ok = word_tag(dw) == tag;
#pragma unroll
        for (int j = 0; j < CH; ++j)
#pragma unroll
          for (int p = 0; p < NP; ++p)
#pragma unroll
            for (int w = 0; w < NW; ++w) ok = ok && word_tag(cw[j][p][w]) == tag;
#ifdef LPC_TRACE
        if (i0 == 0 && blockIdx.x == 0 && blockIdx.y == 0 && tid == 0 && target >= 8 && target < 72)
          g_trace[(target - 8) * 16 + 15] = it + 1;
#endif
        // the scales are shared by the warp: all lanes go on together
        if (__all_sync(0xFFFFFFFFu, ok) || __any_sync(0xFFFFFFFFu, wait_expired(it, t0))) break;
      }
#ifdef LPC_TRACE
      if (i0 == 0) { const int t = (int)target; LPC_TRACE_MARK(3); }
#endif
      const uint32_t dmine = (mine < N) ? (uint32_t)dw : 0u;
#pragma unroll
      for (int j = 0; j < CH; ++j) {
        const float di = __uint_as_float(__shfl_sync(0xFFFFFFFFu, dmine, j));
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          if (b == 32) {
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
              const float val = (cc[p] + e < d && e < NW) ? __uint_as_float((uint32_t)cw[j][p][e < NW ? e : 0]) : 0.f;
              acc[p][e] = add_rn(acc[p][e], mul_rn(di, val));
            }
          } else {
            uint64_t lo = (uint64_t)(uint32_t)cw[j][p][0], hi = 0;
            if constexpr (NW >= 2) lo |= (uint64_t)(uint32_t)cw[j][p][1] << 32;
            if constexpr (NW >= 4) hi = (uint64_t)(uint32_t)cw[j][p][2] | ((uint64_t)(uint32_t)cw[j][p][3] << 32);
            float kf[8];
            if constexpr (BITS == 0) {
#pragma unroll
              for (int e = 0; e < 8; ++e) kf[e] = index_as_float(extract_bits(lo, hi, e * b, b), b);
            } else {
              // this thread's EPT codes start at bit wshift of the word: decode them as the first codes of a group
              // (the entries past EPT are not used and cost nothing)
              if constexpr (TB < 32) lo = ((uint32_t)lo >> wshift) & ((1u << TB) - 1u);
              decode8<BITS ? BITS : 1>(lo, kf);
            }
#pragma unroll
            for (int e = 0; e < EPT; ++e) acc[p][e] = add_scaled_index<BITS>(acc[p][e], di, kf[e]);
          }
        }
      }
    }
    if constexpr (ALPC) {  // the second estimator's words were requested first: they are here by now
      uint64_t t0 = 0;
#pragma unroll 1
      for (uint32_t it = 0;; ++it) {
        bool ok = true;
#pragma unroll
        for (int e = 0; e < NP * EPT; ++e) ok = ok && word_tag(vw[e]) == tag;
        if (ok || wait_expired(it, t0)) break;
        issue_vhat();
      }
    }
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      if (!act[p]) continue;
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        if (cc[p] + e < d) {
          const float v = add_rn(mul_rn(acc[p][e], invN), mur[p][e]);
          if constexpr (ALPC) {  // steps 12-13 of Algorithm 2
            const float vhat = __uint_as_float((uint32_t)vw[p * EPT + e]);
            yr[p][e] = mul_rn(soft_threshold(__fsub_rn(xr[p][e], mul_rn(pa.inv4L, v)), kappa_y), pa.cy);
            zr[p][e] = mul_rn(soft_threshold(__fsub_rn(zr[p][e], mul_rn(pa.alpha, vhat)), kappa_z), pa.cz);
            sr[p][e] = add_rn(sr[p][e], mul_rn(wcur, yr[p][e]));
          } else {
            xr[p][e] = soft_threshold(__fsub_rn(xr[p][e], mul_rn(pa.eta, v)), kappa);
          }
          if (pa.v_tap && worker == 0) pa.v_tap[cc[p] + e] = v;
        }
      }
    }
    if constexpr (ALPC) wcur = mul_rn(wcur, pa.theta);  // the next step's snapshot weight (Algorithm 2's last step)
  };

  int sb = 0;  // first row slot of the current step, (t * B) % RS
#pragma unroll 1
  for (int t = 0; t <= pa.count; ++t) {  // the pass t = count only applies the last step's update (one copy of that code)
    const uint32_t row_parity = (uint32_t)((t >> 1) & 1);
    const uint64_t k = a.k_base + (uint64_t)t;
    const int wpar = (pa.count - 1 - t) & 1;  // parity half of the exchange buffers this step writes
    const bool last = (t == pa.count - 1);    // the last step also leaves its messages in the documented layouts
    const uint32_t tag = pa.tag_base + (uint32_t)(t + 1);
    uint32_t* out = a.codes + (int64_t)worker * a.stride_words;
    int sb_next = sb + B;
    if (sb_next >= RS) sb_next -= RS;
    LPC_TRACE_MARK(0);
    row_cur = row_next; y_cur = y_next; ms_cur = ms_next;
    // a thread that fetches its row of step t+1 only after u is formed keeps this step's label and margin until then
    const int64_t row_use = row_cur;
    const float y_use = y_cur, ms_use = ms_cur;

    // rounding bits of this step: they depend on the counters only, so they are drawn before the data arrives
    // (with fewer than 8 coordinates per thread the lanes of a group draw the same block and keep their own 16-bit lanes
    // of it in the leading words)
    U4 rnd[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      rnd[p] = stream_block(a.seed, TAG_ROUND, (uint32_t)worker, k, (uint32_t)((c0 + p * PSPAN + tid * EPT) >> 3));
      if constexpr (EPT == 4) {
        if (sub) { rnd[p].x = rnd[p].z; rnd[p].y = rnd[p].w; }
      } else if constexpr (EPT == 2) {
        rnd[p].x = (sub == 0) ? rnd[p].x : (sub == 1) ? rnd[p].y : (sub == 2) ? rnd[p].z : rnd[p].w;
      }
    }
    LPC_TRACE_MARK(1);
    // x_t = prox(x_{t-1} - eta v_{t-1})  (Algorithm 2: y_t, z_t).  The first rows of step t+1 are sampled before the
    // loads of the other workers' words go out and requested while those loads are in flight: issued right at the top
    // of the step the loads arrive before the peers' words and cost a second round trip, issued after the whole row
    // fetch they leave a few hundred nanoseconds unused (measured: 5.35 / 5.14 / 4.97 us per step for loads first /
    // fetch first / this order on the least-squares workload).
    const bool more = t + 1 < pa.count;
    if (more) sample_rows(t + 1, 0, PA);
    LPC_TRACE_MARK(2);
    // The snapshot side of this step's coefficients, l'(m~_a), depends on nothing of this step: the owner of a minibatch
    // slot forms it while the peers' words are on their way (for the logistic loss it is half of the fp64 work).
    float gs_use = 0.f;
    auto ahead = [&] {
      if (more) copy_rows(t + 1, sb_next, 0, PA);
      if (tid < B && t < pa.count) gs_use = deriv_out_of_line(a.loss, ms_use, y_use);
    };
    if (t > 0) apply_update((unsigned int)t, ahead);
    else ahead();
    if (t == pa.count) break;
    if constexpr (ALPC) {  // step 6: x = tau1 z + tau2 x~ + (1 - tau1 - tau2) y
#pragma unroll
      for (int p = 0; p < NP; ++p)
#pragma unroll
        for (int e = 0; e < EPT; ++e)
          xr[p][e] = add_rn(add_rn(mul_rn(pa.tau1, zr[p][e]), mul_rn(pa.tau2, xtr[p][e])), mul_rn(tau3, yr[p][e]));
    }
    LPC_TRACE_MARK(4);

    bool ok = true;
    if (width > 0) ok = mbar_wait(&sm.bar[t & 1], row_parity);
    if (!ok) {
      atomicOr(a.dev_status, DEV_TIMEOUT);
      mbar_wait(&sm.bar[t & 1], row_parity);
    }
    LPC_TRACE_MARK(5);
    auto row_ptr = [&](int r) {  // row r of this step
      int slot = sb + r;
      if (slot >= RS) slot -= RS;
      return rows + (size_t)slot * SL;
    };

    // margins <X_a, x_t>: eight rows at a time; their 8*NP per-thread partial sums are reduced across the
    // warp together by recursive halving (9 or 12 shuffles instead of 5 per value)
    constexpr int RG = 8, NVAL = RG * NP, LOGV = (NP == 2) ? 4 : 3;
    constexpr int KB = (NP != 1) ? 0 : (EPT == 8) ? 8 : 16;  // leading rows of a minibatch that a thread keeps in registers
    float xw[NP][EPT];  // x in the order row_vals delivers the row values
#pragma unroll
    for (int p = 0; p < NP; ++p)
#pragma unroll
      for (int e = 0; e < EPT; ++e) xw[p][e] = (EPT == 8 && swz) ? xr[p][e ^ (EPT / 2)] : xr[p][e];
    // The first KB rows of the minibatch (one pass per CTA) stay in REGISTERS from here to the end of u: those slices
    // are read from shared memory once per step instead of twice, and their part of u needs only the coefficients.
    float rv[KB ? KB : 1][EPT];
    if constexpr (KB > 0) {
#pragma unroll
      for (int g8 = 0; g8 < KB; g8 += RG) {
        if (g8 < B) {
          float sv[RG];
#pragma unroll
          for (int j = 0; j < RG; ++j) {
            float pr[EPT];
            row_vals<EPT>(row_ptr(min(g8 + j, B - 1)), tid * EPT, width, swz, rv[g8 + j]);
#pragma unroll
            for (int e = 0; e < EPT; ++e) pr[e] = mul_rn(rv[g8 + j][e], xw[0][e]);
            sv[j] = tree_ept<EPT>(pr);
          }
          WarpHalving<RG, 0>::run(sv, lane);
          if ((lane >> 3) == 0) {
            const int j = halving_index<3>(lane);
            if (g8 + j < B) sm.wpart[(g8 + j) * NP * 8 + warp] = sv[0];
          }
        }
      }
    }
#pragma unroll 1
    for (int r0 = KB; r0 < B; r0 += RG) {
      float sv[NVAL];
#pragma unroll
      for (int j = 0; j < RG; ++j) {
        const float* rp = row_ptr(min(r0 + j, B - 1));
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          float v[EPT], pr[EPT];
          row_vals<EPT>(rp, p * PSPAN + tid * EPT, width, swz, v);
#pragma unroll
          for (int e = 0; e < EPT; ++e) pr[e] = mul_rn(v[e], xw[p][e]);
          sv[j * NP + p] = tree_ept<EPT>(pr);  // exchanged halves only swap the operands of the tree's last addition
        }
      }
      WarpHalving<NVAL, 0>::run(sv, lane);
      if ((lane >> LOGV) == 0) {
        const int q = halving_index<LOGV>(lane);
        const int j = q / NP, p = q % NP;
        if (r0 + j < B) sm.wpart[((r0 + j) * NP + p) * 8 + warp] = sv[0];
      }
    }
    __syncthreads();
    LPC_TRACE_MARK(6);
    // Cluster exchange of the margin partial sums: every CTA stores its partial sum of row b into slot (b, rank)
    // of every CTA of the cluster, tagged with the step; the owner of row b waits until its slots carry the tag.
    const int xpar = t & 1;
    if (tid < B) {
      float part = tree8(&sm.wpart[tid * NP * 8]);
      if (NP == 2) part = add_rn(part, tree8(&sm.wpart[(tid * NP + 1) * 8]));
      float m = part;
      if (CS > 1) {
        for (int q = 0; q < CS; ++q) st_cluster_word(&sm.mx[xpar][tid * PMAXCS + rank], (uint32_t)q, __float_as_uint(part), tag);
        unsigned long long w[PMAXCS];
        uint64_t t0 = 0;
        for (uint32_t it = 0;; ++it) {
          bool ok = true;
#pragma unroll
          for (int q = 0; q < PMAXCS; ++q) {
            w[q] = ld_shared_word(&sm.mx[xpar][tid * PMAXCS + min(q, CS - 1)]);  // past the cluster: the last rank again, unused
            ok = ok && word_tag(w[q]) == tag;
          }
          if (ok || wait_expired(it, t0)) break;
        }
        float mp[PMAXCS];
#pragma unroll
        for (int q = 0; q < PMAXCS; ++q) mp[q] = __uint_as_float((uint32_t)w[q]);
        m = tree_small(mp, CS);
      }
      LPC_TRACE_MARK(7);
      const float c = __fsub_rn(deriv_out_of_line(a.loss, m, y_use), gs_use);
      sm.coef[tid] = c;
      if (rank == 0 && t == pa.count - 1) {
        if (a.idx_tap) a.idx_tap[(int64_t)worker * B + tid] = row_use;
        if (a.coef_tap) a.coef_tap[(int64_t)worker * B + tid] = c;
      }
    }
    __syncthreads();
    LPC_TRACE_MARK(8);

    // u = (1/B) sum_a c_a X_a: four rows are loaded together, the adds keep batch order
    float u[NP][EPT];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      float uw[EPT];  // in the order row_vals delivers the row values
#pragma unroll
      for (int e = 0; e < EPT; ++e) uw[e] = 0.f;
      if constexpr (KB > 0) {  // the rows kept in registers (NP = 1)
#pragma unroll
        for (int g4 = 0; g4 < KB; g4 += 4) {
          if (g4 < B) {
            const float4 c4 = *reinterpret_cast<const float4*>(&sm.coef[g4]);
            const float cf[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (g4 + j < B) {
#pragma unroll
                for (int e = 0; e < EPT; ++e) uw[e] = add_rn(uw[e], mul_rn(cf[j], rv[g4 + j][e]));
              }
            }
          }
        }
      }
#pragma unroll 1
      for (int r0 = KB; r0 < B; r0 += 4) {
        float v[4][EPT], cf[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = min(r0 + j, B - 1);
          row_vals<EPT>(row_ptr(r), p * PSPAN + tid * EPT, width, swz, v[j]);
          cf[j] = sm.coef[r];
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (r0 + j < B) {
#pragma unroll
            for (int e = 0; e < EPT; ++e) uw[e] = add_rn(uw[e], mul_rn(cf[j], v[j][e]));
          }
        }
      }
#pragma unroll
      for (int e = 0; e < EPT; ++e) u[p][e] = mul_rn((EPT == 8 && swz) ? uw[e ^ (EPT / 2)] : uw[e], invB);
    }
    if (a.u_tap && t == pa.count - 1) {
#pragma unroll
      for (int p = 0; p < NP; ++p) {
        const int off = p * PSPAN + tid * EPT;
#pragma unroll
        for (int e = 0; e < EPT; ++e)
          if (off + e < width) a.u_tap[(int64_t)worker * d + c0 + off + e] = u[p][e];
      }
    }

    LPC_TRACE_MARK(9);
    if (is_J) {
      // double sampling (Algorithm 2 step 11): v^ = u_J + mu in full precision, nothing is quantized or counted
#pragma unroll
      for (int p = 0; p < NP; ++p) {
        const int off = p * PSPAN + tid * EPT;
        if (off < SL) {
          unsigned long long* q = pa.ll_vhat + (size_t)wpar * groups * 8 + c0 + off;
#pragma unroll
          for (int e = 0; e < EPT; e += 2) {
            const float vh0 = add_rn(u[p][e], mur[p][e]), vh1 = add_rn(u[p][e + 1], mur[p][e + 1]);
            st_word2(q + e, __float_as_uint(vh0), __float_as_uint(vh1), tag);
            if (last && off + e < width) pa.vhat[c0 + off + e] = vh0;
            if (last && off + e + 1 < width) pa.vhat[c0 + off + e + 1] = vh1;
          }
        }
      }
    } else {
      // scale (Eq. 2): this thread's and this warp's part of max |u| and of the tree sums
      uint32_t mx = 0;
#pragma unroll
      for (int p = 0; p < NP; ++p) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) mx = max(mx, __float_as_uint(fabsf(u[p][e])));
        if (a.clip_mode == CLIP_STD) {
          float sq[EPT];
#pragma unroll
          for (int e = 0; e < EPT; ++e) sq[e] = mul_rn(u[p][e], u[p][e]);
          float s1 = tree_ept<EPT>(u[p]), s2 = tree_ept<EPT>(sq);
#pragma unroll
          for (int m = 1; m < 32; m <<= 1) {
            s1 = add_rn(s1, __shfl_xor_sync(0xFFFFFFFFu, s1, m));
            s2 = add_rn(s2, __shfl_xor_sync(0xFFFFFFFFu, s2, m));
          }
          if (lane == 0) { sm.ws1[p * 8 + warp] = s1; sm.ws2[p * 8 + warp] = s2; }
        }
      }
      mx = warp_max_u32(mx);
      if (lane == 0) sm.wmax[warp] = mx;
    }
    __syncthreads();  // u is formed everywhere: nobody reads this step's rows any more
    LPC_TRACE_MARK(10);
    if (t + 1 < pa.count) fetch_rows(t + 1, sb_next, PA, B);  // into the slots this step's rows leave free
    if (is_J) {
      sb = sb_next;
      continue;
    }
    if (tid == 0) {
      uint32_t m = 0;
      for (int w = 0; w < 8; ++w) m = max(m, sm.wmax[w]);
      float s1 = 0.f, s2 = 0.f;
      if (a.clip_mode == CLIP_STD) {
        s1 = tree8(sm.ws1);
        s2 = tree8(sm.ws2);
        if (NP == 2) { s1 = add_rn(s1, tree8(sm.ws1 + 8)); s2 = add_rn(s2, tree8(sm.ws2 + 8)); }
      }
      LPC_TRACE_MARK(11);
      float S1 = s1, S2 = s2;
      if (CS > 1) {  // the same exchange for the statistics: (max |u|, S1, S2) of every rank
        for (int q = 0; q < CS; ++q) {
          st_cluster_word(&sm.sx[xpar][0 * PMAXCS + rank], (uint32_t)q, m, tag);
          st_cluster_word(&sm.sx[xpar][1 * PMAXCS + rank], (uint32_t)q, __float_as_uint(s1), tag);
          st_cluster_word(&sm.sx[xpar][2 * PMAXCS + rank], (uint32_t)q, __float_as_uint(s2), tag);
        }
        unsigned long long w[3][PMAXCS];
        uint64_t t0 = 0;
        for (uint32_t it = 0;; ++it) {
          bool ok = true;
#pragma unroll
          for (int j = 0; j < 3; ++j) {
#pragma unroll
            for (int q = 0; q < PMAXCS; ++q) {
              w[j][q] = ld_shared_word(&sm.sx[xpar][j * PMAXCS + min(q, CS - 1)]);  // past the cluster: the last rank again
              ok = ok && word_tag(w[j][q]) == tag;
            }
          }
          if (ok || wait_expired(it, t0)) break;
        }
        float p1[PMAXCS], p2[PMAXCS];
        m = 0;
#pragma unroll
        for (int q = 0; q < PMAXCS; ++q) {
          m = max(m, (uint32_t)w[0][q]);
          p1[q] = __uint_as_float((uint32_t)w[1][q]);
          p2[q] = __uint_as_float((uint32_t)w[2][q]);
        }
        if (a.clip_mode == CLIP_STD) { S1 = tree_small(p1, CS); S2 = tree_small(p2, CS); }
      }
      sm.scale = scale_out_of_line(m, S1, S2, d, b, a.clip_mode, a.clip_value);
      // delta travels as a tagged word, one per CTA: the readers of rank r take every worker's rank-r word
      st_word(pa.pub + ((size_t)wpar * PMAXFLAGS + worker * CS + rank) * PUB_STRIDE, __float_as_uint(sm.scale.delta), tag);
      if (rank == 0) {
        if (last) a.delta[worker] = sm.scale.delta;
        if (sm.scale.flags & 2u) atomicOr(a.dev_status, DEV_NONFINITE);
      }
    }
    __syncthreads();
    const Scale sc = sm.scale;
    LPC_TRACE_MARK(12);
    const bool degenerate = (sc.flags & 1u) != 0;

    // quantize (Section 2.2), pack, and send the codes of each group of 8 coordinates as tagged words
    unsigned long long* ll_out = pa.ll + ((size_t)wpar * N + worker) * groups * wpg;
    uint32_t nclip = 0;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int off = p * PSPAN + tid * EPT;
      const int c = c0 + off;
      const bool mine = off < SL;
      unsigned long long* q = ll_out + (size_t)(c >> 3) * wpg;
      if (b == 32) {
        if (mine) {
#pragma unroll
          for (int e = 0; e < EPT; ++e) {
            float v = u[p][e];
            if (a.clip_mode != CLIP_NONE && c + e < d) {
              if (v > sc.T) { v = sc.T; ++nclip; }
              if (v < -sc.T) { v = -sc.T; ++nclip; }
            }
            const uint32_t bits = (c + e < d) ? __float_as_uint(v) : 0u;
            st_word(q + e, bits, tag);
            if (last && c + e < a.pad_words) out[c + e] = bits;
          }
        }
        continue;
      }
      uint64_t lo = 0, hi = 0;  // this thread's EPT * b code bits
      if (mine && c < d) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
          if (c + e < d) {
            uint32_t code = zero_code;
            if (!degenerate) {
              const uint32_t r16 = lane16(rnd[p], e);
              code = BITS ? quantize_code<BITS ? BITS : 2>(u[p][e], sc.rdelta, r16) : quantize_code_rt(u[p][e], sc.rdelta, r16, b);
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
      if constexpr (BITS == 0 || TB >= 32) {
        // whole words per thread
        if (mine) {
          if constexpr (BITS == 8 && NW == 2) {
            st_word2(q + wfirst, (uint32_t)lo, (uint32_t)(lo >> 32), tag);
          } else {
            st_word(q + wfirst, (uint32_t)lo, tag);
            if (NW >= 2 && wpg >= 2) st_word(q + wfirst + 1, (uint32_t)(lo >> 32), tag);
          }
          if (NW >= 4 && wpg >= 4) {
            st_word(q + 2, (uint32_t)hi, tag);
            st_word(q + 3, (uint32_t)(hi >> 32), tag);
          }
        }
      } else {
        // LPW neighbouring lanes hold one word of the group between them (all lanes shuffle; lanes outside the slice hold zeros)
        constexpr int LPW = (32 / TB < LPG) ? 32 / TB : LPG;
        uint32_t word = (uint32_t)lo;
#pragma unroll
        for (int i = 1; i < LPW; ++i) word |= __shfl_down_sync(0xFFFFFFFFu, (uint32_t)lo, i) << (i * TB);
        if (mine && (lane & (LPW - 1)) == 0) st_word(q + wfirst, word, tag);
      }
      if (!last) continue;
      // the caller's copy of the last messages: the packed little-endian bit stream
      if constexpr (BITS != 0) {
        if constexpr (TB >= 32) {
          const int64_t w = ((int64_t)c * BITS) >> 5;
          if (mine && w < a.pad_words) {
            out[w] = (uint32_t)lo;
            if (TB == 64) out[w + 1] = (uint32_t)(lo >> 32);  // pad_words is a multiple of 4: w + 1 is inside as well
          }
        } else {
          constexpr int LPS = 32 / TB;  // lanes per word of the stream
          uint32_t word = (uint32_t)lo;
#pragma unroll
          for (int i = 1; i < LPS; ++i) word |= __shfl_down_sync(0xFFFFFFFFu, (uint32_t)lo, i) << (i * TB);
          const int64_t w = ((int64_t)c * BITS) >> 5;
          if (mine && (lane & (LPS - 1)) == 0 && w < a.pad_words) out[w] = word;
        }
      } else {
        if (p > 0) __syncthreads();
        for (int i = 0; i < b; ++i)
          sm.stage[tid * b + i] = (uint8_t)((i < 8) ? (lo >> (8 * i)) : (hi >> (8 * (i - 8))));
        __syncthreads();
        const int span = min(PSPAN, SL - p * PSPAN);
        const int64_t w0 = (int64_t)((c0 + p * PSPAN) >> 5) * b;
        const uint32_t* st = reinterpret_cast<const uint32_t*>(sm.stage);
        for (int w = tid; w < (span / 32) * b; w += PT)
          if (w0 + w < a.pad_words) out[w0 + w] = st[w];
      }
    }
    LPC_TRACE_MARK(13);
    if (last) {  // clipped-coordinate count of the last step, for the caller
      nclip = __reduce_add_sync(0xFFFFFFFFu, nclip);
      if (lane == 0) sm.wclip[warp] = nclip;
      __syncthreads();
      if (tid == 0) {
        uint32_t tc = 0;
        for (int w = 0; w < 8; ++w) tc += sm.wclip[w];
        a.clipped_part[worker * PMAXCS + rank] = tc;
      }
    }
    LPC_TRACE_MARK(14);
    sb = sb_next;
  }

  // the slices of the final state go back to memory (worker 0's cluster)
  if (worker == 0) {
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int off = p * PSPAN + tid * EPT;
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        if (off + e < width) {
          pa.x_out[c0 + off + e] = xr[p][e];  // Algorithm 2: the coupled point of the last step
          if constexpr (ALPC) {
            pa.y[c0 + off + e] = yr[p][e];
            pa.z[c0 + off + e] = zr[p][e];
            pa.ysum[c0 + off + e] = sr[p][e];
          }
        }
      }
    }
  }
  cluster.sync();  // no CTA leaves while a peer could still address its shared memory
}

void fill_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int cs, int clusters, size_t smem, cudaStream_t st,
                 bool cooperative) {
  *cfg = cudaLaunchConfig_t{};
  cfg->gridDim = dim3((unsigned)cs, (unsigned)clusters, 1);
  cfg->blockDim = dim3(PT, 1, 1);
  cfg->dynamicSmemBytes = smem;
  cfg->stream = st;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;  // all CTAs co-resident or the launch fails
  attr[1].val.cooperative = 1;
  cfg->attrs = attr;
  cfg->numAttrs = cooperative ? 2 : 1;
}

using PersistKernel = void (*)(PersistArgs);

template <int BITS, bool ALPC>
PersistKernel pick_shape(int np, int ept) {
  if constexpr (BITS != 0) {
    if (np == 1 && ept == 4) return persist_kernel<BITS, 1, 4, ALPC>;
    if (np == 1 && ept == 2) return persist_kernel<BITS, 1, 2, ALPC>;
  }
  return np == 2 ? persist_kernel<BITS, 2, 8, ALPC> : persist_kernel<BITS, 1, 8, ALPC>;
}
template <bool ALPC>
PersistKernel pick_width(int b, int np, int ept) {
  switch (b) {
    case 1: return pick_shape<1, ALPC>(np, ept);
    case 2: return pick_shape<2, ALPC>(np, ept);
    case 4: return pick_shape<4, ALPC>(np, ept);
    case 8: return pick_shape<8, ALPC>(np, ept);
    default: return pick_shape<0, ALPC>(np, ept);
  }
}
// The instantiation for code width b, slice SL and algorithm.
PersistKernel pick_kernel(int b, int SL, bool alpc) {
  const int ept = persist_coords_per_thread(b, SL);
  const int np = (SL > PT * ept) ? 2 : 1;
  return alpc ? pick_width<true>(b, np, ept) : pick_width<false>(b, np, ept);
}

int max_clusters(PersistKernel k, int cs, size_t smem) {
  if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  fill_config(&cfg, attr, cs, 1, smem, nullptr, false);
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, k, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

}  // namespace

// Coordinates a thread owns per pass (see the kernel's EPT).
int persist_coords_per_thread(int b, int SL) {
  const bool fixed = (b == 1 || b == 2 || b == 4 || b == 8);
  if (!fixed || SL >= PT * 8) return 8;
  return (SL >= PT * 4) ? 4 : 2;
}

// Cluster size, slice and row buffering for the persistent loop.  All clusters (N, plus one for the shared
// batch J in Algorithm 2) must be co-resident -- the occupancy query says how many clusters of a given size the
// device can hold -- and the B row slices of a step must fit in shared memory; with room for 2B slices the rows of
// the next step are fetched while this one computes, with less the part that fits is fetched then and the rest as
// soon as u is formed.  Among the sizes that fit, the largest cluster whose slices still keep a CTA busy wins: more
// CTAs per worker shorten every serial phase of a step.
bool persist_plan(int d, int N, int B, int b, int alpc, int want_cs, int max_smem, int* CS_out, int* SL_out,
                  size_t* smem_out, int* row_slots_out) {
  int P = 1;
  while (P < d) P <<= 1;
  if (P < 32) P = 32;
  const int clusters = N + (alpc ? 1 : 0);
  if (B > PMAXB || N > PMAXN || clusters > PMAXFLAGS) return false;
  bool found = false;
  for (int cs = 1; cs <= PMAXCS; cs <<= 1) {
    if (want_cs > 0 && cs != want_cs) continue;
    const int SL = P / cs;
    if (SL < 32) break;
    if (SL > PGROUP * PMAXP) continue;
    if (clusters * cs > PMAXFLAGS) break;
    const size_t fixed = (sizeof(PSmem) + 15) & ~(size_t)15;
    const size_t one = (size_t)SL * 4;  // one row slot
    if (fixed + (size_t)B * one > (size_t)max_smem) continue;
    int slots = (int)(((size_t)max_smem - fixed) / one);
    if (slots > 2 * B) slots = 2 * B;
    const size_t smem = fixed + (size_t)slots * one;
    if (max_clusters(pick_kernel(b, SL, alpc != 0), cs, smem) < clusters) continue;
    *CS_out = cs; *SL_out = SL; *smem_out = smem; *row_slots_out = slots;
    found = true;
    if (want_cs > 0) break;
    // (512 threads per CTA with half the coordinates per thread were tried as well: 5.53 against 4.92 us per step on the
    // least-squares workload, 11.7 against 10.15 on the Algorithm 2 workload at b = 2 -- sixteen-warp block barriers and
    // half as many words in flight per thread cost more than the shorter per-thread phases gain)
    // (eight-CTA clusters of narrow-thread variants squeezed two to an SM were tried for the 16-worker least-squares
    // workload: 5.8 us per step against 5.06 with four-CTA clusters -- more peers per exchange, polls that come too early)
    if (SL <= 512) break;  // slices below 512 coordinates leave most of a CTA idle
  }
  return found;
}

cudaError_t launch_persist(const PersistArgs& pa, size_t smem, cudaStream_t st, bool cooperative) {
  PersistKernel k = pick_kernel(pa.in.b, pa.in.SL, pa.alpc != 0);
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  fill_config(&cfg, attr, pa.in.CS, pa.in.N + (pa.alpc ? 1 : 0), smem, st, cooperative);
  return cudaLaunchKernelEx(&cfg, k, pa);
}

namespace {
// Exercises the two kinds of bounded wait of the library on things that never happen: thread 0 waits on an mbarrier
// that nobody arrives at and no copy counts on, thread 32 polls a tagged word for a tag that is never handed out.
// Both give up after limit_ns, record DEV_TIMEOUT and return; nothing is in flight, so the kernel simply ends.
__global__ void __launch_bounds__(64) wait_timeout_kernel(const unsigned long long* word, unsigned int* abort_flag,
                                                          unsigned int* dev_status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
    if (!mbar_wait(&bar, 0, limit_ns)) atomicOr(dev_status, DEV_TIMEOUT);
  } else if (threadIdx.x == 32 && word != nullptr) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
      if (word_tag(ld_word(word)) == 0xFFFFFFFFu) break;  // tags stop short of this value
      if (spin_expired(it, t0, abort_flag, dev_status, limit_ns)) break;
    }
  }
}
}  // namespace

cudaError_t launch_wait_timeout(const unsigned long long* word, unsigned int* abort_flag, unsigned int* dev_status,
                                uint64_t limit_ns, cudaStream_t st) {
  wait_timeout_kernel<<<1, 64, 0, st>>>(word, abort_flag, dev_status, limit_ns);
  return cudaGetLastError();
}

#ifdef LPC_TRACE
extern "C" int lpc_trace_read(unsigned long long* host_out) {
  return cudaMemcpyFromSymbol(host_out, g_trace, sizeof(g_trace)) == cudaSuccess ? 0 : -4;
}
#endif

}  // namespace lpc
