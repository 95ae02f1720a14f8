/*
 * lpc.h -- C ABI of the B200 (sm_100a) implementation of the per-iteration path of LPC-SVRG and
 * ALPC-SVRG (arXiv 1901.08924, "Exploring Fast and Communication-Efficient Algorithms in
 * Large-scale Distributed Networks").
 *
 * The library solves  min_x P(x) = (1/n) sum_a loss(<X_a,x>, y_a) + lambda_l1*||x||_1  (Eq. 1) with
 * N data-parallel workers simulated on one GPU as contiguous row partitions of X.  What the
 * workers would transmit is produced bit for bit (b-bit codes plus one float per message) and
 * counted, never sent.
 *
 * Conventions
 *  - Every function returns an int status: LPC_OK or a negative LPC_ERR_* value.  Nothing throws
 *    or aborts.  lpc_last_error() gives a text for the last failure of a context.
 *  - Unless a parameter says "host", array arguments are DEVICE pointers owned by the caller.
 *    The library never frees or reallocates them.  They must be 16-byte aligned, fp32 data must
 *    be finite.  X is row-major, contiguous, leading dimension d, and d must be a multiple of 4.
 *  - Work is enqueued on the cudaStream_t given to lpc_init (passed as void*); calls return
 *    without waiting unless they hand back a host scalar (said per call).  Device-side problems
 *    (non-finite input, a bounded wait that ran out) are recorded in the context and reported by
 *    the next lpc_sync_status().
 *  - A context may be used by one host thread at a time.
 *
 * Packed message layout (part of the ABI).  Coordinate j of a vector of length len has the
 * b-bit code  c_j = k_j + 2^(b-1)  where k_j in [-2^(b-1), 2^(b-1)-1] is its index in the codebook
 * dom(delta,b) of Section 2.2 (b = 1: c_j in {0,1} for the two points -T,+T; b = 32: the IEEE bits
 * of the number).  Codes form a little-endian bit stream: c_j occupies stream bits [j*b,(j+1)*b),
 * stream bit p is bit p%32 of 32-bit word p/32; unused tail bits are zero.  A message is that
 * stream plus the float delta: 32 + b*len bits (Section 3.2).  In memory, worker i's stream for
 * segment s starts at word  i*stride_words + word_offset[s], both multiples of 4 words
 * (lpc_packed_layout); delta is stored at delta[i*nseg + s].
 */
#ifndef LPC_H_
#define LPC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lpc_ctx lpc_ctx;

/* status codes */
#define LPC_OK 0
#define LPC_ERR_INVALID_ARG (-1)
#define LPC_ERR_UNSUPPORTED (-2)
#define LPC_ERR_NONFINITE (-3) /* a NaN or Inf reached the quantizer */
#define LPC_ERR_CUDA (-4)
#define LPC_ERR_TIMEOUT (-5) /* a bounded device-side wait ran out */

/* loss of the linear model, f_a(x) = loss(<X_a,x>, y_a) (Section 5.1: regression and logistic models) */
#define LPC_LOGISTIC 0      /* log(1 + exp(-y m)), y in {-1,+1} */
#define LPC_LEAST_SQUARES 1 /* (m - y)^2 / 2 */

/* clip rule: the threshold T of Eq. 2, delta = T / (2^(b-1) - 1) */
#define LPC_CLIP_NONE 0   /* T = ||u||_inf                    (Eq. 2 with lambda = 1, unbiased) */
#define LPC_CLIP_LAMBDA 1 /* T = clip_value * ||u||_inf       (Eq. 2, clip_value = lambda in (0,1]) */
#define LPC_CLIP_STD 2    /* T = min(clip_value * std(u), ||u||_inf)  (the [-c sigma, c sigma] region of Section 3.1) */

/* buffers of a context that lpc_get_buffer / lpc_set_buffer can copy (device to device) */
#define LPC_BUF_X 0        /* fp32[d]   current iterate x_t (ALPC: x_{k+1} of the last step) */
#define LPC_BUF_XTILDE 1   /* fp32[d]   snapshot */
#define LPC_BUF_MU 2       /* fp32[d]   grad f(snapshot) */
#define LPC_BUF_MARGINS 3  /* fp32[n]   <X_a, snapshot> */
#define LPC_BUF_Y 4        /* fp32[d]   ALPC y_k */
#define LPC_BUF_Z 5        /* fp32[d]   ALPC z_k */
#define LPC_BUF_YSUM 6     /* fp32[d]   ALPC running sum of y over the epoch */
#define LPC_BUF_CODES 7    /* u32[N*stride_words] packed messages of the last step */
#define LPC_BUF_DELTA 8    /* fp32[N]   their scales */
#define LPC_BUF_CLIPPED 9  /* u32[N]    d_lambda^i: coordinates outside the codebook's hull (Lemma 2) */
#define LPC_BUF_BATCH_IDX 10 /* i64[(N+1)*B] sampled rows of the last step; the last B are ALPC's shared batch J */
#define LPC_BUF_COEF 11    /* fp32[(N+1)*B] l'(m(x)) - l'(m(snapshot)) of those rows */
#define LPC_BUF_U 12       /* fp32[N*d] the unquantized worker differences u^i (only while the tap is on) */
#define LPC_BUF_V 13       /* fp32[d]   v of the last step (only while the tap is on) */
#define LPC_BUF_VHAT 14    /* fp32[d]   ALPC full-precision estimator of the last step */

/* options for lpc_set_option */
#define LPC_OPT_SAMPLE_GLOBAL 0 /* 0 (default): worker i samples its own block of n/N rows; 1: all n rows (the paper's shared-storage setting, Section 2.1) */
#define LPC_OPT_TAP_U 1         /* 1: inner steps also store u^i and v for inspection (slower) */
#define LPC_OPT_CLUSTER_SIZE 2  /* thread-block cluster size per worker for the fused step: 0 = automatic, else 1, 2, 4 or 8 */
#define LPC_OPT_USE_GRAPH 3     /* 1 (default): lpc_inner_steps replays a CUDA graph; 0: plain launches */
#define LPC_OPT_PROFILE 4       /* 1: record CUDA events around every kernel launch (graph replay is off meanwhile) */

#define LPC_OPT_SHARED_SCALE 6  /* 1: lpc_quantize_pack gives every worker the unified scale delta_t = max_i delta_t^i of the parameter-server schemes (b), (c) of Section 3.2; needs b in 2..16 */
#define LPC_OPT_AVERAGE_DIVISOR 7 /* lpc_unpack_average_prox (and only it: the training loops always average over N) divides the decoded sum by this count instead of the context's N (0 = N): the worker count behind a server's sum stream */
#define LPC_OPT_PERSISTENT 5    /* 1 (default): lpc_inner_steps runs the whole loop in one cooperative launch when it fits */
#define LPC_OPT_ONE_LAUNCH_QUANTIZE 8 /* 1 (default): lpc_quantize_pack uses one cooperative launch for inputs of at most LPC_ONE_LAUNCH_BYTES */
#define LPC_ONE_LAUNCH_BYTES (48ll << 20)
#define LPC_OPT_LOOP_COOPERATIVE 9 /* 1 (default): the one-launch loops are cooperative launches (the driver guarantees that all their CTAs are resident together, which they rely on).  0: a plain cluster launch of the same grid, for profilers that cannot replay a cooperative cluster launch; use it only on a GPU that runs nothing else (the launch plan has checked that all clusters fit, and every wait in the kernel is bounded, so a grid that is not resident together ends with LPC_ERR_TIMEOUT instead of hanging) */

/* kernel classes reported by lpc_get_profile */
#define LPC_KERNEL_SNAPSHOT 0    /* the pass over X of lpc_snapshot_full_grad / lpc_objective */
#define LPC_KERNEL_WORKER 1      /* fused sampling + SVRG difference + scale + quantize + pack */
#define LPC_KERNEL_AGGREGATE 2   /* unpack + average + proximal step (or ALPC y/z updates) */
#define LPC_KERNEL_QUANT_STATS 3 /* first pass of lpc_quantize_pack (max, sums) */
#define LPC_KERNEL_QUANT_PACK 4  /* second pass of lpc_quantize_pack (quantize + pack) */
#define LPC_KERNEL_OTHER 5       /* small helper kernels */
#define LPC_KERNEL_INNER_LOOP 6  /* the persistent kernel that runs all steps of one lpc_inner_steps call */
#define LPC_KERNEL_QUANT_FUSED 7 /* lpc_quantize_pack in one launch (vectors that stay in L2 between its two passes) */
#define LPC_KERNEL_KINDS 8

/*
 * Creates a context for problem (1).  Section 1 "Contribution" (Eq. 1), Section 2.1 (N workers),
 * Algorithm 1's inputs.
 *   X        n x d, row-major (may be NULL with n = 0 for a quantizer-only context; then only
 *            lpc_quantize_pack, lpc_unpack_average_prox and the sizing helpers may be called and d is
 *            ignored)
 *   y        n labels / targets
 *   n        rows; must be a multiple of N.  Worker i owns rows [i*n/N, (i+1)*n/N).
 *   d        features, multiple of 4, at most 16384
 *   N        simulated workers, 1..1024;  B minibatch size per worker, 1..1024 (up to 64 rows per worker stay
 *            resident on chip; the one-launch loops are available for N <= 64 and B <= 64 when all worker
 *            clusters fit on the device together; larger minibatches stream through the per-step kernel)
 *   b        bits per coordinate: 1..16 or 32 (32 = full precision, the codes are the floats)
 *   seed     key of every random stream (minibatches, shared batch J, stochastic rounding)
 *   stream   cudaStream_t (NULL = default stream)
 * The iterate starts at zero.  Scratch memory is allocated here and freed by lpc_destroy.
 */
int lpc_init(lpc_ctx** out, const float* X, const float* y, int64_t n, int32_t d, int loss,
             float lambda_l1, int32_t N, int32_t B, int32_t b, int clip_mode, float clip_value,
             uint64_t seed, void* stream);
int lpc_destroy(lpc_ctx* ctx);
int lpc_set_option(lpc_ctx* ctx, int option, int64_t value);
const char* lpc_last_error(const lpc_ctx* ctx);

/* Waits for the stream and returns the first device-side error recorded since the last call
 * (LPC_ERR_NONFINITE, LPC_ERR_TIMEOUT, LPC_ERR_CUDA) or LPC_OK.  Host-synchronous. */
int lpc_sync_status(lpc_ctx* ctx);

/* Copies a context buffer (LPC_BUF_*) to / from caller memory on the stream; `bytes` must not
 * exceed the buffer's size.  Setting XTILDE, MU and MARGINS together replaces the snapshot state;
 * the counter-based random streams carry no state, so copying X (or Y, Z, YSUM), XTILDE, MU and
 * MARGINS and re-using the same iteration numbers resumes a run exactly. */
int lpc_get_buffer(lpc_ctx* ctx, int which, void* dst, size_t bytes);
int lpc_set_buffer(lpc_ctx* ctx, int which, const void* src, size_t bytes);
int lpc_set_iterate(lpc_ctx* ctx, const float* x); /* same as lpc_set_buffer(LPC_BUF_X) with d floats */
int lpc_get_iterate(lpc_ctx* ctx, float* x_out);

/*
 * Communication step 1 (Algorithm 1 step 4, Algorithm 2 step 3): makes the current iterate the
 * snapshot and computes mu = grad f(snapshot) = (1/n) sum_a l'(<X_a,x~>,y_a) X_a in ONE pass over X,
 * keeping the margins <X_a,x~> for the inner steps.  Counts 32*d*N*(N-1) step-1 bits.
 *   mu_out      nullable, receives mu (d floats)
 *   f_snapshot  nullable HOST pointer, receives f(snapshot); when given, the call waits for the
 *               stream.
 */
int lpc_snapshot_full_grad(lpc_ctx* ctx, float* mu_out, double* f_snapshot);

/*
 * One inner iteration of Algorithm 1 (steps 6-10) for all N workers, scheme (a) (Eq. 3):
 * worker i samples B rows (with replacement), forms u^i = (1/B) sum_a [grad f_a(x) - grad f_a(x~)],
 * quantizes it with its own delta (Eq. 2) and packs it; then all messages are decoded, averaged,
 * mu is added and x <- prox_{eta h}(x - eta v).  u^i is never written to memory unless the tap is on.
 *   k  global iteration number s*m + t; it keys the random streams.
 * Counts (32 + b*d)*N*(N-1) step-2 bits (Table 1, broadcast).
 */
int lpc_inner_step(lpc_ctx* ctx, float eta, uint64_t k);
/* `count` consecutive inner steps k0, k0+1, ... replayed from a captured CUDA graph. */
int lpc_inner_steps(lpc_ctx* ctx, float eta, uint64_t k0, int64_t count);

/*
 * Packed layout of a (segmented) vector: word_offsets_out[s] (nseg+1 host entries, nullable) is
 * where segment s starts inside a worker's stream, *stride_words_out the distance between
 * workers' streams, both in 32-bit words and multiples of 4.  seg_offsets: host, nseg+1 element
 * offsets with seg_offsets[0] = 0 and seg_offsets[nseg] = len, or NULL for one segment.
 */
int lpc_packed_layout(int64_t len, int32_t b, const int64_t* seg_offsets, int32_t nseg,
                      int64_t* word_offsets_out, int64_t* stride_words_out);
int lpc_packed_words(int64_t len, int32_t b, int64_t* words_out); /* ceil(len*b/32) */

/*
 * Quantization step (Algorithm 1 step 7; Section 2.2, Eq. 2) of N worker vectors, optionally
 * per tensor segment (each segment gets its own delta, as in layer-wise use), then packing.
 *   U          N x len fp32, row stride ld (elements, multiple of 4)
 *   U_sub      nullable, same shape: when given the quantized vector is U - U_sub (the SVRG
 *              difference of a current and a snapshot gradient), formed on the fly
 *   seg_offsets, nseg   as in lpc_packed_layout (host)
 *   k          iteration number keying the rounding stream
 *   codes_out  N * stride_words words, stride from lpc_packed_layout
 *   delta_out  N * nseg floats
 *   clipped_out nullable, N * nseg counts of coordinates outside the hull
 * Vectors longer than L2 are read twice (once for ||u||_inf and the variance, once to quantize) by three launches;
 * when all N vectors together take at most LPC_ONE_LAUNCH_BYTES the call is ONE cooperative launch whose second look at
 * the values is served by L2 (LPC_OPT_ONE_LAUNCH_QUANTIZE = 0 switches that off).  Same codes either way.
 * N, b and the clip rule come from the context.
 */
int lpc_quantize_pack(lpc_ctx* ctx, const float* U, const float* U_sub, int64_t len, int64_t ld,
                      const int64_t* seg_offsets, int32_t nseg, uint64_t k, uint32_t* codes_out,
                      float* delta_out, uint32_t* clipped_out);

/*
 * Communication step 2 under scheme (a) and Algorithm 1 steps 9-10: decode every worker's message
 * with its own delta, average (Eq. 3), v = u~ + mu, x <- soft-threshold(x - eta v, eta*lambda_l1)
 * (the proximal operator of Section 2.3 for h = lambda_l1*||.||_1).
 *   mu nullable (= 0);  x_inout len floats, updated in place;  v_out nullable, receives v.
 */
int lpc_unpack_average_prox(lpc_ctx* ctx, const uint32_t* codes, const float* delta, int64_t len,
                            const int64_t* seg_offsets, int32_t nseg, const float* mu,
                            float* x_inout, float eta, float lambda_l1, float* v_out);

/*
 * The parameter-server schemes (b) and (c) of "Communication step 2" (Section 3.2, Table 1).  Both first unify the
 * scale: with LPC_OPT_SHARED_SCALE set, lpc_quantize_pack quantizes every worker's vector with
 * delta_t = max_i delta_t^i (per tensor segment) and writes that value to all N rows of delta_out.
 *
 * lpc_server_reduce is the server.  codes: the N streams that lpc_quantize_pack wrote (device, layout of
 * lpc_packed_layout for the context's b).  codes_out: ONE stream (device, 16-byte aligned), laid out by
 * lpc_packed_layout for the output width:
 *   LPC_SCHEME_SERVER_SUM        scheme (b): the sums K_j = sum_i k_ij of the signed grid indices, stored like codes
 *                                in offset binary with b + ceil(log2 N) bits (lpc_sum_bits), nothing lost;
 *   LPC_SCHEME_SERVER_REQUANTIZE scheme (c), Eq. 4: the average K_j / N rounded back to the b-bit grid by rule (1) of
 *                                Section 2.2 with the server's own rounding stream keyed by (seed, k); b bits.
 * A worker then decodes the server's stream with lpc_unpack_average_prox on a context made for ONE stream of the
 * output width, passing one row of delta_out; under scheme (b) that context has LPC_OPT_AVERAGE_DIVISOR = N, so
 * that u~_j = (delta_t * K_j) / N (Eq. 3 with a common scale).
 * Counts N*(64 + b*d + b_out*d) step-2 bits per segment (Table 1: N(64 + 2bd + d ceil(log N)) and N(64 + 2bd)).
 * Errors: LPC_ERR_UNSUPPORTED for b = 1 or 32 (no integer grid to add on) and when b + ceil(log2 N) > 16.
 * lpc_scheme_bits evaluates Table 1's three formulas for one step (host only).
 */
#define LPC_SCHEME_BROADCAST 0
#define LPC_SCHEME_SERVER_SUM 1
#define LPC_SCHEME_SERVER_REQUANTIZE 2
int lpc_server_reduce(lpc_ctx* ctx, const uint32_t* codes, int64_t len, const int64_t* seg_offsets, int32_t nseg,
                      int scheme, uint64_t k, uint32_t* codes_out);
int lpc_sum_bits(int32_t b, int32_t N, int32_t* bits_out); /* b + ceil(log2 N) */
int lpc_scheme_bits(int scheme, int64_t d, int32_t b, int32_t N, uint64_t* bits_out);

/*
 * Entropy-coding count (Section 5.1: the experiments pass the codes through Huffman's code before sending them; the
 * paper gives no format, so the payload is counted and no bit stream is produced).  For every message, i.e. every
 * (worker, tensor segment) pair of the N streams in `codes` (device, layout of lpc_packed_layout for the context's
 * b, as written by lpc_quantize_pack):
 *   hist_dev          device, N * nseg * 2^b 64-bit counts, cleared and filled by the call:
 *                     hist_dev[(worker * nseg + seg) * 2^b + code] = coordinates of that message with that code;
 *   entropy_bits_out  host, N * nseg doubles, nullable: n * H = -sum_c count_c log2(count_c / n), the bound no
 *                     symbol code can beat;
 *   huffman_bits_out  host, N * nseg, nullable: sum_c count_c * len_c under Huffman's code for that histogram (one
 *                     bit per coordinate when a message holds a single value).
 * Neither count includes the code table or the 32-bit scale; compare with the raw b * len of Section 3.2.
 * With both host outputs NULL the call only enqueues the histogram; otherwise it waits for the stream and does the
 * two sums on the host.  Errors: LPC_ERR_UNSUPPORTED unless 1 <= b <= 8.
 */
int lpc_message_entropy(lpc_ctx* ctx, const uint32_t* codes, int64_t len, const int64_t* seg_offsets, int32_t nseg,
                        unsigned long long* hist_dev, double* entropy_bits_out, uint64_t* huffman_bits_out);

/*
 * ALPC-SVRG (Algorithms 2 and 3).  lpc_alpc_begin sets y_0 = z_0 = x and clears the y sum.
 * lpc_alpc_double_sample_step is steps 5-13 of Algorithm 2 for iteration k:
 *   x = tau1*z + tau2*x~ + (1-tau1-tau2)*y;  v from quantized worker differences at x (as in
 *   Algorithm 1);  v^ = (1/B) sum_{j in J}[grad f_j(x) - grad f_j(x~)] + mu on ONE shared batch J drawn
 *   from all n rows, in full precision, nothing transmitted ("double sampling");
 *   y <- soft(x - inv4L*v, inv4L*lambda_l1);  z <- soft(z - alpha*v^, alpha*lambda_l1);  ysum += y.
 * lpc_alpc_end_epoch(m) is Algorithm 3 step 5: x~ candidate = ysum/m becomes the current iterate
 * (call lpc_snapshot_full_grad next) and ysum is cleared; y and z carry over.
 */
int lpc_alpc_begin(lpc_ctx* ctx);
int lpc_alpc_double_sample_step(lpc_ctx* ctx, float tau1, float tau2, float alpha, float inv4L, uint64_t k);
int lpc_alpc_double_sample_steps(lpc_ctx* ctx, float tau1, float tau2, float alpha, float inv4L,
                                 uint64_t k0, int64_t count);
int lpc_alpc_end_epoch(lpc_ctx* ctx, int64_t m);

/*
 * The strongly convex case of ALPC-SVRG (Algorithm 2 as printed, Theorem 3): h(x) = lambda_l1*||x||_1 +
 * (sigma/2)*||x||^2 with sigma > 0.  After this call lpc_alpc_double_sample_step(s) solve the two argmins of steps
 * 12-13 for that h -- the soft-threshold results divided by (1 + sigma/(4L)) and by (1 + alpha*sigma) -- and weigh the
 * y iterate of step t of an epoch by (1 + alpha*sigma)^t (formed by repeated fp32 multiplication on the host);
 * lpc_alpc_end_epoch then takes Algorithm 2's weighted mean instead of Algorithm 3's plain mean, and lpc_objective
 * adds (sigma/2)*||x||^2.  tau1, tau2 and alpha stay the caller's (the theorem's choice: tau1 = sqrt(m sigma/(6L)),
 * alpha = 1/(6 tau1 L)).  lpc_alpc_double_sample_steps runs them in the one-launch loop like the general convex case (each
 * CTA forms the weights of its steps itself); where that loop is not available they run as plain per-step launches,
 * without graph replay, because the weight is a launch argument that changes from step to step.  sigma = 0 restores the general convex case (bit-identical to never having called this).
 * Algorithm 1's proximal step (lpc_inner_step, lpc_unpack_average_prox) keeps h = lambda_l1*||.||_1.
 * lpc_alpc_begin and lpc_alpc_end_epoch restart the weights.  Errors: LPC_ERR_INVALID_ARG for sigma < 0 or not finite.
 */
int lpc_set_strong_convexity(lpc_ctx* ctx, float sigma);

/* P(x) = f(x) + lambda_l1*||x||_1 (Eq. 1) in one pass over X.  x nullable (= current iterate);
 * P_out is a HOST pointer; the call waits for the stream. */
int lpc_objective(lpc_ctx* ctx, const float* x, double* P_out);

/* Launch-plan facts of a context (host scalars): what = LPC_INFO_*. */
#define LPC_INFO_STEP_CLUSTER_SIZE 0       /* CTAs per worker cluster of the per-step kernel (0: d too large) */
#define LPC_INFO_LOOP_CLUSTER_SIZE 1       /* CTAs per worker cluster of the one-launch inner loop (0: not available) */
#define LPC_INFO_LOOP_LAUNCHES 2           /* lpc_inner_steps calls served by the one-launch inner loop so far */
#define LPC_INFO_SNAPSHOT_ROWS_PER_TILE 3  /* rows per shared-memory stage of the snapshot pass */
#define LPC_INFO_SNAPSHOT_STAGES 4         /* shared-memory stages of the snapshot pass */
#define LPC_INFO_ALPC_LOOP_CLUSTER_SIZE 5  /* as LOOP_CLUSTER_SIZE, for the one-launch loop of Algorithm 2 */
#define LPC_INFO_LOOP_ROW_SLOTS 6          /* shared-memory slots for sampled-row slices per CTA of the one-launch loop: between B
                                              (a step's rows are fetched once the step before has formed its u) and 2B (all of them
                                              are fetched a whole step ahead); 0: loop not available */
#define LPC_INFO_ALPC_LOOP_ROW_SLOTS 7     /* the same for the loop of Algorithm 2 */
#define LPC_INFO_STEP_RING_STAGES 8        /* per-step kernel: 0 = minibatch rows resident on chip, else ring stages they stream through */
#define LPC_INFO_LOOP_COORDS_PER_THREAD 11  /* one-launch loop: consecutive coordinates a thread owns (8, 4 or 2; 0: not available) */
#define LPC_INFO_ALPC_LOOP_COORDS_PER_THREAD 12
#define LPC_INFO_QUANT_ONE_LAUNCH 13        /* last lpc_quantize_pack: 1 when it ran as one cooperative launch */
#define LPC_INFO_AGGREGATE_SPLIT 9         /* last lpc_unpack_average_prox: CTAs that shared one tile of 8192 coordinates (1, 2 or 4) */
#define LPC_INFO_QUANT_PIPELINED_RUNS 10   /* last lpc_quantize_pack: runs of 8 tiles per worker that were whole tiles of one segment and
                                              so took the second pass's software-pipelined loop (unless that worker's scale was
                                              degenerate); 0 unless every worker's vector starts on a 16-byte boundary (ld % 4 == 0) */
int lpc_query(const lpc_ctx* ctx, int what, int64_t* out);

/* Per-kernel device time measured with CUDA events on the context's stream while LPC_OPT_PROFILE is
 * on: ms_out[kind] total milliseconds, launches_out[kind] launches (both HOST arrays of
 * LPC_KERNEL_KINDS entries, nullable).  reset != 0 clears the totals.  Host-synchronous. */
int lpc_get_profile(lpc_ctx* ctx, double* ms_out, int64_t* launches_out, int32_t reset);

/* Bits that the simulated workers would have transmitted so far (host counters): step 1 =
 * 32*d*N*(N-1) per snapshot, step 2 = (32+b*len)*N*(N-1) per inner step or quantize call (Table 1). */
int lpc_comm_bits(const lpc_ctx* ctx, uint64_t* step1_bits, uint64_t* step2_bits);

/*
 * The whole LPC-SVRG job from HOST buffers, for callers without device memory of their own:
 * copies X and y to the device, runs S epochs of m inner steps of Algorithm 1 from x_host_inout,
 * copies the final snapshot back and returns P at it.  All pointers are host pointers
 * (pinned memory makes the copies faster).  Host-synchronous.
 */
int lpc_svrg_run_host(const float* X_host, const float* y_host, int64_t n, int32_t d, int loss,
                      float lambda_l1, int32_t N, int32_t B, int32_t b, int clip_mode, float clip_value,
                      uint64_t seed, int32_t S, int64_t m, float eta, float* x_host_inout,
                      double* objective_out, uint64_t* step2_bits_out);

/*
 * Quantize + pack for callers that must not allocate device memory.  The paper has no counterpart:
 * this is the same operation as lpc_quantize_pack on one unsegmented vector per worker (Algorithm 1
 * step 7), offered for code that cannot call cudaMalloc where it runs: a latency-critical loop that may
 * not take the allocator's locks or provoke its implicit synchronisation, a plug-in living inside a
 * host application's fixed memory budget, a process whose device memory is already fully partitioned.
 * It needs no context.  Its working memory (tile partials, scale records) is a fixed array of about
 * 0.8 MB inside the library image, held by every GPU that loads the library until the process exits.
 *   U            N x len fp32, row stride ld (device)
 *   codes_out    N * stride_words words, stride_words from lpc_packed_layout(len, b, NULL, 1) (device,
 *                16-byte aligned);  delta_out N floats;  clipped_out N counts (all required)
 *   stream       cudaStream_t of the device that is current when the call is made (the working memory is looked up
 *                on the current device; with a stream of another device the launches fail with LPC_ERR_CUDA)
 * Limits: N <= LPC_STATIC_MAX_WORKERS and N * ceil(len / 8192) <= LPC_STATIC_MAX_TILES; anything larger
 * returns LPC_ERR_UNSUPPORTED and launches nothing.  Non-finite input yields a NaN delta.
 * The first call on a device looks up the array's device address; make that first call outside any
 * stream capture.  All calls share the array and it keeps the previous call's contents (what has to
 * start from zero is cleared by the call itself), so two calls that can overlap on the GPU (different
 * streams, several host threads) race: serialise them.  The call allocates and frees nothing.
 */
#define LPC_STATIC_MAX_WORKERS 64
#define LPC_STATIC_MAX_TILES 65536
int lpc_quantize_pack_static(const float* U, int64_t len, int64_t ld, int32_t N, int32_t b, int clip_mode,
                             float clip_value, uint64_t seed, uint64_t k, uint32_t* codes_out, float* delta_out,
                             uint32_t* clipped_out, void* stream);

/*
 * Inspection aid for the error path of the bounded device-side waits (every wait of the library on a bulk copy, on
 * another CTA's message or on another worker's codes gives up after about two seconds, records the fact and lets the
 * kernel finish; the next lpc_sync_status then returns LPC_ERR_TIMEOUT).  This call enqueues one tiny kernel whose
 * waits of both kinds -- an mbarrier phase that nothing completes and, on a context with a linear model, a tagged
 * word that nobody writes -- run out after limit_ns (1 us .. 100 ms) through the same code.  Nothing else is in
 * flight, so the kernel ends normally and the context stays usable: lpc_sync_status returns LPC_ERR_TIMEOUT once,
 * then LPC_OK.  The paper has no counterpart.
 */
int lpc_debug_wait_timeout(lpc_ctx* ctx, uint64_t limit_ns);

/*
 * Inspection aid: writes `count` consecutive 4-word blocks, starting at block `block0`, of the
 * counter-based random stream (tag, worker, k) keyed by `seed` to out (device, 4*count words).
 * The streams are Philox4x32-10 (Salmon et al., SC'11) with counter (block, k_lo, worker | tag<<24,
 * k_hi) and key (seed_lo, seed_hi); tag 0 = stochastic rounding (Section 2.2 rule 1; coordinate j
 * uses 16-bit lane j%8 of block j/8), 1 = worker minibatches (Algorithm 1 step 6; slot a uses word 0
 * of block a), 2 = the shared batch J (Algorithm 2 step 11).
 */
int lpc_debug_stream_blocks(uint64_t seed, uint32_t tag, uint32_t worker, uint64_t k, uint32_t block0,
                            int64_t count, uint32_t* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LPC_H_ */
