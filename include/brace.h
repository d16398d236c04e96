/*
 * brace.h -- C ABI of the BRACE ring-aggregation library for NVIDIA B200 (sm_100a).
 *
 * One aggregation round of "Byzantine-Robust Federated Learning over
 * Ring-All-Reduce Distributed Computing" (BRACE): n clients each hold an update
 * vector of d float32 coordinates; the round leaves every client with the same
 * aggregated vector.  The n clients and the ring between them are simulated on
 * one GPU: client c's data are row c of caller-owned device matrices, a hop is
 * a move of one sub-vector from row c's buffers into row (c+1) mod n's.
 *
 * Conventions shared by every call
 *   - returns an int status (BRACE_OK = 0); never throws, aborts or prints;
 *   - device work is enqueued on `stream` (a cudaStream_t passed as void*) and
 *     the call returns without synchronising;
 *   - the library allocates no device memory: mailboxes live in the
 *     caller-provided workspace, inputs and outputs are caller buffers;
 *   - pointers named d_* are device pointers, h_* host pointers;
 *   - clients c and sub-vectors j are 0-based.  Ring direction and the
 *     hop -> sub-vector map follow the three-client worked example of
 *     Section 2.2: at share-reduce hop s client c sends sub-vector
 *     (c - s) mod n to client (c + 1) mod n; after n-1 hops client c owns
 *     sub-vector (c + 1) mod n; at share-only hop t client c sends
 *     sub-vector (c + 1 - t) mod n to client (c + 1) mod n.
 *   - a context must not be used from two host threads, or on two streams,
 *     at the same time.
 */
#ifndef BRACE_H
#define BRACE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct brace_ctx brace_ctx;
typedef void* brace_stream_t; /* cudaStream_t */

/* status codes */
enum {
  BRACE_OK = 0,
  BRACE_ERR_INVALID_ARG = 1, /* null / out-of-range / misaligned argument; nothing was launched */
  BRACE_ERR_UNSUPPORTED = 2, /* valid request the library cannot serve (e.g. n > 32767)         */
  BRACE_ERR_BAD_STEP = 3,    /* hop called out of order; nothing was launched                   */
  BRACE_ERR_WORKSPACE = 4,   /* workspace missing, too small or misaligned                      */
  BRACE_ERR_CUDA = 5,        /* a CUDA runtime call failed; see brace_last_cuda_error           */
  BRACE_ERR_TIMEOUT = 6      /* reserved: a bounded device-side wait ran out                    */
};

/* aggregation rules.  All but SUM share Phases I, II and IV of Section 3 (sign,
 * share-reduce of the signs, 1-bit share-only) and differ in the Phase III map
 * applied to the integer sign-sum S = sum_i sign(g_i[k]):
 *   SIGN_CONSENSUS  +1 if S > lambda, else -1                       (BRACE, Eq. (1))
 *   MAJORITY_SIGN   +1 if S > 0, else -1 (lambda unused)            (signSGD with majority vote run over the
 *                   ring, which Section 5.2 says follows the same procedure; the paper does not say what a tie
 *                   S = 0 gives: here -1, as Eq. (1) does with lambda = 0)
 *   ABS_CONSENSUS   +1 if |S| > lambda, else -1                     (the RLR-style test Section 5.2 describes:
 *                   the absolute value of the sum, positive and negative agreement treated alike; the paper
 *                   gives no formula, strictness of the inequality follows Eq. (1))                          */
enum {
  BRACE_RULE_SIGN_CONSENSUS = 0, /* BRACE, Section 3, Eq. (1)                                     */
  BRACE_RULE_SUM = 1,            /* plain ring-all-reduce sum, Section 2.2 (optionally the mean)  */
  BRACE_RULE_MAJORITY_SIGN = 2,  /* sign of the sign-sum (Section 5.2: signSGD over the ring)     */
  BRACE_RULE_ABS_CONSENSUS = 3   /* |sign-sum| against lambda (Section 5.2: RLR over the ring)    */
};

/* how brace_aggregate runs a round (the result is the same) */
enum {
  BRACE_AGG_AUTO = 0,     /* fused when the layout allows it, else stepwise                        */
  BRACE_AGG_STEPWISE = 1, /* 2(n-1)+1 kernel launches, one per hop, exactly like the step calls    */
  BRACE_AGG_FUSED = 2     /* one kernel that carries each sub-vector tile through all hops         */
};

/* Byzantine alterations applied before the ring starts (threat model, Section 3).
 * "honest" rows are those not listed as Byzantine; statistics over them are
 * accumulated in float64 in increasing client id and rounded once to float32. */
enum {
  BRACE_ATTACK_NONE = 0,
  BRACE_ATTACK_SCALE_OWN = 1,   /* b_i = scale * h_i (own honest update)                           */
  BRACE_ATTACK_GAUSSIAN = 2,    /* b_i = sigma * noise_i                                           */
  BRACE_ATTACK_SCALED_MEAN = 3, /* b_i = scale * mean_honest (same vector for every Byzantine)     */
  BRACE_ATTACK_MEAN_SHIFT = 4,  /* b_i = mean_honest - kappa * std_honest (population std)         */
  BRACE_ATTACK_SPARSE_NOISE = 5 /* b_i[k] = uniform_i[k] < prob ? sigma * noise_i[k] : 0           */
};

/* Parameters of the rule.  Fill with brace_default_params, then edit. */
typedef struct brace_params {
  int32_t rule;      /* BRACE_RULE_*                                                              */
  float lambda;      /* Eq. (1) threshold; any finite value; the sign-sum S is an integer, so
                        S > lambda is evaluated as S > floor(lambda); S == lambda gives -1        */
  int32_t zero_sign; /* what an exactly-zero coordinate votes: -1, 0 (default, abstain) or +1;
                        NaN always votes 0, +-Inf vote +-1                                        */
  int32_t granule;   /* sub-vector boundaries are multiples of this many coordinates
                        (default 128; >= 1).  With Q = ceil(d/granule), sub-vector j is
                        [min(granule*floor(j*Q/n), d), min(granule*floor((j+1)*Q/n), d))          */
  int32_t mean;      /* BRACE_RULE_SUM only: non-zero divides the sum by n                        */
  int32_t agg_mode;  /* BRACE_AGG_*                                                               */
} brace_params;

/* Where the random draws of kinds 2 and 5 come from. */
enum {
  BRACE_DRAWS_SUPPLIED = 0, /* the caller passes noise / uniform matrices                          */
  BRACE_DRAWS_GENERATED = 1 /* the library draws them itself from (seed, round); see below         */
};

/* Description of one attack.
 * draws = SUPPLIED: noise / uniform are [f][*_ld] float32 matrices of standard-normal /
 * uniform[0,1) draws supplied by the caller (row b belongs to the b-th Byzantine id); only
 * the kinds that consume them read them.
 * draws = GENERATED: noise / uniform are ignored; the kernels draw from the library's
 * counter-based generator, so that only the Byzantine rows move through memory.  A draw is
 * a pure function of (seed, round, client id, coordinate, stream): Philox4x32-10 with key
 * (seed mod 2^32, seed div 2^32) and counter (q mod 2^32, q div 2^32, client,
 * round * 256 + stream) serves the four coordinates 4q..4q+3 (word k mod 4 for coordinate
 * k).  Stream 0: uniform = (word >> 8) * 2^-24.  Stream 1: a coordinate pair (2p, 2p+1) with
 * words (a, b) gives u1 = ((a >> 8) + 1) * 2^-24, u2 = (b >> 8) * 2^-24,
 * radius = sqrt(-2 ln u1), z[2p] = radius cos(2 pi u2), z[2p+1] = radius sin(2 pi u2),
 * evaluated in float32 (a few ulp from the exactly rounded value).  round < 2^24. */
typedef struct brace_attack {
  int32_t kind;             /* BRACE_ATTACK_*                                                     */
  float scale;              /* kinds 1, 3                                                         */
  float sigma;              /* kinds 2, 5                                                         */
  float kappa;              /* kind 4                                                             */
  float prob;               /* kind 5                                                             */
  const int32_t* h_byz_ids; /* host array of f distinct client ids, or NULL for clients 0..f-1    */
  const float* noise;       /* device pointer (host pointer for brace_aggregate_host)             */
  int64_t noise_ld;
  const float* uniform;     /* device pointer (host pointer for brace_aggregate_host)             */
  int64_t uniform_ld;
  int32_t draws;            /* BRACE_DRAWS_*                                                      */
  uint32_t round;           /* GENERATED: round index, < 2^24                                     */
  uint64_t seed;            /* GENERATED: seed                                                    */
} brace_attack;

const char* brace_status_string(int status);

/* rule = SIGN_CONSENSUS, lambda = 0, zero_sign = 0, granule = 128, mean = 0, agg_mode = AUTO. */
int brace_default_params(brace_params* params);

/* Bytes of device workspace a context for (n, d, params) needs; 0 if the
 * arguments are invalid.  Holds two sets ("ping-pong") of n mailboxes, each as
 * long as the longest sub-vector rounded up to 128 entries, plus client-id
 * lists for the attack kernels.  Mailbox entries are int8 partial sign-sums
 * for n <= 127, int16 for n <= 32767 (BRACE), float32 (SUM). */
size_t brace_workspace_bytes(int32_t n, int64_t d, const brace_params* params);

/* Create a context (host memory, owned by the library until brace_destroy).
 *   n >= 2 clients, 0 <= f < n of them Byzantine (f is used by the attack call
 *   and by validation only -- Eq. (1) does not take f), d >= 1 coordinates.
 *   d_workspace: device memory, 256-byte aligned, at least brace_workspace_bytes
 *   long, owned by the caller and kept alive and untouched while the context
 *   lives.  Passing d_workspace = NULL with workspace_bytes = 0 creates a
 *   host-only context: brace_segment works, every device call returns
 *   BRACE_ERR_WORKSPACE.  `stream` is accepted for symmetry; init enqueues nothing.
 * Errors: INVALID_ARG (null out, n < 2, f out of range, d < 1, bad params,
 * non-finite lambda), UNSUPPORTED (n > 32767 under SIGN_CONSENSUS),
 * WORKSPACE (too small / misaligned). */
int brace_init(brace_ctx** out, int32_t n, int32_t f, int64_t d, const brace_params* params,
               void* d_workspace, size_t workspace_bytes, brace_stream_t stream);
int brace_destroy(brace_ctx* ctx);

/* Sub-vector j covers coordinates [*begin, *end) (Section 2.2: "n roughly
 * equal-sized sub-vectors"; formula at brace_params.granule).  Host only. */
int brace_segment(const brace_ctx* ctx, int32_t j, int64_t* begin, int64_t* end);

/* cudaError_t of the last failed runtime call on this context (0 if none).  With ctx = NULL: of the
 * last failed runtime call made on the calling host thread by an entry point that takes no context
 * (brace_aggregate_static, brace_draw_matrix, brace_minmax_rate_probe, brace_debug_status). */
int brace_last_cuda_error(const brace_ctx* ctx);

/* Threat model of Section 3: Byzantine clients alter their vectors before the
 * ring starts and then follow the protocol.  Reads the honest update matrix
 * d_honest [n][ld_honest] and writes the f Byzantine rows of d_updates
 * [n][ld_updates]; rows of honest clients are not touched.  d_honest may equal
 * d_updates (in place).  attack->noise / uniform are device pointers.
 * kind NONE or f == 0 does nothing.  The id list is uploaded to the workspace when
 * it differs from the one already there; that upload is refused while `stream` is
 * being captured (BRACE_ERR_UNSUPPORTED): call once with a given id list before
 * capturing.  Errors: INVALID_ARG (null pointers, ld < d, duplicate or
 * out-of-range ids, missing noise/uniform for a kind that needs them with
 * draws = SUPPLIED, round >= 2^24 with draws = GENERATED). */
int brace_inject_attack(brace_ctx* ctx, const brace_attack* attack, const float* d_honest,
                        int64_t ld_honest, float* d_updates, int64_t ld_updates,
                        brace_stream_t stream);

/* Section 3 Phase I (Quantization) on its own: d_q [n][ld_q] int8 receives the
 * element-wise sign of d_updates [n][ld].  The ring calls below fuse this step
 * into their reads; this entry exists for inspection and tests. */
int brace_quantize(brace_ctx* ctx, const float* d_updates, int64_t ld, int8_t* d_q, int64_t ld_q,
                   brace_stream_t stream);

/* One Share-Reduce hop (Section 2.2 Phase I / Section 3 Phase II) for all n
 * clients at once.  Receiver r = (c+1) mod n stores into its mailbox the value
 * it received from c (c's own quantized sub-vector at step 0, c's mailbox
 * content otherwise) plus its own (quantized) sub-vector (c - step) mod n.
 * step must run 0, 1, .., n-2 in order; step 0 may be called at any time and
 * starts a new round.  d_updates [n][ld] float32, ld >= d, must not change
 * during a round.  Errors: BAD_STEP, INVALID_ARG, WORKSPACE, CUDA. */
int brace_ring_reduce_scatter_step(brace_ctx* ctx, int32_t step, const float* d_updates, int64_t ld,
                                   brace_stream_t stream);

/* Section 3 Phase III (Consensus), after the last share-reduce hop: client c,
 * owner of sub-vector (c+1) mod n, applies Eq. (1) to the sign-sums in its
 * mailbox and writes the result into its own output row.
 *   SIGN_CONSENSUS: d_out is uint32 [n][out_ld], out_ld >= ceil(d/32);
 *     coordinate k is bit (k mod 32), least significant first, of word
 *     (k div 32) of the row; 1 means +1, 0 means -1; bits past d in the last
 *     word are 0.
 *   SUM: d_out is float32 [n][out_ld], out_ld >= d; the step copies the sum
 *     (divided by n if params.mean).
 * Only the owner's sub-vector of each row is written here. */
int brace_consensus(brace_ctx* ctx, void* d_out, int64_t out_ld, brace_stream_t stream);

/* One Share-Only hop (Section 2.2 Phase II / Section 3 Phase IV) for all n
 * clients: row (c+1) mod n of d_out receives sub-vector (c + 1 - step) mod n
 * from row c.  step runs 0..n-2 in order after brace_consensus; after the last
 * one every row of d_out holds the same aggregated vector. */
int brace_ring_allgather_step(brace_ctx* ctx, int32_t step, void* d_out, int64_t out_ld,
                              brace_stream_t stream);

/* A whole round (Section 3, Phases I-IV).  The final contents of every row of
 * d_out, and of the mailboxes over the lengths of the sub-vectors they hold,
 * equal those left by calling the step functions in order.  The fused mode needs
 * granule % 128 == 0, ld % 4 == 0 and 16-byte aligned d_updates (and, for SUM,
 * out_ld % 4 == 0 and 16-byte aligned d_out); AUTO falls back to stepwise
 * launches when these do not hold, FUSED returns UNSUPPORTED. */
int brace_aggregate(brace_ctx* ctx, const float* d_updates, int64_t ld, void* d_out, int64_t out_ld,
                    brace_stream_t stream);

/* The step after a round: every client applies the aggregate it now holds to
 * its own parameter vector (row c of d_weights [n][ld_weights] float32,
 * updated in place; ld_weights >= d).
 *   sign rules: w_c[k] <- w_c[k] - eta * (+1 or -1 read from row c of d_out)
 *     (Appendix A, update rule: no 1/n, the aggregate has unit entries);
 *   SUM: w_c[k] <- w_c[k] - (eta / n) * sum[k]  (Section 2.2, per-client update
 *     after plain ring-all-reduce); with params.mean the rows already hold the
 *     mean and the factor is eta.
 * float32 arithmetic, each operation rounded to nearest.  d_out / out_ld as for
 * brace_aggregate; it is only read.  Errors: INVALID_ARG (null, short rows,
 * non-finite eta), WORKSPACE, CUDA. */
int brace_apply_update(brace_ctx* ctx, const void* d_out, int64_t out_ld, float* d_weights,
                       int64_t ld_weights, float eta, brace_stream_t stream);

/* Coordinate-wise statistics over the n client values of every coordinate: the
 * server-side aggregation rules the paper compares against (Section 5.1: Median,
 * Trimmed-mean).  They need all n slices of a coordinate at once, so they are
 * not ring rules (Section 3); this call reads d_updates [n][ld] directly and
 * writes ONE vector d_result [d] float32.  It uses no workspace (a host-only
 * context is accepted).
 *   BRACE_STAT_MEDIAN        the middle value of the n sorted values; for even n
 *                            the mean of the two middle values (float64 add and
 *                            halve, rounded once to float32); `trim` is ignored
 *   BRACE_STAT_TRIMMED_MEAN  drop the `trim` smallest and the `trim` largest
 *                            values (0 <= 2*trim < n), then the mean of the rest,
 *                            summed in float64 in ascending order and rounded once
 * +-Inf take part in the ordering; a NaN input makes that coordinate's result
 * unspecified.  n <= 128 (else BRACE_ERR_UNSUPPORTED). */
enum { BRACE_STAT_MEDIAN = 0, BRACE_STAT_TRIMMED_MEAN = 1 };
int brace_coordinate_stat(brace_ctx* ctx, int32_t kind, int32_t trim, const float* d_updates, int64_t ld,
                          float* d_result, brace_stream_t stream);

/* Rows of the library's own random draws (the generator described at
 * brace_attack), for inspection and as a building block of synthetic inputs:
 * row i of d_out [rows][ld] belongs to client first_client + i;
 *   what = BRACE_DRAW_UNIFORM  d_out[i][k] = the uniform of (seed, round, client, k)
 *   what = BRACE_DRAW_NORMAL   d_out[i][k] = mu + sigma * z, z the normal of (seed, round, client, k)
 * Needs no context.  Errors: INVALID_ARG (null, rows < 1 or > 65535, d < 1, ld < d,
 * first_client < 0, round >= 2^24), CUDA. */
enum { BRACE_DRAW_UNIFORM = 0, BRACE_DRAW_NORMAL = 1 };
int brace_draw_matrix(int32_t what, uint64_t seed, uint32_t round, int32_t first_client, int32_t rows, int64_t d,
                      float* d_out, int64_t ld, float mu, float sigma, brace_stream_t stream);

/* Same round with HOST inputs and outputs: copies h_updates [n][ld] to the
 * caller's device staging matrix d_updates_stage [n][ld], applies `attack`
 * there if attack != NULL (with draws = SUPPLIED attack->noise / uniform are HOST
 * [f][*_ld] matrices, copied to d_noise_stage / d_uniform_stage of the same
 * shape; with draws = GENERATED nothing but the updates is copied and the two
 * staging pointers may be NULL), aggregates into
 * d_out_stage [n][out_ld] and copies that to h_out.  All copies are
 * cudaMemcpyAsync on `stream`: pinned host memory makes them asynchronous, and
 * h_out is valid once the stream has been synchronised. */
int brace_aggregate_host(brace_ctx* ctx, const brace_attack* attack, const float* h_updates, int64_t ld,
                         void* h_out, int64_t out_ld, float* d_updates_stage, float* d_noise_stage,
                         float* d_uniform_stage, void* d_out_stage, brace_stream_t stream);

/* Bits each client sends in one round, from this context's actual partition
 * (Section 2.2 and Section 3 cost paragraphs, Table 1).  m_bits = width of one
 * gradient coordinate on the wire (the paper's m).  Host only.
 *   sc_bits               m*n*d (server-client)
 *   rar_bits_min/max      plain ring-all-reduce: client c sends every sub-vector but (c+1) mod n during
 *                         share-reduce and every one but (c+2) mod n during share-only, m bits per coordinate;
 *                         closed form 2*m*d*(n-1)/n when n divides d
 *   brace_bits_min/max    sign rules: the same share-reduce at m bits, share-only at 1 bit per coordinate;
 *                         closed form d*(n-1)*(m+1)/n
 *   packed_bits_min/max   as brace_bits with share-reduce at the width the mailboxes really use
 *   partial_bits_used     8 or 16 (mailbox entry width); partial_bits_min = ceil(log2(2n+1)), the fewest
 *                         bits that can hold a partial sign-sum in [-n, n]                                 */
typedef struct brace_cost {
  int64_t sc_bits;
  int64_t rar_bits_min, rar_bits_max;
  int64_t brace_bits_min, brace_bits_max;
  int64_t packed_bits_min, packed_bits_max;
  double rar_closed_form, brace_closed_form;
  int32_t partial_bits_used, partial_bits_min;
} brace_cost;
int brace_comm_cost(const brace_ctx* ctx, int32_t m_bits, brace_cost* cost);

/* Test aid: device pointer, length (entries) and sub-vector id of the mailbox
 * that client `client` filled at the most recent share-reduce hop
 * (hops_back = 0) or at the hop before it (hops_back = 1; the other mailbox
 * set).  Valid after at least 1 + hops_back hops of the current round.
 * *entry_bytes is 1, 2 or 4.  segment and entry_bytes may be NULL. */
int brace_debug_mailbox(const brace_ctx* ctx, int32_t client, int32_t hops_back, const void** d_ptr,
                        int64_t* len, int32_t* segment, int32_t* entry_bytes);

/* Expert knob for measurements: pick the fused kernel's shape.  fused_variant
 * 0 = library default; 1..6 = (float4 per thread per client, clients
 * prefetched, threads per CTA) in {(1,8,256),(2,4,256),(1,4,256),(2,8,256),
 * (1,16,256),(1,8,128)}.  fused_grid = 0 launches one CTA per tile, > 0 caps the
 * grid (CTAs then loop over tiles).
 * Adding 10, 20 or 40 to fused_variant makes the share-reduce hop kernel process
 * 1, 2 or 4 float4 per thread (default: 4, fewer for short sub-vectors); adding
 * 100, 200 or 400 picks the staged statistics kernel with 1, 2 or 4 floats per
 * thread, 800 makes the register-resident statistics kernel address rows through
 * its offset table even when they are consecutive, 900 makes attack 5 with
 * generated draws compute its normals block by block instead of for a compacted
 * list of the coordinate pairs that need one.  On large problems
 * (n*d >= 2^27) the fused kernel writes each sub-vector's bits to its owner's row
 * and one share-only launch spreads them to the other rows; adding 1000 forces
 * that at any size, adding 2000 makes the fused kernel write all n rows itself.
 * Results do not depend on any of these. */
int brace_set_tuning(brace_ctx* ctx, int32_t fused_variant, int32_t fused_grid);

/* Calibration for brace_coordinate_stat's roofline (no counterpart in the paper): launches `blocks` CTAs of
 * 256 threads that each execute iters * 64 register-to-register min/max operations (the operation the sorting
 * network of the Section 5.1 baselines is made of) and writes one float per thread to d_out
 * [blocks * 256].  *ops receives the number of min/max operations the launch performs; time the launch
 * with events on `stream` to get this GPU's min/max rate.  Errors: INVALID_ARG, CUDA. */
int brace_minmax_rate_probe(int32_t blocks, int32_t iters, float* d_out, int64_t* ops, brace_stream_t stream);

/* Debug build only (library compiled with -DBRACE_DEBUG; paper_2501_17392_b200.build.build_debug()): the
 * ring kernels (the share-reduce, consensus and share-only steps of Section 3 and the fused round) check that
 * the sub-vector they were handed lies inside the buffers they index and that client indices are in range.
 * A failed check never traps: it records a code and the CTA skips the sub-vector.  This call waits for the
 * device, returns the code of the first failed check since the previous call in *h_code (0 = none;
 * 1 = update row, 2 = mailbox, 3 = output row, 4 = client index) and clears it.  The release build performs no
 * checks and returns BRACE_ERR_UNSUPPORTED with *h_code = 0.  Errors: INVALID_ARG (null), CUDA. */
int brace_debug_status(int32_t* h_code);

/* Bytes of mailbox scratch built into the library for brace_aggregate_static. */
#define BRACE_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)

/* A whole round without a context and without a workspace (no counterpart in
 * the paper: this is a packaging variant of brace_aggregate's fused kernel).
 *
 * Who needs it: code that may not obtain device memory at the point where it
 * aggregates -- a plugin running inside a host application whose allocator owns
 * all of HBM and offers no scratch to plugins, a service whose memory budget is
 * frozen after start-up, a callback that runs where cudaMalloc is forbidden.
 * Such callers still own their input and output buffers, but cannot size and
 * allocate the mailbox workspace brace_init asks for.  Here the mailboxes live
 * in a fixed array of BRACE_STATIC_SCRATCH_BYTES compiled into the library's
 * device image (each GPU that loads the library keeps it until the process
 * ends).  The call makes no cudaMalloc / cudaFree and calls no allocating
 * routine; the context it uses internally lives on the host stack.
 *
 * Arguments as for brace_init (n, d, params; f is not needed) and
 * brace_aggregate (d_updates [n][ld] float32, d_out [n][out_ld] packed uint32
 * rows, or float32 rows for the sum rule).  Always runs the fused kernel, so it
 * needs granule % 128 == 0, ld % 4 == 0 and 16-byte aligned d_updates (sum rule:
 * also out_ld % 4 == 0 and aligned d_out); otherwise BRACE_ERR_UNSUPPORTED.
 * Limit: 2 * round_up(n * round_up(longest sub-vector, 128) * entry bytes, 256)
 * must not exceed BRACE_STATIC_SCRATCH_BYTES (about d <= 4.1 million for n <= 127
 * under the sign rule, d <= 1.0 million under the sum rule); larger requests
 * return BRACE_ERR_WORKSPACE and launch nothing.
 *
 * Every call looks up the array's device address for the device that is current
 * (cudaGetSymbolAddress: no allocation; nothing is cached, so the call stays
 * valid after a device reset).  The first call on a device also makes the CUDA
 * runtime load the library's kernels there: make that first call outside any
 * stream capture.  A CUDA failure of this call is kept per host thread and
 * returned by brace_last_cuda_error(NULL).  All calls on a device share the one
 * array: it keeps whatever the previous call left
 * (nothing in it has to start at zero -- the kernel only writes it), and two
 * calls whose kernels may overlap on the GPU (different streams) race on it:
 * serialise them.  Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
int brace_aggregate_static(int32_t n, int64_t d, const brace_params* params, const float* d_updates,
                           int64_t ld, void* d_out, int64_t out_ld, brace_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* BRACE_H */
