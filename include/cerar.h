/*
 * cerar.h - C ABI of the CERAR coding pipeline for one B200.
 *
 * CERAR (communication-efficient ring all-reduce) lets N ring workers, each
 * holding a length-d gradient split into c chunks of p = d/c values, obtain an
 * approximation of the sum of all gradients in L = c + N - 2 rounds of
 * length-p messages (problem statement, Sec. I; protocol, Sec. II).  In this
 * library the N logical workers live in one GPU's memory and a ring hand-off
 * is a store into the neighbour's buffer; there is no inter-GPU transport.
 * (The cerar_rank_* calls further down are the one-worker-per-GPU form of the
 * same protocol, with the neighbour's buffer given as a pointer.)
 *
 * Conventions for every call
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA
 *     device memory on the device that was current when the plan was created.
 *   - The caller owns every data buffer.  The library owns the plan (host fp64
 *     matrices and fp32 device copies of them) and allocates nothing in the
 *     data-path calls (encode, ring_round, decode, allreduce_sim).
 *   - Data-path calls are asynchronous on the given stream and report
 *     argument and launch errors only.  Nothing throws across this boundary.
 *   - A plan is not synchronised internally: calls on the SAME plan from several
 *     host threads must be serialised by the caller (its round state, counters and
 *     status word are per plan); different plans are independent.  The tuning
 *     knobs (cerar_set_tuning) are process-wide and meant to be set before use.
 *   - All matrices are row-major.  Gradients are fp32 on the device; the
 *     coefficient matrices are built in fp64 on the host and rounded to fp32
 *     for the device.
 *
 * Workspace layout (device, fp32): worker i owns a row-major (c+N) x p matrix
 * at ws + i*(c+N)*p.  Row ("slot") s of worker i holds
 *     s = 0 .. N-2      : B_{i,1} .. B_{i,N-1}  (first N-1 received messages)
 *     s = N-1           : C_i                    (landing slot of message N)
 *     s = N .. N+c-1    : D_{i,1} .. D_{i,c}     (encoded vectors delta_{i,j})
 * which is exactly the (c+N) p values per worker of the paper's storage rate
 * 1 + N/c (Sec. II-B).  Message k of worker i-1 lands in slot k-1 of worker i,
 * so after L rounds slots 0..L-1 hold y_{i,1}..y_{i,L} in order and slot L+1
 * holds y_{i,L+1} = delta_{i,c}; slot L keeps a stale delta_{i,c-1} that the
 * decoder does not read.
 */
#ifndef CERAR_H_
#define CERAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cerar_plan cerar_plan_t;          /* opaque, library-owned */
typedef struct CUstream_st* cerar_stream_t;      /* a cudaStream_t */

typedef enum {
    CERAR_OK = 0,
    CERAR_ERR_INVALID_ARG = 1,   /* null pointer, N < 2, c < N, bad parameter          */
    CERAR_ERR_SHAPE = 2,         /* c does not divide d, stride too small, d <= 0       */
    CERAR_ERR_SINGULAR = 3,      /* non-finite coefficients or a singular window        */
    CERAR_ERR_NOT_CONVERGED = 4, /* kappa design: constraint not met after the last step */
    CERAR_ERR_STATE = 5,         /* rounds out of order, decode before the last round    */
    CERAR_ERR_CUDA = 6,          /* a CUDA runtime call failed, or no device             */
    CERAR_ERR_NOMEM = 7,
    CERAR_ERR_TIMEOUT = 8,
    CERAR_ERR_TOO_LARGE = 9,     /* request exceeds the built-in workspace (see below)    */
    CERAR_ERR_BOUNDS = 10        /* checked build only: a kernel formed an address outside its buffer */
} cerar_status_t;

typedef enum {
    CERAR_VANDERMONDE = 0,   /* param = tau   (Sec. II-B.2)                     */
    CERAR_EPSILON = 1,       /* param = eps   (Sec. II-C, D = I + eps H)        */
    CERAR_KAPPA = 2          /* param = C, the bound on kappa_2(M_i) (Sec. II-D) */
} cerar_construction_t;

/* Optional settings for cerar_plan_create_ex.  Zero-initialise for defaults. */
typedef struct {
    uint64_t      seed;       /* seed of the built-in N(0,1) generator used for B when B == NULL */
    const double* B;          /* host, N x c: base matrix of the epsilon / kappa designs, or NULL */
    const double* h;          /* host, length c: diag(H) (epsilon, kappa) or the nodes xi_j
                                 (Vandermonde); NULL = c equally spaced values in [-1, 1]        */
    double        eps_init;   /* kappa design: eps of the initial epsilon-construction; 0 = 0.1  */
    int           als_iters;  /* kappa design: maximum ALS iterations; 0 = 200                   */
    double        als_tol;    /* kappa design: stop when Phi changes by less (relative); 0 = 1e-6 */
    int           host_only;  /* 1 = never touch CUDA (plan usable for get_U / get_R / info only) */
} cerar_options_t;

typedef struct {
    int      N, c, L;
    int      construction;       /* cerar_construction_t, or 3 for a custom plan            */
    double   param;
    double   phi;                /* Phi(U,R) = sum_i ||M_i(U) R_i - T||_F^2 (Eq. F_unreg);
                                    closed form of Prop. 2 for the explicit constructions   */
    double   kappa_U_max;        /* max_k kappa_2(U_k)                                       */
    double   kappa_M_max;        /* max_i kappa_2(M_i(U))                                    */
    double   inv_residual_max;   /* max_k ||U_k A_{N-1-k} - I||_max (explicit constructions) */
    double   abs_U_max, abs_R_max;
    int      als_iters_done;
    int      on_device;          /* 1 if fp32 copies were uploaded                            */
} cerar_plan_info_t;

typedef struct {
    int      encoded;                      /* 1 after cerar_encode                          */
    int      rounds_done;                  /* k of the last completed cerar_ring_round      */
    uint64_t bytes_forwarded_per_worker;   /* sum over completed rounds of 4 p              */
    uint64_t bytes_forwarded_last_round;   /* 4 p                                           */
    uint64_t bytes_stored_per_worker;      /* 4 p (c + N)                                   */
    uint64_t bytes_gradient;               /* 4 d, the denominator of both rates            */
} cerar_counters_t;

/* ---- plan: coefficient matrices U_0..U_{N-1} (c x c) and R_0..R_{N-1} ((L+1) x c) ----
 *
 * cerar_plan_create builds the multiplicative perturbation construction of
 * Sec. II-B.1 (a_{r+mN} = b_r D^m, A_l = [a_l; ..; a_{l+c-1}], U_k = A_{N-1-k}^{-1},
 * R_i[l,:] = a_{l-i}) for the Vandermonde (Sec. II-B.2) or epsilon (Sec. II-C)
 * choice of (B, D), or runs the alternating least-squares heuristic of Sec. II-D
 * started from an epsilon-construction.  Requires 2 <= N <= c.  On success *out
 * is a new plan; on failure *out is NULL.  If a CUDA device is available (and
 * host_only is 0) fp32 copies are uploaded to the current device. */
cerar_status_t cerar_plan_create(int N, int c, cerar_construction_t kind, double param,
                                 cerar_plan_t** out);
cerar_status_t cerar_plan_create_ex(int N, int c, cerar_construction_t kind, double param,
                                    const cerar_options_t* opt, cerar_plan_t** out);
/* Plan from caller-supplied matrices (host, fp64): U is N*c*c, R is N*(L+1)*c.
 * Any finite numbers are accepted: the data path is the protocol of Algorithm 1
 * with these coefficients, whatever they decode to. */
cerar_status_t cerar_plan_create_custom(int N, int c, const double* U, const double* R,
                                        int host_only, cerar_plan_t** out);
void           cerar_plan_destroy(cerar_plan_t* plan);

/* Copies of the fp64 matrices (host buffers of c*c and (L+1)*c doubles). */
cerar_status_t cerar_plan_get_U(const cerar_plan_t* plan, int worker, double* out_cxc);
cerar_status_t cerar_plan_get_R(const cerar_plan_t* plan, int worker, double* out_Lp1xc);
/* Diagnostics (computed on first request: a few SVDs on the host). */
cerar_status_t cerar_plan_info(cerar_plan_t* plan, cerar_plan_info_t* out);

/* gamma(B, H) = min_{l=0..N-1} sigma_min(K^(l)(B, H)) for H = diag(h): the constant that the
 * analysis of the epsilon-construction assumes positive (Sec. II-C, the Assumption before the
 * theorem on singular value scaling; K^(l) = [B; BH; ..; BH^(beta-1); (BH^beta)_{E_l}] with
 * c = beta N + s, E_l = {l, .., l+s-1} mod N).  sigma_min(A_l(eps)) = Theta(eps^r*) carries it
 * as its constant, so among several trial H (which Sec. II-C allows) the one with the largest
 * gamma is the natural pick.  Host only, no CUDA.
 * B: N x c row-major or NULL (built-in N(0,1) generator with `seed`); h: length c or NULL
 * (equally spaced in [-1, 1]). */
cerar_status_t cerar_design_gamma(int N, int c, const double* B, uint64_t seed, const double* h,
                                  double* gamma_out);
/* A deterministic choice of H from B (the paper's appendix on the numerical experiments mentions
 * that H can be derived deterministically from B and gives no rule; this is the library's
 * reading): coordinate ascent on gamma(B, H).  Start: h as passed (use_start != 0)
 * or equally spaced in [-1, 1]; scaled to max|h| = 1; coordinates are visited in order, each moves
 * to the first of `grid` equally spaced values of [-1, 1] with the largest gamma if that beats the
 * current gamma and leaves max|h| = 1; at most `sweeps` passes.  h (c doubles, host) receives the
 * result, which goes into cerar_options_t.h; gamma_out / moves_out may be NULL.  Host only. */
cerar_status_t cerar_design_optimize_h(int N, int c, const double* B, uint64_t seed, double* h, int use_start,
                                       int sweeps, int grid, double* gamma_out, int* moves_out);

/* Smallest d' >= d that is a multiple of 4c.  The protocol needs c | d (the caller pads the
 * gradient with zeros, Sec. II); the fast kernels additionally need rows of p = d/c values to
 * start on 16-byte boundaries, i.e. 4 | p.  With c | d but p not a multiple of 4 (or buffers
 * that start off a 16-byte boundary) every call still works: the contractions then bring
 * every row in with a copy of its own that starts at the 16-byte boundary below the row and
 * ends at the one above it, i.e. they may READ up to 12 bytes before and after a row, inside
 * 16-byte groups that hold at least one element of the buffer (nothing outside a buffer is
 * ever written), and run at 0.8-0.9 of the aligned speed for c <= 64, far less beyond.
 * Padding to this length avoids all that (zeros in, the padded tail of the result is zero
 * as well). */
int64_t        cerar_padded_length(const cerar_plan_t* plan, int64_t d);

/* Bytes of the device workspace for gradient length d: 4 * N * (c+N) * (d/c);
 * 0 if c does not divide d. */
size_t cerar_workspace_bytes(const cerar_plan_t* plan, int64_t d);

/* ---- data path (device buffers, fp32) ----
 *
 * cerar_encode: Delta_i = G_i U_i for every worker (Sec. II, Initialization):
 *   D_{i,j}[q] = sum_l U_i[l, j-1] * g_i[l*p + q].  grads: worker i's gradient
 *   at grads + i*grads_stride (stride in floats, >= d).  In place: pass
 *   grads = ws + N*p and grads_stride = (c+N)*p, i.e. the gradient already sits
 *   in the D rows.  Resets the round counter.
 *
 * cerar_ring_round(k), k = 1..L in order: every worker forms the message of
 *   round k, x_{i,k} = sigma_{i,k-1} (+ delta_{i,k} if k <= c) with
 *   sigma_{i,k-1} = y_{i,k-1} (- delta_{i,k-N} if k-1 >= N), sigma_{i,0} = 0
 *   (Eq. update_eqns; Algorithm 1 with the cancel step of round k-1 fused into
 *   the send step of round k), and hands it to W_{i+1} by storing it in slot
 *   k-1 of that worker's workspace.
 *
 * cerar_decode: g_hat_i = scale * Y_i R_i (Sec. II-A), Y_i = [y_{i,1} .. y_{i,L+1}].
 *   out: worker i's result at out + i*out_stride (floats, >= d); every worker
 *   gets its own (slightly different) approximation.  scale = 1 is the paper's
 *   approximate sum, scale = 1/N the mean.  In place: out = ws + N*p with
 *   out_stride = (c+N)*p overwrites the D rows.  Needs all L rounds done.
 *
 * cerar_allreduce_sim: encode, rounds 1..L, decode, on one stream.
 *
 * These four calls only enqueue kernels on `stream` (no allocation, no
 * synchronisation), so after one warm-up call with the same shapes a caller
 * may capture them in a CUDA graph and replay it; for small d, where the L+2
 * launches dominate, that is 1.3-1.8 times faster.
 *
 * d must be a positive multiple of c (the caller zero-pads, Sec. II) else
 * CERAR_ERR_SHAPE.  ws must hold cerar_workspace_bytes(plan, d) bytes.  Input,
 * output and workspace may alias only in the two in-place forms above.
 */
cerar_status_t cerar_encode(cerar_plan_t* plan, const float* grads, int64_t grads_stride,
                            float* ws, int64_t d, cerar_stream_t stream);
cerar_status_t cerar_ring_round(cerar_plan_t* plan, float* ws, int64_t d, int k,
                                cerar_stream_t stream);
/* Rounds k_first .. k_last (k_first must follow the last completed round) in ONE launch: a block
 * of N warps owns 32 (x 4) positions, warp i plays worker i; every message is stored into the
 * neighbour's slot as in cerar_ring_round and, besides, handed to the neighbour's warp through
 * shared memory, so a round costs a block barrier instead of a launch and the operands of the
 * next round are already in flight.  Same slots afterwards bit for bit, same counters; but the
 * receiver takes the message from shared memory, not from its slot, so this is not the in-HBM
 * hand-off that cerar_ring_round performs (per steady round 2 reads + 1 write reach memory
 * instead of 3 + 1).  (N > 32: one thread per position runs its N workers in turn.)
 * cerar_allreduce_sim uses it on its own (it measured faster than L launches at every shape
 * tried); only a workspace above 64 MB with N > 32, or with d/c > 65536 not a multiple of 4,
 * goes round by round. */
cerar_status_t cerar_ring_rounds(cerar_plan_t* plan, float* ws, int64_t d, int k_first, int k_last,
                                 cerar_stream_t stream);
cerar_status_t cerar_decode(cerar_plan_t* plan, const float* ws, float* out, int64_t out_stride,
                            int64_t d, float scale, cerar_stream_t stream);
cerar_status_t cerar_allreduce_sim(cerar_plan_t* plan, const float* grads, int64_t grads_stride,
                                   float* out, int64_t out_stride, float* ws, int64_t d,
                                   float scale, cerar_stream_t stream);

/* Same pipeline with HOST gradients and results (pinned memory makes the copies
 * asynchronous and lets them overlap the kernels).  Positions are independent, so
 * the library cuts the job into position slices: while slice i is encoded, sent
 * round the ring and decoded in place on `stream`, slice i+1 is copied in and
 * slice i-1 copied out on two internal copy streams.  worker i's gradient is at
 * h_grads + i*h_grads_stride, its result goes to h_out + i*h_out_stride (d floats
 * each).  ws: device scratch of cerar_workspace_bytes(plan, d) bytes (only three
 * slice-sized parts of it are used).  The call returns after everything is
 * enqueued; `stream` is complete when all results are on the host. */
cerar_status_t cerar_allreduce_sim_host(cerar_plan_t* plan, const float* h_grads,
                                        int64_t h_grads_stride, float* h_out,
                                        int64_t h_out_stride, float* ws, int64_t d,
                                        float scale, cerar_stream_t stream);

/* Variant with the ring on chip (the paper's protocol, a different memory system:
 * not the in-HBM pipeline above and reported separately from it).  One launch
 * carries every position through encode (Sec. II), the L rounds of Algorithm 1
 * and decode (Sec. II-A) with the (c+N) slots of all workers in shared memory,
 * so HBM sees each gradient element once and each result element once and no
 * workspace is needed; the hand-offs between workers happen in shared memory.
 * Same arithmetic and order of operations as the FMA kernels (fp32).  Only for
 * c <= 32 (a multiple of 4, or 5 or 6) and N (c+N) small enough for shared
 * memory: cerar_fused_supported says so, otherwise CERAR_ERR_INVALID_ARG.
 * grads / out as in cerar_allreduce_sim (device, no aliasing).  The counters
 * afterwards describe the L logical rounds. */
cerar_status_t cerar_allreduce_fused(cerar_plan_t* plan, const float* grads, int64_t grads_stride,
                                     float* out, int64_t out_stride, int64_t d, float scale,
                                     cerar_stream_t stream);
int            cerar_fused_supported(const cerar_plan_t* plan);

/* ---- One worker per GPU (the ring the paper runs between machines, Sec. II and
 * Algorithm 1; its Sec. IV names the fused compute/transfer form as future work).
 * Each call serves ONE worker `rank` in 0..N-1, whose state is its own workspace of
 * cerar_rank_workspace_bytes(plan, d) = (c+N+1) (d/c) 4 bytes on this GPU: row
 * ("slot") k-1 receives message k, slot N+j holds delta_{rank,j}.  The one row more
 * than the single-GPU layout is the landing buffer of the transport: the slot that
 * the previous worker writes in round k is not one that its owner reads in round k.
 *
 * cerar_rank_encode: Delta = G U_rank from the worker's gradient `grad` (d floats,
 *   device; may be the D rows of ws itself: ws + (N+1) (d/c)) into slots N+1..N+c.
 * cerar_rank_round: forms message k, x = (y_{k-1} - delta_{k-N}) + delta_k with the
 *   terms that exist (Eq. update_eqns), from this worker's slots and stores it into
 *   slot k-1 of `peer_ws`, the workspace of worker rank+1 (mod N).  peer_ws may point
 *   into another GPU's memory (peer access enabled by the caller): the kernel uses
 *   plain 16-byte stores.  The CALLER orders the rounds: round k of a worker may
 *   start once round k-1 has completed on this worker and on both neighbours (one
 *   barrier per round between all workers is enough); the library keeps no round
 *   state for these calls and waits on nothing.
 * cerar_rank_decode: out (d floats, device) = scale * Y_rank R_rank after round L.
 * cerar_rank_round_slots: the slots round k reads (-1 where the term is absent) and
 *   the landing slot, for callers that schedule or check the transfers themselves.
 * Errors as for the calls above; rank or k out of range is CERAR_ERR_INVALID_ARG /
 * CERAR_ERR_STATE.  All device work is asynchronous on `stream`. */
size_t         cerar_rank_workspace_bytes(const cerar_plan_t* plan, int64_t d);
cerar_status_t cerar_rank_round_slots(const cerar_plan_t* plan, int k, int* slot_prev, int* slot_cancel,
                                      int* slot_add, int* slot_land);
cerar_status_t cerar_rank_encode(cerar_plan_t* plan, int rank, const float* grad, float* ws, int64_t d,
                                 cerar_stream_t stream);
cerar_status_t cerar_rank_round(cerar_plan_t* plan, int rank, const float* ws, float* peer_ws, int64_t d, int k,
                                cerar_stream_t stream);
/* Same message as cerar_rank_round, but written to `msg`, a device buffer of d/c floats of the
 * caller's, instead of the neighbour's memory: for a transport that moves it itself (a
 * send/receive pair between GPUs without peer access, as in the paper's own runs over PCIe);
 * the receiver takes it straight into slot k-1 of its workspace (a contiguous row). */
cerar_status_t cerar_rank_round_msg(cerar_plan_t* plan, int rank, const float* ws, float* msg, int64_t d, int k,
                                    cerar_stream_t stream);
/* Low-precision transport (the paper notes that quantisation is complementary to the coding, Sec. I,
 * Related Work; the combination is this library's): cerar_rank_round_msg_bf16 forms the same message in
 * binary32 and leaves it in `msg` (d/c values of 2 bytes, device memory, 2-byte aligned; 8-byte aligned
 * for the vector path) rounded to bfloat16, nearest with ties to even; cerar_rank_recv_bf16 expands a
 * message that has arrived into slot k-1 of the receiver's workspace.  The worker's own arithmetic
 * and its slots stay binary32; half the bytes cross the transport.  The decoded sum then carries the
 * messages' relative rounding error of 2^-8 amplified by the decoder (kappa_2(M_i)), so this is for
 * well-conditioned designs only. */
cerar_status_t cerar_rank_round_msg_bf16(cerar_plan_t* plan, int rank, const float* ws, uint16_t* msg, int64_t d,
                                         int k, cerar_stream_t stream);
cerar_status_t cerar_rank_recv_bf16(cerar_plan_t* plan, int rank, float* ws, const uint16_t* msg, int64_t d, int k,
                                    cerar_stream_t stream);
/* 8-bit transport (same remark on the paper as for bfloat16: Sec. I, Related Work only notes that
 * quantisation is complementary; the combination is this library's).  cerar_rank_round_msg_fp8 forms the
 * message of round k in binary32 and writes, per tile of CERAR_FP8_TILE consecutive positions, one
 * power-of-two scale 2^e (binary32; e the smallest integer with max|x| 2^-e <= 448 over the tile, 0 for a
 * tile of zeros, kept within [-100, 100]) and per position the 8-bit code of x 2^-e in the e4m3 format
 * (4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest value 448), rounded to nearest
 * with ties to even.  msg: device memory of cerar_fp8_message_bytes(plan, d) bytes, 16-byte aligned:
 * d/c codes, padding to a multiple of 16 bytes, then the scales.  cerar_rank_recv_fp8 expands a message
 * that has arrived into slot k-1 of the receiver's workspace (code value times scale, exact in binary32).
 * A quarter of the bytes cross the transport; every message carries a relative error of up to 2^-4 of
 * its tile's largest magnitude, which the decoder amplifies by about kappa_2(M_i): for designs with a
 * condition number of order 1..100 only (c = N, or the constrained design with a small bound). */
#define CERAR_FP8_TILE 1024
size_t         cerar_fp8_message_bytes(const cerar_plan_t* plan, int64_t d);
cerar_status_t cerar_rank_round_msg_fp8(cerar_plan_t* plan, int rank, const float* ws, void* msg, int64_t d, int k,
                                        cerar_stream_t stream);
cerar_status_t cerar_rank_recv_fp8(cerar_plan_t* plan, int rank, float* ws, const void* msg, int64_t d, int k,
                                   cerar_stream_t stream);
cerar_status_t cerar_rank_decode(cerar_plan_t* plan, int rank, const float* ws, float* out, int64_t d,
                                 float scale, cerar_stream_t stream);

/* All L rounds in one launch per worker, ordered tile by tile instead of round by round.
 * The positions are cut into cerar_ring_tiles(plan, d) tiles (CERAR_RING_TILE positions each,
 * four times that from p = 2^23); per tile a worker keeps two 32-bit
 * counters in its OWN memory that its neighbours write: `landed` (the previous worker has
 * stored message k of that tile here: value epoch (L+1) + k) and `freed` (the next worker
 * has finished round k on that tile, so the slot that message k+1 overwrites may be
 * written).  The kernel polls its local counters, stores messages and counters into the
 * neighbours' memory with system-scope release, and returns when message L has landed
 * too; there is no barrier between rounds.  Every wait is bounded (2 s): on expiry the
 * launch ends and cerar_device_status reports CERAR_ERR_TIMEOUT.
 *   counters must be zero before the first use and `epoch` must grow by one with every
 *   aggregation on the same buffers (nothing is reset in between).  Encode before and
 *   decode after are cerar_rank_encode / cerar_rank_decode; across aggregations the
 *   caller still orders "all decodes done" before "next encode" (stream order or one
 *   barrier per aggregation).
 * cerar_rank_rounds_fused: one worker (this GPU's); landed_local / freed_local: this
 *   worker's counters (cerar_ring_tiles(plan, d) each); landed_next: the NEXT worker's
 *   landed counters, freed_prev: the PREVIOUS worker's freed counters (peer-mapped).  All
 *   N workers' kernels must be running at the same time on N GPUs; never launch several
 *   of them on one GPU.
 * cerar_ring_rounds_fused_local: all N workers of the plan on THIS GPU in one cooperative
 *   launch (N <= 32): ws = host array of the N workspace pointers, counters = device array
 *   of 2 N cerar_ring_tiles(plan, d) words.  This is the form that can be run and checked
 *   on a single GPU. */
#define CERAR_RING_TILE 8192
int64_t        cerar_ring_tiles(const cerar_plan_t* plan, int64_t d);
cerar_status_t cerar_rank_rounds_fused(cerar_plan_t* plan, int rank, const float* ws, float* peer_ws,
                                       const unsigned* landed_local, const unsigned* freed_local,
                                       unsigned* landed_next, unsigned* freed_prev, int64_t d, unsigned epoch,
                                       cerar_stream_t stream);
cerar_status_t cerar_ring_rounds_fused_local(cerar_plan_t* plan, float* const* ws, unsigned* counters, int64_t d,
                                             unsigned epoch, cerar_stream_t stream);

/* The same pipeline as cerar_allreduce_sim for callers that cannot provide a
 * workspace because they cannot allocate device memory at this point: for
 * instance a host program whose framework has already claimed all free memory
 * for its own pool, or a step loop in which cudaMalloc's device-wide
 * synchronisation would stall the other streams.  (The paper has no counterpart:
 * it is a convenience of this library, not part of CERAR.)
 *
 * The workspace is a fixed array inside the library's device image: 16 Mi floats
 * (64 MiB), held by every GPU on which the library's device code is loaded until
 * the process exits.  The call allocates nothing (no cudaMalloc / cudaFree, no
 * allocating library routine).  Requests that need more than that, i.e.
 * cerar_workspace_bytes(plan, d) > 64 MiB, are refused with
 * CERAR_ERR_TOO_LARGE and a message saying how much was needed.
 *
 * grads / out: device buffers as in cerar_allreduce_sim; they must not alias each
 * other or the workspace (the in-place forms are not available here).  The
 * device the plan was created on must be current.
 * First call on a device: after checking that the plan has device copies and that
 * its device is current, looks up the array's device address (once per device).
 * The CUDA runtime may load this part of the library's device image only then, so
 * that first call is where the 64 MiB are actually reserved on the device: it can
 * fail (CERAR_ERR_NOMEM / CERAR_ERR_CUDA) if the device has no room left.  A caller
 * whose framework is about to claim all free memory makes one call before that
 * happens.  Make the first call before any stream capture begins.
 * All calls share the one array, which keeps whatever the previous call left in
 * it.  Nothing needs clearing between calls (every slot is written before it is
 * read), but two calls whose kernels overlap on the GPU (different streams, or
 * different host threads) race on it: serialise them. */
cerar_status_t cerar_allreduce_sim_static(cerar_plan_t* plan, const float* grads, int64_t grads_stride,
                                          float* out, int64_t out_stride, int64_t d, float scale,
                                          cerar_stream_t stream);

/* Rate counters (Sec. II-B: communication rate 1+(N-2)/c = bytes_forwarded /
 * bytes_gradient after L rounds; storage rate 1+N/c = bytes_stored / bytes_gradient). */
cerar_status_t cerar_get_counters(const cerar_plan_t* plan, cerar_counters_t* out);

/* Number of kernels this library has launched through this plan so far. */
uint64_t       cerar_launch_count(const cerar_plan_t* plan);

/* 1 if this library is the checked build (libcerar_checked.so, compiled with
 * -DCERAR_BOUNDS_CHECK), 0 otherwise.  In the checked build the kernels of the in-HBM
 * pipeline that use plain loads, stores and 1-D bulk copies (the FMA contractions, the ring
 * rounds in all their forms, the tensor-core contraction on rows that are not 16-byte
 * aligned) compare every address they form with the extent of its buffer;
 * an address outside is not accessed, and the next cerar_device_status returns
 * CERAR_ERR_BOUNDS.  It is the stand-in for a memory checker where none can be run; it
 * costs bandwidth and is not what bench.py times.  The paper has no counterpart. */
int            cerar_build_is_checked(void);

/* Synchronises `stream` and reports CERAR_ERR_TIMEOUT if a kernel of this plan
 * gave up on one of its bounded device-side waits since the last check (the
 * results of that call are then invalid); CERAR_OK otherwise. */
cerar_status_t cerar_device_status(cerar_plan_t* plan, cerar_stream_t stream);

/* Failure-path self test: launches a one-warp kernel whose bounded wait cannot be
 * satisfied (nothing ever arrives on its barrier), so that it gives up after
 * limit_ms (1..1000) and flags the status word like the pipelined kernels do when a
 * wait runs out; the next cerar_device_status then returns CERAR_ERR_TIMEOUT and
 * clears the flag.  The device context stays usable. */
cerar_status_t cerar_selftest_wait_timeout(cerar_plan_t* plan, int limit_ms, cerar_stream_t stream);

/* Kernel selection for encode/decode: 0 = automatic, 1 = plain per-position
 * kernel, 2 = staged FMA kernel, 3 = tensor-core (3 x TF32) kernel; a forced
 * kernel that cannot take the shape makes the call fail instead of falling
 * back.  Returns the previous value. */
int            cerar_set_kernel_mode(cerar_plan_t* plan, int mode);

/* Process-wide tuning knobs, for experiments and tests; value 0 restores the default.
 *   "kc", "stages", "jt", "slabs"   staged FMA kernel: input rows per pipeline stage, stages,
 *                                   outputs per thread (4, 8, 16 or 20), position slabs per CTA
 *   "tc_kc", "tc_stages"            tensor-core kernels: rows per stage, stages
 *   "tc_variant"                    1 = always tiles of 128 positions (default: tiles of 256
 *                                   positions for c <= 64); 2 / 3 = tiles of 256 with one /
 *                                   two MMA issuers per half
 *   "tc_split"                      tensor-core kernels with tiles of 256 positions: 1 = each splitter warp
 *                                   takes all rows of one half of the tile, 2 = half of the rows of both
 *                                   halves (default: 1 where a tile has two or more chunks)
 *   "tc_epi"                        epilogue of the tensor-core kernels: 1 = a group of four warps
 *                                   per tile parity, 2 = all eight warps on every tile, 3 = one group
 *                                   of four warps for all tiles (one output tile less in shared
 *                                   memory), 4 = two groups (default: chosen by shape)
 *   "round_split"                   ring round with few positions: 1 = never, 2 = always one thread per
 *                                   group of 4 workers (default: where the plain grid has at most 148 blocks)
 *   "checked_shrink"                checked build, tests only: the extents that stores are checked
 *                                   against end this many floats early (the buffers do not change)
 *   "ring_wait_ms"                  limit of the waits of the fused ring rounds (default 2000)
 *   "ring_tile"                     positions per tile of the fused ring rounds (a multiple of 4;
 *                                   default 8192, 32768 from p = 2^23); set before sizing counters
 *   "pdl_off"                       1 = launch without programmatic stream serialization
 *   "serpentine_off"                1 = every ring round walks the positions upwards
 *   "tc_min_c"                      smallest c that runs on the tensor-core kernel (default 24; 17 for
 *                                   rows that do not start on 16-byte boundaries)
 *   "staged_unaligned_off"          1 = rows that do not start on 16-byte boundaries never run on the
 *                                   staged FMA kernel (they take the tiled plain-load kernel)
 *   "tc_unaligned_off"              1 = rows that do not start on 16-byte boundaries never run on the
 *                                   tensor-core kernel (they take the tiled plain-load kernel)
 *   "rounds_one_launch_off"         1 = cerar_allreduce_sim always launches round by round
 *   "rounds_one_launch_mb"          if set, cerar_allreduce_sim runs the rounds in one launch exactly
 *                                   for workspaces up to this many MB (default rule: see
 *                                   cerar_ring_rounds)
 *   "rounds_coop_shape"             vectors per lane of the warp-per-worker kernel (0 = automatic, 1, 2)
 *   "rounds_hints"                  L2 residency hints of that kernel (0 = automatic: from N = 8, 1 = off, 2 = on)
 *   "rounds_multi_form"             kernel of cerar_ring_rounds: 0 = warp per worker (16-byte
 *                                   accesses where there are enough positions), 3 = the same with
 *                                   4-byte accesses, 1 = thread per position
 * Returns 0, or -1 for an unknown name. */
int            cerar_set_tuning(const char* name, int value);

const char*    cerar_status_string(cerar_status_t s);
const char*    cerar_last_error(void);   /* thread-local detail of the last failure */

#ifdef __cplusplus
}
#endif
#endif /* CERAR_H_ */
