/*
 * turboboa.h -- C ABI of the B200 (sm_100a) implementation of the TurboBoA
 * out-channel-group weight quantizer and of its prerequisites (calibration
 * Hessians, inverse Cholesky factors, propagated-error operands).
 *
 * General conventions
 *   - Unless a parameter says "host", every tensor pointer is a DEVICE pointer
 *     owned by the caller.  The library never allocates or frees device
 *     memory: scratch comes from the caller as a workspace whose size the
 *     matching *_workspace() function returns (bytes; the pointer must be
 *     256-byte aligned).
 *   - Matrices are dense row-major.  A weight W is [d_out][d_in], one row per
 *     out-channel; attention heads are contiguous blocks of d_head rows
 *     (Algorithm 1 takes W in R^{H x d_h x d}).
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it
 *     and the call returns without synchronising.  Inputs are never modified.
 *   - Shape, pointer and alignment errors are found on the host before any
 *     launch and reported through the return value; nothing is enqueued in
 *     that case.  Numerical failures (a non-positive pivot) are reported in
 *     device words described with each call.  No call aborts, traps or throws.
 *   - One GPU per call: the current device of the calling thread.
 */
#ifndef TURBOBOA_H_
#define TURBOBOA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TB_OK = 0,
  TB_ERR_INVALID_ARG = 1, /* NULL pointer, bad shape, misaligned pointer        */
  TB_ERR_UNSUPPORTED = 2, /* a valid request outside the implemented range      */
  TB_ERR_WORKSPACE = 3,   /* workspace NULL, misaligned or too small            */
  TB_ERR_NOT_SPD = 4,     /* reserved for host-side checks of info words        */
  TB_ERR_CUDA = 5,        /* a CUDA runtime call failed (launch, attribute)     */
  TB_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (see
                             tb_device_error_flag)                              */
} tb_status;

typedef enum { TB_F32 = 0, TB_BF16 = 1 } tb_dtype;

/* flags of tb_layer_desc */
enum {
  TB_F_ADAPTIVE_GRID = 1, /* grid chosen per out-channel group just before it is
                             quantized (Algorithm 1, grid step; Section 3.3).  Off:
                             the grid of every row is chosen once from the
                             original weights (the fixed grid of BoA).         */
  TB_F_CD_REFINE = 2,     /* coordinate-descent scale refinement after the loop
                             (Algorithm 1, refinement; Proposition 3.3)        */
  TB_F_DYNAMIC_GRID = 4   /* variant for column groups (which the paper does not
                             have): the (scale, zero) of a column group is searched
                             when the column sweep arrives at the group, from the
                             group's current values, i.e. after the error feedback
                             of every earlier column of the row (same candidates,
                             same score).  Overrides the two grid modes above; with
                             quant_group = 0 it is TB_F_ADAPTIVE_GRID.  Groups of at
                             most 128 columns.  Runs group by group (one grid
                             search, one panel, one update per group), not through
                             the fused sweep kernel.                            */
};

/* Problem description of one projection (Algorithm 1, inputs). */
typedef struct {
  int d_out, d_in;   /* W is [d_out][d_in]; d_in must be a multiple of 128       */
  int n_heads;       /* H; n_heads * d_head == d_out                             */
  int d_head;        /* d_h                                                      */
  int n_hin;         /* 1: one H_in shared by all heads (W_Q, W_K rows of
                        Table 1); n_heads: one per head (the W_V row)            */
  int bits;          /* b in 2..8; codes lie in {0 .. 2^b - 1}                   */
  int quant_group;   /* columns per (scale, zero) pair: 0 = the whole row, else
                        a multiple of 32 that divides d_in                       */
  int out_block;     /* N of Algorithm 1: out-channels of a head quantized
                        jointly; must divide d_head.  1 = BoA's sequential rule  */
  int n_cand;        /* grid candidates 1..32; candidate k clips the row's
                        min/max range by p_k = 1 - k/32                          */
  int cd_iters;      /* passes of Algorithm 3 (the paper uses 1)                 */
  unsigned flags;    /* TB_F_*                                                   */
} tb_layer_desc;

/* Counters written by tb_quantize_layer (device memory, 64 bytes). */
typedef struct {
  unsigned long long near_tie_codes; /* rounding decisions whose pre-rounding value
                                        lay within 1e-6 of a boundary between two
                                        distinct codes                           */
  unsigned long long clamped_codes;  /* decisions that hit 0 or 2^b - 1 by clamp  */
  unsigned long long column_steps;   /* dependent column steps executed          */
  unsigned long long reserved[5];
} tb_stats;

const char* tb_status_string(tb_status st);

/* --------------------------------------------------------------------------
 * Calibration Hessians (Table 1; Algorithm 1, statistics steps).
 * -------------------------------------------------------------------------- */

/* H += X^T X, the un-normalised running sum of the input Hessian X X^T of
 * Table 1 (X here is token-major [n_tok][d], the transpose of the paper's X).
 * H: [d][d] float, fully written (both triangles).  X: bf16 or float.
 * d must be a multiple of 8.  May be called repeatedly over token chunks. */
tb_status tb_accumulate_hessian(float* H, const void* X, tb_dtype x_type,
                                long long n_tok, int d, void* stream);

/* The bf16 path of tb_accumulate_hessian runs on the tensor cores and waits on
 * hardware barriers with a bound of about two seconds.  If a bound ever runs
 * out the kernel gives up (H is then incomplete) and raises a device word that
 * this call reads and clears: 0 = no such event, 1 = a wait ran out
 * (TB_ERR_TIMEOUT), -1 = the word could not be read.  Synchronises the device.
 * No counterpart in the paper. */
int tb_device_error_flag(void);

/* Self-test of that mechanism, with no counterpart in the paper: launches one
 * small CTA that waits, through the library's bounded wait, on a hardware barrier
 * at which nothing ever arrives, with a budget of budget_cycles SM clock cycles
 * (0 .. 2e8, i.e. at most about 0.1 s).  The wait gives up, the kernel returns
 * normally, *gave_up (device int, may be NULL) becomes 1 and the next
 * tb_device_error_flag() returns 1.  Nothing faults and the context stays usable. */
tb_status tb_selftest_bounded_wait(long long budget_cycles, int* gave_up, void* stream);

/* R += alpha * (X - Xfp)^T X, the deviation correlation alpha (X - X~) X^T of
 * Algorithm 1 (deviation step) in the same un-normalised form: R[a][b] accumulates
 * alpha * sum_t (x_t[a] - xfp_t[a]) * x_t[b].  R: [d][d] float, not symmetric.
 * bf16 activations run on the tensor cores (same bounded waits and error word
 * as tb_accumulate_hessian): the deviation is split into two bf16 pieces held
 * in ws, a DEVICE workspace of tb_accumulate_cross_workspace bytes (256-byte
 * aligned; 0 bytes and ws = NULL for float activations, which run on the FP32
 * pipe).  X, Xfp and R must be 16-byte aligned for bf16. */
size_t tb_accumulate_cross_workspace(tb_dtype x_type, long long n_tok, int d);
tb_status tb_accumulate_cross(float* R, const void* X, const void* Xfp, tb_dtype x_type,
                              long long n_tok, int d, float alpha, void* ws, size_t ws_bytes,
                              void* stream);

/* H <- H / n_total + damp * mean(diag(H / n_total)) * I ; R <- R / n_total when
 * R is not NULL.  The paper does not mention damping; damp = 0 reproduces
 * Table 1 up to the 1/n_total normalisation, which changes no quantized
 * weight.  Optionally keeps the undamped H / n_total in Hsum_out (or NULL). */
tb_status tb_finalize_hessian(float* H, float* R, float* Hsum_out, int d, long long n_total,
                              float damp, void* stream);

/* Out-channel Hessians of Table 1 from the partner projection G
 * ([g_heads * d_head][d] float, one block of d_head rows per head):
 *   Hsum != NULL: block b gives G_b Hsum G_b^T  (= K_h^T K_h when W_Q is
 *                 quantized and G = W_K, since K_h = (W_K,h X)^T; likewise
 *                 Q_h^T Q_h with G = W_Q);
 *   Hsum == NULL: block b gives G_b G_b^T (W_out,h^T W_out,h with G = W_out^T).
 * If g_heads > n_heads (grouped-query attention, key/value side) head h sums
 * the blocks of its g_heads / n_heads query heads; if g_heads < n_heads head h
 * takes block h / (n_heads / g_heads).  Then damp * mean(diag) is added to
 * the diagonal of each head.  H_out: [n_heads][d_head][d_head] float.
 * Workspace: tb_build_hout_workspace bytes. */
size_t tb_build_hout_workspace(int g_heads, int d_head, int d);
tb_status tb_build_hout(float* H_out, const float* G, const float* Hsum, int n_heads,
                        int g_heads, int d_head, int d, float damp, void* ws, size_t ws_bytes,
                        void* stream);

/* --------------------------------------------------------------------------
 * Factors (Eq. 2): U upper triangular with H^{-1} = U^T U.
 * -------------------------------------------------------------------------- */

/* H: [n_batch][d][d] float, symmetric positive definite (only read).
 * U: [n_batch][d][d] float; the strictly lower triangle is written as zeros.
 * Hinv (optional, may be NULL): [n_batch][d][d] float, U^T U.
 * info (device, [n_batch] int): 0, or the 1-based index (counted in the
 * elimination order, which runs from the last row to the first) of the first
 * pivot that was not positive; U of that matrix is then meaningless.
 * For matrices of 1024 columns or more the work is spread over helper streams
 * of the library (per device, created at the first such call and kept until
 * exit; the chain of panel factorisations on one of the highest priority,
 * trailing updates and the inverse of the finished blocks beside it), forked
 * from and joined back into `stream` by events.  All calls on a device share
 * these streams and events: do not factor such sizes on one device from two
 * host threads at once. */
size_t tb_factor_workspace(int n_batch, int d);
tb_status tb_factor(const float* H, int n_batch, int d, float* U, float* Hinv, int* info,
                    void* ws, size_t ws_bytes, void* stream);

/* tb_factor without a caller-provided workspace and without any allocation.
 * The paper has no counterpart: this entry point exists for callers that must
 * not, or cannot, obtain device memory when they need a factor -- a process
 * that has handed all free device memory to its own pool at start-up (a later
 * cudaMalloc would fail), or a latency-critical loop in which cudaMalloc /
 * cudaFree are banned because they synchronise the whole device.
 *
 * The scratch is a fixed array of tb_factor_static_capacity() bytes (32 MiB)
 * inside the library; every GPU on which the library is loaded holds it until
 * the process exits.  Inputs and outputs are still the caller's.  Same results
 * and same info semantics as tb_factor (no Hinv output).  A problem whose
 * tb_factor_workspace(n_batch, d) exceeds the capacity is rejected with
 * TB_ERR_UNSUPPORTED before anything is enqueued (64 matrices of 128 x 128, or
 * one of 1024 x 1024, fit).
 *
 * The first call on each device looks up the array's device address (the
 * device must be current); make that first call outside any stream capture.
 * Under CUDA's lazy module loading the array may only come into existence at
 * that first look-up, so make the first call at start-up, while the device
 * still has 32 MiB free: a process that first fills the device and only then
 * calls this for the first time can get TB_ERR_CUDA.  The address is kept per
 * device ordinal for the life of the process (no lock: make the first call of
 * a device from one thread).
 * All calls share the one array: it keeps whatever the previous call left
 * (the call clears what it needs zeroed), and two calls whose work overlaps on
 * the GPU -- different streams, or different host threads -- race on it.
 * Calls on one stream are safe.  No cudaMalloc, cudaFree or other allocating
 * routine is called. */
size_t tb_factor_static_capacity(void);
tb_status tb_factor_static(const float* H, int n_batch, int d, float* U, int* info, void* stream);

/* Operands of the propagated-error terms from R and U_in:
 *   P = ((R U^T) masked to its strictly upper triangle) U   (Algorithm 2, masked operand)
 *   C = R U^T U = R H_in^{-1}                               (Proposition 3.2)
 * All [n_batch][d][d] float.  U must have a zero strictly-lower triangle.
 * The three products run in double; P and C are rounded to float once. */
size_t tb_prepare_correction_workspace(int n_batch, int d);
tb_status tb_prepare_correction(const float* R, const float* U_in, int n_batch, int d, float* P,
                                float* C, void* ws, size_t ws_bytes, void* stream);

/* --------------------------------------------------------------------------
 * The quantizer (Algorithm 1, the group loop and its closing steps, for one
 * projection W).
 * -------------------------------------------------------------------------- */

/* For every head, and for every group of out_block rows in turn: choose the
 * grid of the group's rows (grid step), run the column sweep with in-row error
 * feedback through U_in (Algorithm 2; Eq. 2), then update the rows of
 * the head not yet quantized with the closed-form joint compensation
 * (Propositions 3.1 and 3.2).  After the loop optionally refine the
 * scales by coordinate descent (Proposition 3.3 / Algorithm 3) and
 * write Q = diag(s)(W_int - z) (final step).
 *
 * Inputs
 *   W      [d_out][d_in] float
 *   H_in   [n_hin][d_in][d_in] float, symmetric (for groups of at most 128
 *          columns the grid search reads the upper triangle of its diagonal
 *          blocks only)
 *   U_in   [n_hin][d_in][d_in] float, upper factor of H_in^{-1}
 *   H_out  [n_heads][d_head][d_head] float, or NULL for the identity (the GPTQ /
 *          GPTAQ row of Table 1: every row of a head is quantized at once and
 *          there is no compensation); U_out likewise (NULL iff H_out is NULL)
 *   R, P, C  [n_hin][d_in][d_in] float each, or all three NULL (no propagated
 *          error: the first block of a model)
 * Outputs
 *   codes  [d_out][d_in] unsigned char, W_int
 *   scales [d_out][n_g] float, n_g = d_in / quant_group (1 if quant_group = 0)
 *   zeros  [d_out][n_g] int, integer zero-points z (the paper's grid has none;
 *          every formula holds with W_int replaced by W_int - z)
 *   cand   [d_out][n_g] unsigned char or NULL: index k of the chosen grid candidate
 *   W_hat  [d_out][d_in] float or NULL: Q
 *   W_comp [d_out][d_in] double or NULL: the compensated weights, row r as it stood
 *          when its group was taken for quantization (the rows W~_B that Algorithm 1
 *          hands to the sweep: the original row plus every joint compensation it
 *          received from the groups of its head quantized before it)
 *   loss   [n_heads] double or NULL: tr(dW H_in dW^T H_out) + 2 tr(H_out W R dW^T),
 *          dW = Q - W (the objective in the proofs of Propositions 3.1 / 3.2)
 *   stats  tb_stats (device) or NULL
 * The arithmetic of the loop is IEEE double precision: codes are integer
 * decisions taken inside an error-feedback chain d_in steps long, and they
 * only reproduce across implementations when the chain is carried in double. */
size_t tb_quantize_layer_workspace(const tb_layer_desc* desc, int with_r, int with_loss);
tb_status tb_quantize_layer(const tb_layer_desc* desc, const float* W, const float* H_in,
                            const float* U_in, const float* H_out, const float* U_out,
                            const float* R, const float* P, const float* C,
                            unsigned char* codes, float* scales, int* zeros, unsigned char* cand,
                            float* W_hat, double* W_comp, double* loss, tb_stats* stats, void* ws,
                            size_t ws_bytes, void* stream);

/* --------------------------------------------------------------------------
 * Bit-packed integer weights.  Section 2.1 writes the quantized weight as
 * Q = diag(s) W_int with W_int in {0 .. 2^b - 1}: what is stored and shipped is
 * W_int at b bits per weight, with the scales (and here the zero-points).
 * -------------------------------------------------------------------------- */

/* Packed format: every row is a little-endian bit stream; code j of the row
 * occupies bits [j b, (j + 1) b), counted from the least significant bit of the
 * row's first 32-bit word (a code may straddle two words when b does not divide
 * 32).  A row takes d_in * b / 32 words; d_in must be a multiple of 32.
 * tb_packed_bytes: size of the packed matrix, 0 for an invalid shape.
 * tb_pack_codes: codes [d_out][d_in] unsigned char (16-byte aligned, values
 * below 2^bits) -> packed.  bits in 2..8. */
size_t tb_packed_bytes(int d_out, int d_in, int bits);
tb_status tb_pack_codes(const unsigned char* codes, int d_out, int d_in, int bits,
                        unsigned int* packed, void* stream);

/* Unpacks, dequantizes and optionally compares in one pass over the packed
 * matrix: Q[r][j] = scales[r][g] * (code - zeros[r][g]) in float, g = j /
 * quant_group (the final step of Algorithm 1 from what a deployment holds:
 * packed codes, float scales, integer zero-points).
 *   codes_out, W_hat_out  [d_out][d_in], either may be NULL
 *   codes_ref             or NULL: unpacked codes are compared byte for byte
 *   W_hat_ref             or NULL: |Q - ref| <= tol * |ref| is checked per
 *                         element (tb_quantize_layer forms W_hat from the scales
 *                         in double and rounds once, so the two may differ by an
 *                         ulp: tol = 2^-22 passes, 0 asks for equal bits)
 *   mismatch              device, 2 words, required when a reference is given:
 *                         [0] codes that differ, [1] values beyond tol; cleared
 *                         by the call */
tb_status tb_unpack_dequant(const unsigned int* packed, const float* scales, const int* zeros,
                            int d_out, int d_in, int bits, int quant_group,
                            unsigned char* codes_out, float* W_hat_out,
                            const unsigned char* codes_ref, const float* W_hat_ref, float tol,
                            unsigned long long* mismatch, void* stream);

/* --------------------------------------------------------------------------
 * Block level: Algorithm 1's outer loop over the projections of an attention
 * layer.
 * -------------------------------------------------------------------------- */

/* One prepared projection: exactly the arguments of tb_quantize_layer. */
typedef struct {
  tb_layer_desc desc;
  const float *W, *H_in, *U_in, *H_out, *U_out, *R, *P, *C;
  unsigned char* codes;
  float* scales;
  int* zeros;
  unsigned char* cand;
  float* W_hat;
  double* W_comp;
  double* loss;
  tb_stats* stats;
  void* ws;
  size_t ws_bytes;
} tb_projection_job;

/* Quantizes up to 5 prepared projections (Algorithm 1 loops over W_Q, W_K, W_V;
 * heads and projections are independent problems).  concurrent = 0: one after
 * the other on `stream`.  concurrent != 0: job 0 on `stream`, the others on
 * helper streams of the library (per device, created at the first such call and
 * kept until exit), forked from and joined back into `stream` by events, so that
 * the latency-bound phases of one projection run beside the throughput-bound
 * phases of another; every job then needs a workspace of its own.  Results are
 * those of separate tb_quantize_layer calls, bit for bit.  All descriptions and
 * workspaces are checked before the first launch. */
tb_status tb_quantize_block(const tb_projection_job* jobs, int n_jobs, int concurrent, void* stream);

/* A whole attention layer from its calibration activations (Algorithm 1 for
 * W_Q, W_K, W_V, and the output projection in the H_out = I mode of Table 1's
 * GPTQ row). */
typedef struct {
  int d_model;     /* width d of the attention input; W_Q, W_K, W_V have d columns  */
  int n_q_heads;   /* W_Q is [n_q_heads * d_head][d]; W_O is [d][n_q_heads * d_head] */
  int n_kv_heads;  /* W_K, W_V are [n_kv_heads * d_head][d]; divides n_q_heads
                      (grouped-query attention when smaller)                        */
  int d_head;
  int bits, quant_group, out_block, n_cand, cd_iters; /* as in tb_layer_desc        */
  unsigned flags;  /* TB_F_*                                                        */
  long long n_tok; /* calibration tokens in every activation tensor                 */
  float damp;      /* damping of every Hessian built here (see tb_finalize_hessian) */
  float alpha;     /* stabilisation coefficient of R (Algorithm 1, deviation step)  */
  int on_host;     /* 0: every pointer of tb_attention_io is device memory;
                      1: every pointer is host memory (pinned memory makes the
                      copies asynchronous) and the call synchronises `stream`      */
  int concurrent;  /* != 0: independent parts on helper streams side by side        */
} tb_attention_desc;

typedef struct {
  /* activations, bf16, token-major */
  const void* X;      /* [n_tok][d]  input of W_Q, W_K, W_V on the quantized path                  */
  const void* X_fp;   /* same shape or NULL: the full-precision path's input X~; when given,
                         R = alpha (X - X~) X^T enters W_Q and W_K (and W_V if X_v is NULL)       */
  const void* X_v;    /* [n_kv_heads][n_tok][d] or NULL: the attention-weighted inputs A_h X of
                         the value projection, one H_in per head (Table 1, W_V row; no R then);
                         NULL: W_V shares the Hessian of X                                        */
  const void* X_o;    /* [n_tok][n_q_heads * d_head]  input of the output projection             */
  const void* X_o_fp; /* same shape or NULL: its full-precision twin (R of the output projection) */
  /* weights, float, in the order q, k, v, o */
  const float* W[4];
  /* results per projection, same order; W_hat and loss entries may be NULL */
  unsigned char* codes[4];
  float* scales[4];
  int* zeros[4];
  float* W_hat[4];
  double* loss[4];    /* [n_heads] of that projection (1 for the output projection)               */
  int* info;          /* tb_attention_layer_info_count ints or NULL: the info words of every
                         factorisation (H_in of X, of X_o, of each X_v head, then H_out of the
                         q, k, v heads); 0 = positive definite                                    */
} tb_attention_io;

/* H_out follows Table 1: W_Q against K_h^T K_h (from W_K and the Hessian of X),
 * W_K against Q_h^T Q_h (from W_Q), W_V against W_out,h^T W_out,h (the head's
 * columns of W_O); with grouped-query attention a query head takes the block of
 * its key/value head and a key/value head the sum over its query heads.  The
 * output projection runs with H_out = NULL (all rows at once, GPTAQ if X_o_fp
 * is given).  The workspace query only looks at which optional pointers of io
 * are non-NULL.  With on_host = 1 the activations cross to the device in pieces
 * of 16384 tokens on a copy stream (eight staging slots in the workspace) while
 * the Hessian of the pieces already there accumulates on a stream of its own
 * (the Hessian's sums do not depend on the pieces; the deviation correlation
 * adds its two bf16 pieces per call, so its float sums differ from a single
 * call's in the last bits).  The inputs cross in the order X, X_o, then the
 * value heads of X_v; factors and quantizer calls follow each finished Hessian
 * on the caller's stream (q, o and k are quantized while the value heads still
 * cross, each value head is factored alone, with the batched factor's numbers),
 * every projection's results are copied back as soon as it is done, and the call returns TB_ERR_NOT_SPD /
 * TB_ERR_TIMEOUT like tb_quantize_from_host; with on_host = 0 it only enqueues
 * and the caller reads `info`.  Helper streams as for tb_quantize_block. */
int tb_attention_layer_info_count(const tb_attention_desc* desc, int per_head_v);
size_t tb_attention_layer_workspace(const tb_attention_desc* desc, const tb_attention_io* io);
tb_status tb_attention_layer(const tb_attention_desc* desc, const tb_attention_io* io, void* ws,
                             size_t ws_bytes, void* stream);

/* Profiling aid with no counterpart in the paper.  While enabled, every
 * tb_quantize_layer call records CUDA events on its stream around its phases;
 * tb_profile_read waits for them, adds the elapsed milliseconds per phase into
 * ms_by_phase[0..n) (host memory; order: setup, grid search, column sweep,
 * compensation, coordinate descent, output, loss, then the prerequisites as
 * tb_attention_layer runs them: Hessian accumulation, deviation correlation,
 * H_out build, factorisations, propagated-error operands, result copies),
 * forgets them and returns the number of phases (13).  Phases that ran side by
 * side on different streams each count their own elapsed time.  Process-wide
 * and not thread-safe; off by default. */
void tb_profile_enable(int on);
int tb_profile_read(double* ms_by_phase, int n);

/* Number of kernels the library has launched in this process so far (every launch
 * of one of its own kernels counts once; copies and memsets do not).  Not
 * thread-safe.  No counterpart in the paper. */
unsigned long long tb_launch_count(void);

/* Whole path for one projection from HOST buffers: copies X (and G) to the
 * device, accumulates and finalises H_in, builds H_out, factors both, runs
 * tb_quantize_layer and copies codes / scales / zeros / W_hat / loss back.
 * Every *_host pointer is host memory (pinned memory makes the copies
 * asynchronous); dev_ws is a DEVICE workspace of
 * tb_quantize_from_host_workspace bytes.  The call synchronises the stream
 * before it returns.  A helper stream of the library (one per device, created
 * at the first call and kept until exit), forked from and joined back into
 * `stream` by events, carries X to the device in pieces while the Hessian of
 * the pieces that have arrived accumulates, and later runs the H_out build and
 * its factor beside the factor of H_in.  X_host is bf16 [n_tok][d_in]; G_host is the partner
 * projection [g_heads*d_head][d_in] float or NULL (then H_out = identity).
 * The description is validated in full before anything is enqueued.  If a step
 * fails after that, the call still joins its helper stream and waits for every
 * copy it started before it returns the error, so the host buffers are never
 * in use on return.  Returns TB_ERR_NOT_SPD if a factorisation met a
 * non-positive pivot and TB_ERR_TIMEOUT if a bounded wait of a tensor-core
 * kernel ran out (it reads and clears the word of tb_device_error_flag). */
size_t tb_quantize_from_host_workspace(const tb_layer_desc* desc, long long n_tok, int g_heads);
tb_status tb_quantize_from_host(const tb_layer_desc* desc, const float* W_host,
                                const void* X_host, long long n_tok, const float* G_host,
                                int g_heads, float damp_in, float damp_out,
                                unsigned char* codes_host, float* scales_host, int* zeros_host,
                                float* W_hat_host, double* loss_host, void* dev_ws,
                                size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TURBOBOA_H_ */
