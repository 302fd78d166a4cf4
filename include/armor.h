/*
 * armor.h -- C ABI of the B200 (sm_100a) implementation of ARMOR's per-layer
 * block coordinate descent (arXiv 2510.05528).
 *
 * One linear layer W [d_out, d_in] is factorised as  W ~ A * S * B  with
 * block-diagonal wrappers A, B (blocks of d_block x d_block) around an N:M
 * sparse core S = W' (.) M  (Section 3.1 of the paper).  The library minimises
 * the layer-wise proxy loss  L = tr(E H_w E^T),  E = W - A S B,  where
 * H_w = diag(X^T X) is the paper's weighting (Eq. proxy_loss, Section 3.2) and
 * H_w = X^T X is the full-Gram generalisation (the mode the benchmark times).
 *
 * Conventions for every call
 *   - All d_* pointers are DEVICE pointers owned by the caller; tensors are
 *     row-major and contiguous unless a leading dimension is given.
 *   - The library allocates no device memory.  Scratch comes from the
 *     workspace handed to armor_create (size from armor_workspace_bytes).
 *   - Work is enqueued on the given stream; no call synchronises the device.
 *     Calls on one context must be issued in stream order (they share the
 *     workspace).
 *   - Argument errors are returned immediately.  Conditions found on the
 *     device (a block that is not positive definite, a bounded wait that ran
 *     out) are recorded in a device status buffer; read it with
 *     armor_get_device_status after synchronising the stream yourself.
 *   - A, B: [d/d_block, d_block, d_block] fp32.  S: [d_out, d_in] fp32 with
 *     zeros outside the mask.  M: one byte per group of m_group consecutive
 *     columns, uint8 [d_out, d_in/m_group]; bit p set <=> column m*c+p kept.
 *   - N:M patterns: 2:4, and 4:8, 5:8, 6:8 (Section 4.4 of the paper names them).
 */
#ifndef ARMOR_H
#define ARMOR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct armor_ctx armor_ctx;
typedef struct CUstream_st* armor_stream_t; /* == cudaStream_t */

typedef enum {
  ARMOR_OK = 0,
  ARMOR_ERR_INVALID_ARG = 1,
  ARMOR_ERR_SHAPE = 2,
  ARMOR_ERR_WORKSPACE = 3,
  ARMOR_ERR_CUDA = 4,
  ARMOR_ERR_NOT_SPD = 5,
  ARMOR_ERR_TIMEOUT = 6,
  ARMOR_ERR_UNSUPPORTED = 7,
  ARMOR_ERR_TOO_LARGE = 8
} armor_status;

enum { ARMOR_H_FULL = 0, ARMOR_H_DIAG = 1 };
/* Group selection of the sparse-core update (Section 3.3.2; the other three are the ablation of Appendix E.1) */
enum { ARMOR_SELECT_L1_RANDOM = 0, ARMOR_SELECT_L1_GREEDY = 1, ARMOR_SELECT_UNIFORM_RANDOM = 2, ARMOR_SELECT_L2_RANDOM = 3 };
enum { ARMOR_S_EXACT = 0, ARMOR_S_BETA = 1 };
/* Wrapper updates: exact (proximal) block solves, or the paper's own gradient steps with the 1/beta steps of
 * Eq. lrA and Eq. lrB (Algorithm 2; defined for the diagonal weighting, so ARMOR_AB_GD needs ARMOR_H_DIAG). */
enum { ARMOR_AB_EXACT = 0, ARMOR_AB_GD = 1, ARMOR_AB_ADAM = 2 };
/* ARMOR_AB_ADAM: what the paper runs in practice (Section 3.3.1): one joint Adam step on A, B and W' per
 * iteration in place of the three sequential updates (s_step is then ignored), followed by the sparse-core
 * update.  The moment estimates live in the context's workspace; armor_init and a call with t_first == 0
 * reset them, later calls on the same context continue them. */
/* How the dense contractions (Gram, .H) are evaluated on the tensor cores:
 *   FP32X3 : operands split into tf32 high and low parts, three tcgen05 passes
 *            accumulated in fp32 -- fp32-grade results (the parity mode);
 *   TF32   : one pass, operands rounded to tf32 (10-bit mantissa);
 *   SIMT   : fp32 CUDA-core reference path (slow; for debugging and checks);
 *   FP16X3 : operands scaled by exact powers of two into the fp16 range and split into fp16 high and low
 *            parts (22 significant bits, as two tf32 parts), three kind::f16 passes at twice the tf32 rate,
 *            the accumulator rescaled in the epilogue -- fp32-grade results like FP32X3.  The products
 *            with the block-diagonal wrappers are the same in both modes. */
enum { ARMOR_PREC_FP32X3 = 0, ARMOR_PREC_TF32 = 1, ARMOR_PREC_SIMT = 2, ARMOR_PREC_FP16X3 = 3 };
enum { ARMOR_PHASE_A = 1, ARMOR_PHASE_B = 2, ARMOR_PHASE_S = 4, ARMOR_PHASE_MASK = 8 };
enum { ARMOR_DTYPE_F32 = 0, ARMOR_DTYPE_BF16 = 1, ARMOR_DTYPE_BF16_SPARSE = 2 };

typedef struct {
  int64_t d_out, d_in;
  int32_t d_block;     /* divides d_out and d_in; multiple of m_group; at most 256 */
  int32_t n_keep;      /* N of N:M: 2 (with m_group 4) or 4, 5, 6 (with m_group 8; Section 4.4) */
  int32_t m_group;     /* M of N:M: 4 or 8 */
  int32_t h_mode;      /* ARMOR_H_* */
  int32_t select_mode; /* ARMOR_SELECT_* (Section 3.3.2 / Appendix E.1) */
  int32_t s_step;      /* ARMOR_S_EXACT: exact line search along Gamma (.) M; ARMOR_S_BETA: the paper's
                          step 1/beta_W' (Eq. lrWprime) */
  int32_t precision;   /* ARMOR_PREC_* */
  int32_t normalize;   /* 1: armor_init applies the NoWag normalisation */
  int32_t phases;      /* bitmask of ARMOR_PHASE_*; 0 means all four */
  int32_t ab_step;     /* ARMOR_AB_* */
  int32_t mask_sweeps; /* sparse-core updates (Algorithm 3) per iteration, each from the state the previous one
                          left, run k of iteration t drawing its groups with the counter t*K + k; 0 means 1,
                          the paper's alternation; at most 64 */
  int32_t mask_groups; /* groups drawn per block in one sparse-core update: the k smallest race keys, each solved on
                          its own, all kept or dropped together by the exact joint change of the loss (either
                          weighting); 0 means 1, the paper's single group; at most 8 */
  float ridge;         /* relative proximal ridge of the block solves (1e-6) */
  float adam_lr;       /* ARMOR_AB_ADAM: step size (0: 1e-4, Appendix F of the paper) */
  float adam_beta1;    /* moment decay rates and epsilon (0: 0.9, 0.999, 1e-8, the defaults of the Adam paper) */
  float adam_beta2;
  float adam_eps;
  uint64_t seed;       /* seed of the counter-based group selection */
} armor_config;

/* One record per BCD iteration, written on the device.  The losses after the
 * sub-steps follow from loss_start by the exact decrease of each quadratic
 * step.  loss_start is evaluated from the residual in the first iteration of a
 * call and every 64 iterations after it (and in every iteration with
 * ARMOR_AB_ADAM); in between it is the previous iteration's loss_mask. */
typedef struct {
  double loss_start, loss_A, loss_B, loss_S, loss_mask;
  double delta_L_mask;   /* exact loss change of the iteration's group updates (summed over the sweeps) */
  float tau_B, tau_S;    /* exact step lengths of the B-step and S-step */
  int32_t groups_changed;/* groups whose mask changed, summed over the sweeps (rejected sweeps count 0) */
  int32_t mask_accepted; /* sweeps whose group updates were kept (0 or 1 with one sweep) */
  int32_t chol_failed;   /* blocks skipped because a Cholesky pivot was <= 0 */
  int32_t reserved;
} armor_iter_stats;

/* Scratch size for a configuration.  Error: INVALID_ARG (null), SHAPE
 * (d_block does not divide the dims, m_group does not divide d_block),
 * UNSUPPORTED (N:M other than 2:4, 4:8, 5:8, 6:8; d_block > 256, not a multiple of 4, or above 128 and not a
 * multiple of 32; tensor-core precisions with full weighting need d_out and d_in multiples of 128). */
armor_status armor_workspace_bytes(const armor_config* cfg, size_t* bytes);

/* Creates a context over caller-owned device scratch (256-byte aligned, at
 * least armor_workspace_bytes).  The context holds the configuration and the
 * carve-up of the workspace only, plus two non-blocking streams and a few events of its own (graph capture of the
 * iterations, staging of the Gram).  Must be called with the device current. */
armor_status armor_create(armor_ctx** ctx, const armor_config* cfg, void* d_workspace, size_t bytes);
armor_status armor_destroy(armor_ctx* ctx);

/* Calibration Gram (Section 2 / Eq. proxy_loss: its diagonal is ||X_j||^2).
 * d_H [d_in, d_in] fp32 += X^T X for a chunk X [n_rows, d_in] with leading
 * dimension ldx (elements).  The caller zeroes d_H before the first chunk.
 * x_dtype: ARMOR_DTYPE_F32 or ARMOR_DTYPE_BF16 (bf16 values are exact tensor-core
 * operands, so their Gram needs one pass in every tensor-core precision; not
 * available with ARMOR_PREC_SIMT).  n_rows == 0 is a no-op.  A chunk is worked through in pieces of 16,384 rows
 * (transposed, scaled and split into a staging buffer, then contracted); with ARMOR_PREC_FP16X3 a call of several
 * pieces stages piece p + 1 on a stream of the context's own while piece p is contracted on `stream` (the result does
 * not depend on it; the call returns with all of its work ordered before later work on `stream`, as always). */
armor_status armor_gram(armor_ctx* ctx, const void* d_X, int32_t x_dtype, int64_t n_rows, int64_t ldx,
                        float* d_H, armor_stream_t stream);

/* Normalisation and initialisation (Section 3.2 display after Eq. proxy_loss;
 * Eq. init): optionally W_bar = W / r1 / r2 (zero norms read as 1), then
 * A = B = I, M = top-n_keep of every group by W_bar^2 * H_jj (ties keep the
 * lower column), S = W_bar (.) M.  d_Wbar receives the matrix the later calls
 * take as W (a copy of d_W when cfg.normalize == 0; may alias d_W).  d_r1
 * [d_in], d_r2 [d_out] are written only when cfg.normalize == 1 (else may be
 * NULL). */
armor_status armor_init(armor_ctx* ctx, const float* d_W, const float* d_H, float* d_Wbar, float* d_r1,
                        float* d_r2, float* d_A, float* d_B, float* d_S, uint8_t* d_M,
                        armor_stream_t stream);

/* n_iters iterations of Algorithm 1's loop, numbered t_first .. t_first +
 * n_iters - 1: A-step, B-step, S-step (the continuous update of Algorithm 2,
 * with exact block solves / exact line searches in place of the 1/beta
 * gradient steps) and the greedy sparse-core update of Algorithm 3 (one group
 * per block, closed-form solve over all masks, Eq. mask_loss_opt and
 * mask_loss_opt_sol).  A, B, S, M are updated in place.  d_stats may be NULL,
 * else [n_iters].  The iterations of a call are a function of (state, W, H,
 * t_first, n_iters); runs are reproducible bit for bit.  With h_mode DIAG every
 * iteration depends on the state alone, so splitting a run into several calls
 * gives the same bits in A, B, S and M; with h_mode FULL the product S B H is
 * carried from iteration to iteration inside a call and rebuilt by a dense
 * product at its start, so a split changes the rounding (fp32 accuracy). */
armor_status armor_bcd_step(armor_ctx* ctx, const float* d_Wbar, const float* d_H, float* d_A, float* d_B,
                            float* d_S, uint8_t* d_M, int64_t t_first, int32_t n_iters,
                            armor_iter_stats* d_stats, armor_stream_t stream);

/* Proxy loss L = tr(E H_w E^T), E = W - A S B (Eq. proxy_loss; full-Gram form
 * when h_mode == FULL), written to *d_loss (device, double). */
armor_status armor_proxy_loss(armor_ctx* ctx, const float* d_Wbar, const float* d_H, const float* d_A,
                              const float* d_B, const float* d_S, double* d_loss, armor_stream_t stream);

/* Deployment form (Section 3.1): y_t = A (S (B x_t)) for the rows of
 * x [n_tokens, d_in] -> y [n_tokens, d_out].  With d_r1, d_r2 non-NULL the
 * normalisation is undone: y_t = r2 (.) A S B (r1 (.) x_t).  xy_dtype:
 * ARMOR_DTYPE_F32, or ARMOR_DTYPE_BF16 for bf16 x and y: the deployment form, in
 * which the core S and the wrapped activations B x are rounded to bf16 and
 * multiplied on the bf16 tensor-core path with fp32 accumulation (the two thin
 * wrapper products stay fp32-grade; y is rounded to bf16 once).
 * ARMOR_DTYPE_BF16_SPARSE: the same bf16 x and y, with the core on the sparse
 * tensor cores (the 2:4 speed-up the paper's inference measurements rely on,
 * Section 4.3): S is packed to its kept values (bf16) and 2-bit positions taken
 * from d_M on every call; needs the 2:4 pattern, d_M non-NULL and d_out, d_in
 * multiples of 128, else UNSUPPORTED / INVALID_ARG.  A group of d_M with more
 * than two kept positions is counted in device status word 4 and contributes
 * its first two.  With the other two dtypes d_M may be NULL (S already carries
 * the zeros). */
armor_status armor_apply(armor_ctx* ctx, const float* d_A, const float* d_B, const float* d_S,
                         const uint8_t* d_M, const float* d_r1, const float* d_r2, const void* d_x,
                         void* d_y, int32_t xy_dtype, int64_t n_tokens, armor_stream_t stream);

/* The deployment form with the core packed once (Section 3.1; the paper's inference measurements, Section 4.3,
 * use a 2:4 core in the hardware's compressed format).  armor_packed_core_bytes: size of the packed core,
 * d_out*d_in bytes of kept values (bf16, two of every four, in order) followed by d_out*d_in/8 bytes of 2-bit
 * positions in the order the sparse tensor cores read them (needs 2:4 and d_out, d_in multiples of 128, else
 * UNSUPPORTED).  armor_pack_core: packs S with the kept positions of d_M into d_packed (device, caller-owned,
 * 128-byte aligned); a group of d_M with more than two kept positions is counted in device status word 4.
 * armor_apply_packed: y = A S B x for bf16 x [n_tokens, d_in] -> bf16 y [n_tokens, d_out] with the packed
 * core on the sparse tensor cores (fp32 accumulation; the wrapper products as in armor_apply; d_r1, d_r2 as
 * there).  Equal to armor_apply with ARMOR_DTYPE_BF16_SPARSE, which packs on every call. */
armor_status armor_packed_core_bytes(const armor_config* cfg, size_t* out_bytes);
armor_status armor_pack_core(armor_ctx* ctx, const float* d_S, const uint8_t* d_M, void* d_packed,
                             armor_stream_t stream);
armor_status armor_apply_packed(armor_ctx* ctx, const float* d_A, const float* d_B, const void* d_packed,
                                const float* d_r1, const float* d_r2, const void* d_x, void* d_y,
                                int64_t n_tokens, armor_stream_t stream);

/* The whole layer packed for a bf16 forward that touches no fp32 intermediate (Section 3.1 and the last
 * paragraph of Section 3.2: the normalisation's scales are folded into the wrappers).  The packed layer is the
 * packed core of armor_pack_core followed by the blocks of B with their columns scaled by r1 and the blocks of A
 * with their rows scaled by r2, both rounded to bf16 (d_r1 and d_r2 both NULL: no scales).
 * armor_packed_layer_bytes gives its size (needs 2:4, d_out and d_in multiples of 128, d_block 128 or 256, else
 * UNSUPPORTED); d_packed is caller-owned device memory, 128-byte aligned.
 * armor_apply_layer: bf16 x [n_tokens, d_in] -> bf16 y [n_tokens, d_out] (both 16-byte aligned), three kernels
 * per chunk of tokens: z1 = (r1 . x) B^T and y = r2 . (z2 A^T) as batched bf16 tensor-core products over the
 * blocks, z2 = z1 S^T on the sparse tensor cores; fp32 accumulation, z1 and z2 rounded to bf16 in the
 * context's workspace. */
armor_status armor_packed_layer_bytes(const armor_config* cfg, size_t* out_bytes);
armor_status armor_pack_layer(armor_ctx* ctx, const float* d_A, const float* d_B, const float* d_S, const uint8_t* d_M,
                              const float* d_r1, const float* d_r2, void* d_packed, armor_stream_t stream);
armor_status armor_apply_layer(armor_ctx* ctx, const void* d_packed, const void* d_x, void* d_y, int64_t n_tokens,
                               armor_stream_t stream);

/* Copies up to n (at most 16) device status words to h_codes (host).
 *   word 0: Cholesky failures since the context was created; word 1: first failing block id + 1;
 *   word 2: bounded waits that gave up; word 3: last armor_status recorded by a kernel;
 *   word 4: mask groups the sparse forward could not represent;
 *   words 5-9, written by the input screening that armor_init and armor_bcd_step run first:
 *     5: NaN / Inf entries seen in W, 6: NaN / Inf entries seen in H, 7: negative diagonal entries of H
 *     (all three cumulative), 8: zero diagonal entries of H in the last screened call (legal: a channel
 *     without weight), 9: 1 if the last screened call met any of 5-7.  Such a call withholds every update:
 *     A, B, S and M come back bit for bit as they went in (armor_init still writes its outputs), word 3 reads
 *     ARMOR_ERR_INVALID_ARG, and the next call with clean inputs runs normally.
 *   word 10 (ARMOR_PREC_FP16X3): entries of H that, after the scaling by its diagonal, lie beyond the fp16 range and
 *     were clamped (cumulative).  A positive semidefinite H has none; a non-zero count means the products with H
 *     were not those of the H that was passed.
 * The caller must have synchronised the stream the context's work ran on.  (This call itself copies
 * synchronously.) */
armor_status armor_get_device_status(armor_ctx* ctx, int32_t* h_codes, int32_t n);

const char* armor_status_string(armor_status s);

/* Self-test of the bounded waits (no counterpart in the paper): every wait of the tensor-core kernels on an
 * mbarrier gives up after a cycle budget, raises status word 2, records ARMOR_ERR_TIMEOUT in word 3 and lets the
 * kernel end normally.  This call runs one warp that waits, with a limit of limit_cycles (1 .. 2e9) clock
 * cycles, on a barrier nothing arrives on, and writes d_result[0] = 0 (the wait gave up; 1 would mean it was
 * satisfied) and d_result[1] = 1 (the abort flag the other roles of a kernel watch).  d_result: two int32 on
 * the device.  The context stays usable. */
armor_status armor_selftest_wait_timeout(armor_ctx* ctx, int64_t limit_cycles, int32_t* d_result,
                                         armor_stream_t stream);

/* Number of kernel launches the context has enqueued so far (host counter). */
int64_t armor_launch_count(const armor_ctx* ctx);

/* Measurement aid for the tensor-core GEMM that carries the Gram and the dense
 * .H contractions (the dominant kernel of the FULL mode).  While enabled, every
 * launch of that kernel is bracketed by CUDA events on its stream (up to 4096
 * launches are kept, later ones are not timed).  armor_gemm_timing synchronises
 * on the recorded events and returns the number of timed launches, their total
 * duration in milliseconds and their algorithmic flops (2*M*N*K per launch;
 * M*N*K + M*128*K for the symmetric Gram launches), then clears the record.
 * Events are created on first use; no device memory is allocated. */
armor_status armor_gemm_timing_enable(armor_ctx* ctx, int32_t enable);
armor_status armor_gemm_timing(armor_ctx* ctx, int64_t* n_launches, double* total_ms, double* total_flops);

/* The same measurement aid for every kernel class (no counterpart in the paper).  Level 0: off; 1: the dense
 * tensor-core products only (what armor_gemm_timing_enable(ctx, 1) sets); 2: every launch of the context is
 * bracketed by a pair of events on its stream (at most 8192 launches are recorded between two reads; the pairs
 * cost about a microsecond each, so time a step as a whole with level 0 or 1).
 * armor_kernel_timing waits for the recorded events and returns, for the classes 0 .. n_classes - 1, the number
 * of launches, their summed device time in ms and their summed algorithmic work: flops for ARMOR_KC_GEMM
 * (single-pass, 2 M N K; M (N + 128) K for the lower-triangle Gram) and ARMOR_KC_CHOLESKY, bytes that must cross
 * HBM for all others (0 for classes of small kernels).  It clears the record. */
enum {
  ARMOR_KC_GEMM = 0,           /* dense tensor-core products: Gram, .H, the forward's core */
  ARMOR_KC_BLOCK_PRODUCT = 1,  /* products of a W-shaped matrix with the block-diagonal wrappers: 8 B / element, 12 with an addend */
  ARMOR_KC_BLOCK_GRAM = 2,     /* per-block Gram matrices over d_in or d_out: two W-shaped operands read */
  ARMOR_KC_CHOLESKY = 3,       /* per-block factorisation and two triangular solves: (7/3) d_block^3 flops per block */
  ARMOR_KC_AXPY = 4,           /* y += a x on W-shaped arrays (12 B / element), column scale, Adam update */
  ARMOR_KC_DOT = 5,            /* dot products of W-shaped arrays: 8 B / element */
  ARMOR_KC_MASKED_COPY = 6,    /* Gamma (.) M with its squared norm */
  ARMOR_KC_MASK_SELECT = 7,    /* scoring, selection and mask sweep: one read of Gamma, 4 B / element */
  ARMOR_KC_MASK_GUARD = 8,     /* the other kernels of the sparse-core update (vectors, thin product with H, commit, carry) */
  ARMOR_KC_OPERAND_SPLIT = 9,  /* high / low parts of a dense product's operands: 8 B / element */
  ARMOR_KC_GRAM_STAGING = 10,  /* channel maxima, transposition and split of a chunk of activations */
  ARMOR_KC_INIT = 11,          /* normalisation, initial masks and core, input screening */
  ARMOR_KC_SMALL = 12,         /* reductions, bookkeeping, small block products */
  ARMOR_KC_FORWARD = 13,       /* conversions, packing and wrapper products of the deployment form */
  ARMOR_KC_COUNT = 14
};
armor_status armor_kernel_timing_enable(armor_ctx* ctx, int32_t level);

/* armor_bcd_step replays the iterations of a call that enqueue identical launches (all but the first, and the
 * every-64th that re-evaluates the loss) from a CUDA graph, captured once per call on a stream of the context's
 * own and launched on the caller's stream; which iteration runs reaches the kernels through a device counter.
 * On by default; it is skipped when the caller's stream is itself being captured, when every launch is being timed
 * (armor_kernel_timing_enable level 2), for calls of fewer than four iterations, and after any failure to capture
 * (the call then continues with direct launches).  While only the dense products are timed (level 1), the iteration
 * is captured in pieces that end at each dense product with H; the replay alternates the pieces with those products,
 * launched directly between their events.  Results are identical in every case.  enable = 0 switches it off for the context.  (No counterpart
 * in the paper.) */
armor_status armor_use_graphs(armor_ctx* ctx, int32_t enable);
/* The A-step needs G_i = P_i T_i^T and Gamma_i = (E H_w)_i T_i^T, the B-step C_j = U_j^T U_j and Gamma_j = U_j^T (E H_w)_j
 * (Section 3.2): per step the two per-block Grams share an operand.  On the tensor cores they run as ONE launch that
 * reads every shared chunk once (on by default; the column-block pair needs d_block = 128); enable = 0 runs them as
 * two launches.  Same MMAs per accumulator in the same order: the results are identical.  For tests and measurements. */
armor_status armor_fuse_grams(armor_ctx* ctx, int32_t enable);
armor_status armor_kernel_timing(armor_ctx* ctx, int32_t n_classes, int64_t* launches, double* total_ms,
                                 double* total_work);

/* One product with a block-diagonal wrapper (Section 3.1: A and B are applied as batched d_block x d_block
 * products), exposed for tests and measurements; armor_bcd_step and armor_apply are built from it.
 *   side 0: d_out[:, j-th block] = alpha * d_in[:, j-th block] * Q_j (+ beta * d_add[:, j-th block])
 *   side 1: d_out[i-th block, :] = alpha * Q_i * d_in[i-th block, :] (+ beta * d_add[i-th block, :])
 * with Q = d_blocks [n_blocks, d_block, d_block] or, if transpose != 0, its blocks transposed.  d_in, d_out,
 * d_add (may be NULL; may equal d_out) are [rows, cols] fp32; d_in must not overlap d_out.  path 0: fp32
 * CUDA-core kernel; path 1: tensor-core kernel (tcgen05, operands split in shared memory into tf32 high and
 * low parts, three passes; needs d_block a multiple of 128 and a tensor-core precision, else UNSUPPORTED);
 * path 2: the same arithmetic with the wrapper block held in tensor memory as the M-side operand and two tiles per
 * instruction (d_block = 128 only, else UNSUPPORTED; same bits as path 1);
 * any other value: what the library itself would use (path 1 where it applies).  Errors: INVALID_ARG, SHAPE (the blocked dimension is
 * not a multiple of d_block, or cols is not a multiple of 4). */
armor_status armor_block_product(armor_ctx* ctx, int32_t side, int32_t transpose, const float* d_blocks,
                                 const float* d_in, float* d_out, int64_t rows, int64_t cols, float alpha,
                                 const float* d_add, float beta, int32_t path, armor_stream_t stream);

/* A product with both wrappers (Section 3.1; the gradient of the core, Gamma = A^T (E H_w) B^T, is one):
 *   d_out[i-th block row, j-th block column] = alpha * Lop_i * d_in[i, j] * Rop_j,
 * Lop_i = d_left[i] or, if transpose_left != 0, its transpose; Rop_j likewise from d_right.  d_left is
 * [d_out / d_block, d_block, d_block], d_right [d_in / d_block, d_block, d_block], d_in and d_out [d_out, d_in] of the
 * context (device fp32, distinct).  path 3: one fused tensor-core launch in which Lop_i d_in[i, j] stays in tensor
 * memory (d_block = 128 and a tensor-core precision, else UNSUPPORTED); paths 0, 1, 2: the two one-sided products
 * on the kernel armor_block_product names; any other value: what the library itself uses (path 3 where it applies).
 * Paths 1, 2 and 3 give the same bits.  Exposed for tests and measurements. */
armor_status armor_block_product_two_sided(armor_ctx* ctx, const float* d_left, int32_t transpose_left, const float* d_in,
                                           const float* d_right, int32_t transpose_right, float* d_out, float alpha,
                                           int32_t path, armor_stream_t stream);

/* The pair of products behind the step length of a line search (Section 3.2: the exact step along a direction
 * V needs tr(V H_w V^T) = <V H_w, V> with V = A R and V H_w = A (R H_w)):
 *   d_out = Q d_in2 per block row (side 1 above, alpha 1, no addend) and *d_dot = <Q d_in1, Q d_in2>,
 * Q = d_blocks [d_out / d_block, d_block, d_block]; d_in1, d_in2, d_out are [d_out, d_in] of the context (device
 * fp32, d_out distinct from both inputs), d_dot one device double.  path 1: one fused tensor-core launch in which
 * Q d_in1 only exists as an accumulator (needs d_block a multiple of 128 and a tensor-core precision, else
 * UNSUPPORTED); path 2: the same with Q in tensor memory and both inputs of a tile in one instruction (d_block = 128
 * only); path 0: two CUDA-core products and a dot product; any other value: what the library itself uses (path 2
 * where it applies, else path 1).
 * The sum is formed in a fixed order (deterministic).  Exposed for tests and measurements. */
armor_status armor_block_product_dual(armor_ctx* ctx, const float* d_blocks, const float* d_in1, const float* d_in2,
                                      float* d_out, double* d_dot, int32_t path, armor_stream_t stream);

/* The paper has no counterpart to this entry point; it exists for deployment reasons only.
 *
 * armor_normalize_noalloc computes the same row/column normalisation that armor_init applies when
 * cfg.normalize == 1 (W_bar = W / r1 / r2, r1 = column norms of W, r2 = row norms of W / r1, zero
 * norms read as 1), but needs neither a context nor a workspace.  It is meant for callers that are
 * not allowed to obtain device memory at the point where they need the result: a process whose
 * whole device memory has already been handed to another allocator or to a fixed serving pool, a
 * plugin running inside a host application that forbids device allocations after start-up, or a
 * latency-critical loop that cannot afford the device-wide synchronisation an allocation implies.
 * The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Its scratch (ARMOR_NOALLOC_ROW_CHUNKS x ARMOR_NOALLOC_MAX_COLS doubles = 4 MiB) is a fixed array
 * inside the library's device image: every GPU that loads the library holds those 4 MiB until the
 * process exits.  Limits: d_in <= ARMOR_NOALLOC_MAX_COLS and d_out <= ARMOR_NOALLOC_MAX_ROWS, else
 * ARMOR_ERR_TOO_LARGE.  Inputs and outputs are the caller's device buffers: d_W and d_Wbar
 * [d_out, d_in] (distinct buffers), d_r1 [d_in], d_r2 [d_out].
 *
 * The first call on each device looks up the device address of the built-in array (with that
 * device current); make that first call outside any stream capture.  All calls on a device share
 * the array and it keeps the previous call's contents; nothing in it has to start at zero because
 * every slot is written before it is read within a call.  Two calls that overlap on the same GPU
 * (different streams, or different host threads) race on the array: serialise them. */
#define ARMOR_NOALLOC_MAX_COLS 8192
#define ARMOR_NOALLOC_MAX_ROWS 65536
#define ARMOR_NOALLOC_ROW_CHUNKS 64
armor_status armor_normalize_noalloc(const float* d_W, int64_t d_out, int64_t d_in, float* d_Wbar,
                                     float* d_r1, float* d_r2, armor_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* ARMOR_H */
