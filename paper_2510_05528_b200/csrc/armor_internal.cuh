// Internal declarations shared by the translation units of libarmor.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "armor.h"

// ---------------------------------------------------------------- scalars
// Device-resident double scalars (one set per context).  Kernels read step
// lengths and accept flags from here so that no sub-step needs the host.
enum {
  SC_L0 = 0,     // <E H_w, E> at the start of the iteration
  SC_DEC_A,      // exact decrease of the A-step
  SC_GD_B,       // <Gamma^B, Delta>
  SC_Q_B,        // tr(V H_w V^T) of the B direction
  SC_NRM_S,      // ||Gamma (.) M||_F^2
  SC_Q_S,        // tr(V H_w V^T) of the S direction
  SC_EHV_M,      // <E H_w, V> of the group updates
  SC_Q_M,        // tr(V H_w V^T) of the group updates
  SC_TAU_B,
  SC_TAU_S,
  SC_ACCEPT,     // 1.0 if the group updates are kept
  SC_DL_M,       // exact loss change of the group updates
  SC_LOSS,       // running loss inside an iteration
  SC_BETA_A,     // ||A^T A||_F^2 (BETA step)
  SC_BETA_K,     // ||B H_w B^T||_F^2 (BETA step)
  SC_TMP0,
  SC_TMP1,
  SC_TAU_A,      // step of the A gradient step (ab_step GD)
  SC_HB_A,       // beta_A / 2 of Eq. lrA
  SC_HB_B,       // beta_B / 2 of Eq. lrB
  SC_COUNT = 32
};

// status words in the device status buffer
enum {
  ST_CHOL_FAILS = 0, ST_FIRST_FAIL = 1, ST_WAIT_TIMEOUTS = 2, ST_LAST_ERR = 3, ST_SPARSE_BAD_GROUPS = 4,
  ST_NONFINITE_W = 5,    // NaN / Inf entries seen in W by the input screening (cumulative)
  ST_NONFINITE_H = 6,    // NaN / Inf entries seen in H
  ST_NEG_DIAG_H = 7,     // negative diagonal entries of H (H cannot be a Gram matrix)
  ST_DEAD_CHANNELS = 8,  // zero diagonal entries of H in the last screened call (legal: the channel carries no weight)
  ST_POISON = 9,         // 1 while the last screened call had unusable inputs: its updates were all withheld
  ST_H_RANGE = 10,       // entries of the scaled H beyond the fp16 range (FP16X3; H not positive semidefinite): clamped
  ST_COUNT = 16
};

static const int ARMOR_MAX_PIECES = 16;   // graph pieces of one iteration when it is captured around its dense products

// One selected group per (i, j) block of the sparse core (Algorithm 3).
struct SelRec {
  int32_t valid;      // 0: nothing selected in this block
  int32_t row;        // global row r
  int32_t cgrp;       // group index inside the row (columns m*cgrp ..)
  int32_t new_mask;   // bit p <=> position p kept
  int32_t old_mask;
  float new_val[8];
  float old_val[8];
};

static const int ARMOR_DOT_BLOCKS = 592;  // 4 x 148 partial sums per reduction

struct armor_ctx {
  armor_config cfg;
  int64_t d_out, d_in, wn;  // wn = d_out * d_in
  int db, nbo, nbi;
  char* ws;
  size_t ws_bytes;
  // W-shaped fp32 scratch
  float *T, *E, *EH, *P, *U, *V, *VH, *Gam, *Tmp, *WH;
  // low parts of the left operands / of H for the three-pass tensor-core mode
  float *Lo, *Hlo;
  // [nb, db, db] scratch
  float *G, *GamA, *dA, *C, *GamB, *Delta, *Hjj, *Kfull, *Ktmp;
  float* Hinv;           // (H_jj + mu I)^-1 per column block, formed once per armor_bcd_step call
  int32_t* hinv_fail;    // [nbi] 1 where that block was not positive definite
  float *alpha, *hdiag;
  float *mA, *vA, *mB, *vB, *mS, *vS;   // Adam moment estimates (ab_step ADAM)
  float *Hq1, *Hq2;      // [d_in, d_in] scratch of the paper's step size (s_step BETA, full weighting)
  float* gemm_slabs;     // 128 x 256 slabs of partial sums of the dense product's split tail tiles
  int64_t gemm_slab_count;
  float* gpart;          // partial products of split contractions
  int64_t gpart_floats;
  // sparse-core update: per selected group z = delta^T B_j[rows of the group, :] and a = A_i[:, r]
  float *Zsel, *Acol, *Ysel;  // [nbi][nbo_pad][db], [nbo][nbi][db], [nbi][nbo_pad][d_in]
  int nbo_pad;                // nbo rounded up to a multiple of 32
  // three-pass fp16 mode: column scales derived from diag(H), per-row output scales of the two operands,
  // per-channel maxima and output scales of a Gram chunk
  float *hpow, *rowscale, *rowscale2, *gscale;
  float* gscale2;       // output scales of the chunk staged in Xt_hi2
  unsigned* gmax;
  // Gram staging (transposed, split chunk of X)
  float *Xt_hi, *Xt_lo;
  float* Xt_hi2;        // second staging buffer (FP16X3): chunk p + 1 is staged on side_stream while chunk p is contracted
  cudaStream_t side_stream;
  cudaEvent_t ev_fork, ev_staged[2], ev_used[2];
  int64_t gram_rows;  // rows of X staged per pass
  double* sc;         // [SC_COUNT]
  double* partials;   // [2][8 * npart] partial sums of the fused / streaming reductions
  int64_t npart;
  double* partblk;    // [max(4 * nbo, 4 * nbi, nbo * nbi)] per-block partial sums
  double* quadpart;   // [nbo * nbi] per-block terms of the group updates' quadratic form
  double* colpart;    // [64][d_in] column partial sums of the normalisation
  int32_t* failflag;  // [max(nbo, nbi)]
  SelRec* sel;        // [nbo * nbi]
  float* tab_key;     // [nbo * nbi] winning race key of every block (single draw)
  unsigned long long* tab_g;   // its global group index
  int32_t* status;    // [ST_COUNT]
  int32_t* screen;    // [4] per-call counters of the input screening
  int64_t* it_dev;    // iteration index inside the running armor_bcd_step call (advanced by the last kernel of an iteration)
  int use_graphs;     // 1: repeated iterations of a call are replayed from a CUDA graph
  cudaStream_t cap_stream;   // the context's own stream, used only to capture that graph
  // Capture in pieces (while the dense products are being timed with events, which a graph cannot replay): every
  // dense product with H closes the piece being captured, is remembered with its arguments and opens the next
  // piece; the replay alternates graph pieces and directly launched products.
  int cap_split;             // 1 while such a capture runs
  int cap_n;                 // pieces closed so far (= products remembered)
  int cap_failed;            // too many pieces or a failed capture call: the iteration is enqueued directly instead
  cudaGraph_t cap_graph[ARMOR_MAX_PIECES];
  struct RmulCall { const float* in; const float* H; float* out; int64_t rows; const float* d1; double* out1;
                    const float* d2; double* out2; } cap_call[ARMOR_MAX_PIECES];
  int64_t launches;
  int device;           // the device that was current at armor_create; every call must be issued with it current
  int n_sm;             // its number of SMs
  int tc_blocks;        // 1, 2, 3: block products and per-block Grams on the tensor cores where the shape allows.
                        // 1: the streaming kernel for every product; 2: with d_block = 128 the kernel that keeps the
                        // wrapper block in tensor memory for every product; 3 (default): that kernel for the dual
                        // product, where it halves the shared-memory traffic, and the streaming kernel elsewhere
                        // (the two measure equal on single products at 4096 x 4096);
                        // 0: always the fp32 CUDA-core kernels (exact products with 0 and 1)
  int gram_pairs;       // 1: the two per-block Grams of a step in one launch (shared operand read once)
  armor_status host_err;   // first launch failure inside the running call that no fallback covers
  int kg;               // groups drawn per block in one sparse-core update (mask_groups, at least 1)
  int block_one_pass;   // 1: products with the wrappers take one tf32 pass (the bf16 forward, whose operands are
                        // rounded to 8 bits anyway); 0: three passes, fp32-grade
  // identity of the H whose low part is cached in Hlo
  const float* h_cached;
  // optional event timing of the launches: 0 off, 1 the dense tensor-core products only, 2 every kernel class
  int timing_on;
  int timing_n;              // launches recorded
  cudaEvent_t* ev_beg;       // [ARMOR_MAX_TIMED]
  cudaEvent_t* ev_end;
  int32_t* ev_cls;           // kernel class of the recorded launch (ARMOR_KC_*)
  double* ev_work;           // its algorithmic work: flops (dense products, Cholesky) or bytes (everything else)
  int ev_created;
};
static const int ARMOR_MAX_TIMED = 8192;

// Brackets the launches made during its lifetime with a pair of events on the launching stream when timing is on.
struct KTimer {
  armor_ctx* c; cudaStream_t s; int slot;
  KTimer(armor_ctx* c_, int cls, double work, cudaStream_t s_) : c(c_), s(s_), slot(-1) {
    if (!c->timing_on || (c->timing_on == 1 && cls != ARMOR_KC_GEMM) || c->timing_n >= c->ev_created) return;
    slot = c->timing_n++;
    c->ev_cls[slot] = cls;
    c->ev_work[slot] = work;
    cudaEventRecord(c->ev_beg[slot], s);
  }
  ~KTimer() { if (slot >= 0) cudaEventRecord(c->ev_end[slot], s); }
  KTimer(const KTimer&) = delete;
  KTimer& operator=(const KTimer&) = delete;
};

#define ARMOR_CUDA_OK(expr)                                  \
  do {                                                       \
    cudaError_t _e = (expr);                                 \
    if (_e != cudaSuccess) return ARMOR_ERR_CUDA;            \
  } while (0)

// ---------------------------------------------------------------- launchers
// Generic strided batched fp32 GEMM on CUDA cores:
//   C_b[m][n] = alpha * sum_k A_b[m][k] B_b[k][n] + beta * D_b[m][n]
// element (m,k) of A_b lives at A + b*sAb + m*sAm + k*sAk (likewise B, C, D).
struct BGemm {
  const float* A; int64_t sAb, sAm, sAk;
  const float* B; int64_t sBb, sBk, sBn;
  float* C; int64_t sCb, sCm, sCn;
  const float* D; int64_t sDb, sDm, sDn;
  int M, N, K, batch;
  float alpha, beta;
  // two-level batch: batch index b = bo * batch_inner + bi, operand offset bo * s?b2 + bi * s?b
  // (batch_inner == 0: one level)
  int batch_inner;
  int64_t sAb2, sBb2, sCb2, sDb2;
  // split of the contraction into ksplit equal chunks whose partial products are summed in a fixed order
  // (needs c->gpart; only without D)
  int ksplit;
};
void launch_bgemm(armor_ctx* c, const BGemm& g, cudaStream_t s);
// number of chunks a long contraction is cut into so that batch * tiles * chunks fills the GPU about twice
inline int pick_ksplit(int64_t batch, int64_t tiles, int64_t K) {
  int64_t ks = (296 + batch * tiles - 1) / (batch * tiles);
  if (ks > K / 256) ks = K / 256;
  while (ks > 1 && K % (16 * ks)) --ks;
  return ks < 1 ? 1 : (int)ks;
}

// block-diagonal products on row-major [rows, cols] matrices
//  right: out[:, jblk] = alpha * in[:, jblk] * Bblk[j] (+ beta * add[:, jblk]); transB uses Bblk[j]^T
//  left : out[iblk, :] = alpha * Ablk[i] * in[iblk, :] (+ beta * add[iblk, :]); transA uses Ablk[i]^T
void bd_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
              int64_t cols, float alpha, const float* add, float beta, cudaStream_t s);
void bd_left(armor_ctx* c, const float* Ablk, bool transA, const float* in, float* out, int64_t rows,
             int64_t cols, float alpha, const float* add, float beta, cudaStream_t s);
// out = alpha * Lop X Rop with both wrappers (Lop_i = Lblk[i] or its transpose, Rop_j likewise): one fused launch on
// the tensor cores where the shape allows (d_block 128; the intermediate stays in tensor memory), else the two
// one-sided products through tmp
void bd_two_sided(armor_ctx* c, const float* Lblk, bool transL, const float* X, const float* Rblk, bool transR, float* tmp,
                  float* out, int64_t rows, int64_t cols, float alpha, cudaStream_t s);
// out = Ablk in2 and partial sums of <Ablk in1, Ablk in2> at part, *n_part of them (the consumer adds them up): one
// fused launch on the tensor cores (Ablk in1 never reaches memory), else two products (the first into tmp) and a dot
void bd_left_dual(armor_ctx* c, const float* Ablk, const float* in1, const float* in2, float* tmp, float* out,
                  int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s);

// the same two products on the tensor cores (block_tcgen05.cu); d_block must be a multiple of 128
bool tc_block_ok(const armor_ctx* c, int64_t rows, int64_t cols);
armor_status tc_bd_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
                         int64_t cols, float alpha, const float* add, float beta, cudaStream_t s);
armor_status tc_bd_left(armor_ctx* c, const float* Ablk, bool transA, const float* in, float* out, int64_t rows,
                        int64_t cols, float alpha, const float* add, float beta, cudaStream_t s);

// out = P in2 per block row, with the partial sums of <P in1, P in2> (four per 128 x 128 tile) at part
armor_status tc_bd_left_dual(armor_ctx* c, const float* Ablk, bool transA, const float* in1, const float* in2, float* out,
                             int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s);

// both wrappers in one launch (block2_tcgen05.cu); d_block = 128
bool tc_block2_ok(const armor_ctx* c, int64_t rows, int64_t cols);
armor_status tc_two_sided(armor_ctx* c, const float* Lblk, bool transL, const float* X, const float* Rblk, bool transR,
                          float* out, int64_t rows, int64_t cols, float alpha, cudaStream_t s);

// E = add - Ablk in, EH = E diag(colw), partial sums of <E, EH> at part: one launch
armor_status tc_bd_left_residual(armor_ctx* c, const float* Ablk, const float* in, const float* add, const float* colw,
                                 float* E, float* EH, int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s);

// the same with the wrapper block held in tensor memory (blockres_tcgen05.cu); d_block = 128
bool tc_blockres_ok(const armor_ctx* c);
armor_status tc_blockres_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
                               int64_t cols, float alpha, const float* add, float beta, cudaStream_t s);
armor_status tc_blockres_left(armor_ctx* c, const float* Ablk, bool transA, const float* in, float* out, int64_t rows,
                              int64_t cols, float alpha, const float* add, float beta, cudaStream_t s);

armor_status tc_blockres_left_dual(armor_ctx* c, const float* Ablk, const float* in1, const float* in2, float* out,
                                   int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s);

// per-block Grams over a long contraction on the tensor cores
bool tc_gram_ok(const armor_ctx* c);
armor_status tc_rowblock_gram(armor_ctx* c, const float* P, const float* T, float* G, cudaStream_t s);
armor_status tc_colblock_gram(armor_ctx* c, const float* U, const float* Y, float* Cm, cudaStream_t s);
// two Grams with a shared operand in one launch (the shared chunks are read once)
armor_status tc_rowblock_gram_pair(armor_ctx* c, const float* P, const float* P2, const float* T, float* G, float* G2,
                                   cudaStream_t s);
armor_status tc_colblock_gram_self_pair(armor_ctx* c, const float* U, const float* Y, float* Cm, float* Cm2, cudaStream_t s);
armor_status tc_select_rows_times_H(armor_ctx* c, const float* Z, const float* H, float* Y, int nbo_pad, cudaStream_t s);
// A tensor-core launch that is refused for its shape or alignment (UNSUPPORTED) is replaced by the CUDA-core
// kernel; any other failure is an error of the call: it is recorded and the entry point returns it.
inline bool tc_done(armor_ctx* c, armor_status st) {
  if (st == ARMOR_OK) return true;
  if (st == ARMOR_ERR_UNSUPPORTED) return false;
  if (c->host_err == ARMOR_OK) c->host_err = st;
  return true;
}
// what an entry point returns: the recorded launch failure, else the state of the runtime
inline armor_status finish_call(armor_ctx* c) {
  const armor_status st = c->host_err;
  c->host_err = ARMOR_OK;
  if (st != ARMOR_OK) return st;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

// Function attributes (the dynamic shared-memory limit) hold per device: one bit per device ordinal and call
// site remembers where the attribute has been set.
struct PerDeviceOnce {
  std::atomic<unsigned long long> mask{0};
  bool done(int dev) const { return dev >= 0 && dev < 64 && ((mask.load(std::memory_order_relaxed) >> dev) & 1ull); }
  void set(int dev) { if (dev >= 0 && dev < 64) mask.fetch_or(1ull << dev, std::memory_order_relaxed); }
};
template <typename K>
inline armor_status ensure_dynamic_smem(PerDeviceOnce& once, int device, K kernel, size_t bytes) {
  if (once.done(device)) return ARMOR_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
    return ARMOR_ERR_CUDA;
  once.set(device);
  return ARMOR_OK;
}

// out = in * H_w (FULL: dense GEMM by cfg.precision; DIAG: column scale) with up to two
// fused dot products <out, d1> -> sc[slot1], <out, d2> -> sc[slot2] (slot < 0: none).
armor_status rmul_H(armor_ctx* c, const float* in, const float* H, float* out, int64_t rows,
                    const float* d1, double* out1, const float* d2, double* out2, cudaStream_t s);
// per-call preparation of everything derived from H (diagonal, diagonal blocks, split copy)
armor_status prepare_H(armor_ctx* c, const float* H, cudaStream_t s);
armor_status gram_accumulate(armor_ctx* c, const void* X, int x_dtype, int64_t n_rows, int64_t ldx, float* H,
                             cudaStream_t s);
// z2 [n, d_out] = z1 [n, d_in] * S^T
armor_status apply_core(armor_ctx* c, const float* z1, const float* S, const void* packed, float* z2, int64_t n,
                        bool bf16, cudaStream_t s);

// operand preparation of the three-pass fp16 mode (split_f16.cu)
void launch_f16_prepare_H(armor_ctx* c, const float* H, cudaStream_t s);   // hpow, scaled H as fp16 hi | lo in Hlo
void launch_f16_split_rows(armor_ctx* c, const float* in, int64_t ld, int64_t rows, int64_t cols, const float* colscale,
                           float post, void* hi, void* lo, float* out_scale, cudaStream_t s);
float f16_H_post_scale();
armor_status launch_f16_gram_stage(armor_ctx* c, const void* X, int x_dtype, int64_t ldx, int64_t rows, int64_t cols,
                                   void* Thi, void* Tlo, int64_t ldt, float* gscale, cudaStream_t s);

// deterministic reductions (two stages, fixed order)
void dot_to_ptr(armor_ctx* c, const float* x, const float* y, int64_t n, double* out, cudaStream_t s);
void dot_partials(armor_ctx* c, const float* x, const float* y, int64_t n, double* part, cudaStream_t s);
void reduce_partials_to(armor_ctx* c, const double* part, int n, double* out, cudaStream_t s);

// streaming kernels (kernels_stream.cu)
void launch_colscale(armor_ctx* c, const float* in, const float* h, float* out, int64_t rows, int64_t cols,
                     cudaStream_t s);
void launch_extract_hblocks(armor_ctx* c, const float* H, cudaStream_t s);   // hdiag, Hjj (per h_mode)
void launch_masked_copy(armor_ctx* c, const float* Gam, const uint8_t* M, float* out, double* part,
                        cudaStream_t s);              // out = Gam (.) M; ARMOR_DOT_BLOCKS partial sums of ||out||^2
void launch_axpy_slot(armor_ctx* c, float* y, const float* x, int64_t n, int slot, float sign,
                      cudaStream_t s);
void launch_axpy_multi(armor_ctx* c, float* y0, const float* x0, float s0, float* y1, const float* x1, float s1, float* y2,
                       const float* x2, float s2, int64_t n, int slot, cudaStream_t s);                                       // y += sign * sc[slot] * x
void launch_init(armor_ctx* c, const float* W, const float* H, float* Wbar, float* r1, float* r2,
                 float* A, float* B, float* S, uint8_t* M, cudaStream_t s);
// st: base of the iteration records (the kernels add c->it_dev), or null
void launch_zero_scalars(armor_ctx* c, bool carry_loss, armor_iter_stats* st, cudaStream_t s);
void launch_advance_iteration(armor_ctx* c, cudaStream_t s);   // ++*c->it_dev
// Input screening at the top of a call: counts non-finite entries of W and H and negative / zero diagonal
// entries of H into the status words and sets or clears ST_POISON for the call.
armor_status launch_screen_inputs(armor_ctx* c, const float* W, const float* H, cudaStream_t s);
// One Adam step (Kingma & Ba, Algorithm 1) on n parameters with gradient g = -2 * gamma; step counts from 1.
// M != nullptr: theta is the N:M core, one mask byte per m_group entries, masked-out entries stay zero.
void launch_adam(armor_ctx* c, float* theta, const float* gamma, float* m, float* v, int64_t n, const uint8_t* M,
                 int64_t step_base, cudaStream_t s);   // step = step_base + *c->it_dev
// part[b] = weight_b * || X_b ||_F for the nblk blocks of db x db floats in X; weight_b = 1, or the Euclidean
// norm of hdiag over the (b % nbi)-th block of columns; out = sum of the parts (fixed order)
void launch_block_fro_sum(armor_ctx* c, const float* X, int nblk, const float* hdiag, double* out, cudaStream_t s);
void launch_zero_flags(armor_ctx* c, cudaStream_t s);
// per-iteration bookkeeping on the device: stage 0 start, 1 after A, 2 after B, 3 after S, 4 mask accept
// (p1, n1, slot1), (p2, n2, slot2): partial sums the stage first adds up into sc[slot] (a preceding dot product)
void launch_stage(armor_ctx* c, armor_iter_stats* st, int stage, const double* part, int npart, int nflag,
                  cudaStream_t s, const double* p1 = nullptr, int n1 = 0, int slot1 = 0, const double* p2 = nullptr,
                  int n2 = 0, int slot2 = 0);
void launch_scale_rows_cols(armor_ctx* c, const float* in, const float* colscale, const float* rowscale,
                            float* out, int64_t rows, int64_t cols, cudaStream_t s);
void launch_split_hilo(armor_ctx* c, const float* in, float* hi, float* lo, int64_t n, cudaStream_t s);
void launch_transpose_split(armor_ctx* c, const void* X, int x_dtype, int64_t ldx, int64_t rows, int64_t cols,
                            float* Thi, float* Tlo, int64_t ldt, cudaStream_t s);
void launch_mirror_lower(armor_ctx* c, float* H, int64_t n, cudaStream_t s);
void launch_bf16_to_f32(armor_ctx* c, const void* in, const float* colscale, float* out, int64_t rows, int64_t cols,
                        cudaStream_t s);
void launch_f32_to_bf16(armor_ctx* c, const float* in, const float* colscale, void* out, int64_t rows, int64_t cols,
                        cudaStream_t s);

// block solves (kernels_chol.cu)
// mode 0: X = rhs (G + lam I)^-1, A += X, out = X, part[b] = exact decrease of block b
// mode 1: out = (G + lam I)^-1 rhs
// mode 2: out = rhs (G + lam I)^-1, part[b] = <dotw, out>
// partial sums written per block by launch_chol (modes 0 and 2)
int chol_parts_per_block(int db, int nb);
// (H_jj + mu I)^-1 for every column block into c->Hinv (H_jj does not change inside a call), failures into c->hinv_fail
armor_status launch_hjj_inverse(armor_ctx* c, cudaStream_t s);
// after Delta = Y Hinv: zeroes the blocks whose H_jj was not positive definite (raising their failflag, as a failed
// solve would) and writes part[j] = <dotw_j, Delta_j>
void launch_delta_finish(armor_ctx* c, float* Delta, const float* dotw, double* part, cudaStream_t s);
armor_status launch_chol(armor_ctx* c, int mode, const float* Gmat, const float* rhs, float* out, const float* dotw,
                         float* A, int nb, double* part, cudaStream_t s);

// sparse-core update (kernels_mask.cu)
void launch_alpha(armor_ctx* c, const float* A, cudaStream_t s);
// alpha and the m x m diagonal blocks of K_j = Y_j B_j^T (Y = B_j H_jj, [nbi, db, db]) in one launch
void launch_mask_prep(armor_ctx* c, const float* A, const float* B, const float* Y, cudaStream_t s);
// selection counter t = t_base + t_mul * (*c->it_dev)
void launch_mask_select(armor_ctx* c, const float* Gam, const float* S, const uint8_t* M, uint64_t t_base, uint64_t t_mul,
                        cudaStream_t s);
// exact loss change of the iteration's group updates without a dense product: fills quadpart with the per-block
// terms of tr(V H_w V^T), V = A dS B, from the selection records (the stage kernel adds them into sc[SC_Q_M])
void launch_mask_quadratic(armor_ctx* c, const float* A, const float* B, const float* H, cudaStream_t s);
void launch_mask_commit(armor_ctx* c, float* S, uint8_t* M, armor_iter_stats* st, cudaStream_t s);
// P += dS B H_w for the accepted group updates, from the rows the guard has formed (full weighting only)
void launch_mask_carry_P(armor_ctx* c, float* P, cudaStream_t s);

// tensor-core GEMM (gemm_tcgen05.cu):  C[M][N] (+)= sum_k A[m][k] * B[n][k]  (both K-major, fp32 storage).
// passes == 3 uses the split operands (A, Alo, B, Blo).  Partial dot products of the output tile with up
// to two W-shaped tensors go to dot partial buffers.
struct TcGemm {
  const void* A; const void* Alo; int64_t lda;   // fp32 arrays (passes 1, 3) or 16-bit arrays (passes 0, 6)
  const void* B; const void* Blo; int64_t ldb;
  float* C; int64_t ldc;
  int64_t M, N, K;
  int passes;            // 1 or 3 tf32 passes on fp32 operands; 0: A and B are 16-bit arrays (one kind::f16 pass);
                         // 6: 16-bit high and low parts, three kind::f16 passes
  int fp16;              // passes 0 / 6: the 16-bit type is fp16 (1) or bf16 (0)
  const float* row_scale; const float* col_scale;   // both or neither: C = acc * row_scale[m] * col_scale[n]
  int64_t k_segment;     // K extent accumulated in tensor memory before it is folded into C (0: all of K)
  int accumulate;        // C += (read-modify-write) instead of C =
  int symmetric_lower;   // only the lower triangle (tiles with n0 <= m0, elements with column <= row) is computed (M == N)
  const float* d1; const float* d2;  // optional dot operands (ld = ldc)
  double* part1; double* part2;      // [tiles] partial sums
};
armor_status launch_tc_gemm(armor_ctx* c, const TcGemm& g, int* n_tiles, cudaStream_t s);
bool tc_gemm_shape_ok(int64_t M, int64_t N, int64_t K);
// the 2:4 core on the sparse tensor cores (sparse_tcgen05.cu)
bool tc_sparse_ok(const armor_ctx* c);
size_t tc_sparse_values_bytes(const armor_ctx* c);
void launch_compress_24(armor_ctx* c, const float* S, const uint8_t* M, void* Sc, void* E, cudaStream_t s);
armor_status launch_tc_sparse(armor_ctx* c, const void* Sc, const void* E, const void* z1_bf16, void* z2, bool out_bf16,
                              int64_t n, cudaStream_t s);
// the wrapper products of the bf16 forward (fwd_tcgen05.cu)
bool fwd_block_ok(const armor_ctx* c);
void launch_pack_blocks(armor_ctx* c, const float* P, const float* rowscale, const float* colscale, void* Q, int nb,
                        cudaStream_t s);
armor_status launch_fwd_block(armor_ctx* c, const void* X, const void* Q, void* out, int64_t rows, int64_t d,
                              cudaStream_t s);
