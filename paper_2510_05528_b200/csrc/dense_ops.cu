// Dense contractions of the ARMOR iteration, dispatched by the configured precision:
// right-multiplication by the weighting H_w, the calibration Gram, and the core product of the
// deployment form.  SIMT = fp32 CUDA cores; TF32 / FP32X3 = tcgen05 tensor cores (1 or 3 tf32 passes);
// FP16X3 = three fp16 passes on operands scaled into the fp16 range (split_f16.cu).
#include <cuda_fp16.h>

#include "armor_internal.cuh"

// The tensor-core accumulator adds with truncation, so a long run of same-sign terms drifts by about
// (K / 8) * passes * 2^-24.  The GEMM therefore drains its accumulator every K_SEGMENT columns of the
// contraction into running sums held by its epilogue warps (ordinary round-to-nearest fp32 adds).
static const int64_t K_SEGMENT = 1024;

armor_status prepare_H(armor_ctx* c, const float* H, cudaStream_t s) {
  launch_extract_hblocks(c, H, s);
  if (c->cfg.h_mode == ARMOR_H_FULL && c->cfg.precision == ARMOR_PREC_FP32X3)
    launch_split_hilo(c, H, nullptr, c->Hlo, c->d_in * c->d_in, s);
  if (c->cfg.h_mode == ARMOR_H_FULL && c->cfg.precision == ARMOR_PREC_FP16X3)
    launch_f16_prepare_H(c, H, s);
  return ARMOR_OK;
}

armor_status rmul_H(armor_ctx* c, const float* in, const float* H, float* out, int64_t rows, const float* d1,
                    double* out1, const float* d2, double* out2, cudaStream_t s) {
  const int64_t d_in = c->d_in;
  if (c->cap_split && c->cfg.h_mode == ARMOR_H_FULL) {
    // capture in pieces: close the piece, remember this product, open the next piece (s is the capturing stream)
    if (c->cap_failed) return ARMOR_OK;
    if (c->cap_n >= ARMOR_MAX_PIECES - 1 || cudaStreamEndCapture(s, &c->cap_graph[c->cap_n]) != cudaSuccess) {
      c->cap_failed = 1;
      return ARMOR_OK;
    }
    c->cap_call[c->cap_n] = {in, H, out, rows, d1, out1, d2, out2};
    ++c->cap_n;
    if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) c->cap_failed = 1;
    return ARMOR_OK;
  }
  if (c->cfg.h_mode == ARMOR_H_DIAG) {
    launch_colscale(c, in, c->hdiag, out, rows, d_in, s);
  } else if (c->cfg.precision == ARMOR_PREC_SIMT) {
    BGemm g{};
    g.A = in; g.sAm = d_in; g.sAk = 1;
    g.B = H; g.sBk = d_in; g.sBn = 1;
    g.C = out; g.sCm = d_in; g.sCn = 1;
    g.M = (int)rows; g.N = (int)d_in; g.K = (int)d_in; g.batch = 1; g.alpha = 1.f;
    launch_bgemm(c, g, s);
  } else {
    TcGemm g{};
    g.lda = d_in; g.ldb = d_in; g.ldc = d_in;
    g.M = rows; g.N = d_in; g.K = d_in;
    g.C = out;
    if (c->cfg.precision == ARMOR_PREC_FP32X3) {
      // left operand as a high part plus the fp32 remainder.  The tensor core ignores the low 13 bits of a
      // 32-bit operand, so the operand itself serves as its high part and only the remainder is written.
      launch_split_hilo(c, in, nullptr, c->Lo, rows * d_in, s);
      g.A = in; g.Alo = c->Lo; g.B = H; g.Blo = c->Hlo; g.passes = 3;
    } else if (c->cfg.precision == ARMOR_PREC_FP16X3) {
      // in . H = rowscale . [(in d) rho] [H / (d d^T) 2^12] . d : both factors as fp16 high and low parts
      __half* ahi = reinterpret_cast<__half*>(c->Lo);
      __half* hhi = reinterpret_cast<__half*>(c->Hlo);
      launch_f16_split_rows(c, in, d_in, rows, d_in, c->hpow, f16_H_post_scale(), ahi, ahi + rows * d_in, c->rowscale, s);
      g.A = ahi; g.Alo = ahi + rows * d_in; g.B = hhi; g.Blo = hhi + d_in * d_in; g.passes = 6; g.fp16 = 1;
      g.row_scale = c->rowscale; g.col_scale = c->hpow;
    } else {
      g.A = in; g.B = H; g.passes = 1;
    }
    g.d1 = d1; g.d2 = d2;
    g.k_segment = (g.passes >= 3) ? K_SEGMENT : 0;   // one-pass tf32 rounding (2^-11) dwarfs the accumulator drift
    g.part1 = d1 ? c->partials : nullptr;
    g.part2 = d2 ? c->partials + 8 * c->npart : nullptr;
    int tiles = 0;
    armor_status st = launch_tc_gemm(c, g, &tiles, s);
    if (st != ARMOR_OK) return st;
    if (d1) reduce_partials_to(c, c->partials, 8 * tiles, out1, s);
    if (d2) reduce_partials_to(c, c->partials + 8 * c->npart, 8 * tiles, out2, s);
    return ARMOR_OK;
  }
  if (d1) dot_to_ptr(c, out, d1, rows * d_in, out1, s);
  if (d2) dot_to_ptr(c, out, d2, rows * d_in, out2, s);
  return ARMOR_OK;
}

armor_status gram_accumulate(armor_ctx* c, const void* Xv, int x_dtype, int64_t n_rows, int64_t ldx, float* H,
                             cudaStream_t s) {
  const int64_t d_in = c->d_in;
  const float* X = static_cast<const float*>(Xv);
  const bool bf16 = (x_dtype == ARMOR_DTYPE_BF16);
  if (c->cfg.precision == ARMOR_PREC_SIMT) {
    if (bf16) return ARMOR_ERR_UNSUPPORTED;
    // H += X^T X, element (m, k) of the left operand is X[k][m]
    const int64_t step = 1 << 20;
    for (int64_t r0 = 0; r0 < n_rows; r0 += step) {
      const int64_t n = n_rows - r0 < step ? n_rows - r0 : step;
      BGemm g{};
      g.A = X + r0 * ldx; g.sAm = 1; g.sAk = ldx;
      g.B = X + r0 * ldx; g.sBk = ldx; g.sBn = 1;
      g.C = H; g.sCm = d_in; g.sCn = 1;
      g.D = H; g.sDm = d_in; g.sDn = 1;
      g.M = (int)d_in; g.N = (int)d_in; g.K = (int)n; g.batch = 1; g.alpha = 1.f; g.beta = 1.f;
      launch_bgemm(c, g, s);
    }
    return ARMOR_OK;
  }
  if (c->cfg.precision == ARMOR_PREC_FP16X3) {
    // every chunk is scaled per channel into the fp16 range; bf16 activations are then exact in one fp16 part
    const size_t esz = bf16 ? 2 : 4;
    // A call of several chunks stages chunk p + 1 (HBM bound) on the context's side stream while the tensor cores
    // contract chunk p on the caller's stream: two staging buffers with their scales, an event per hand-over.  The
    // contractions stay in the caller's stream in chunk order, so H is the same bit for bit.
    const int64_t n_chunks = (n_rows + c->gram_rows - 1) / c->gram_rows;
    bool overlap = n_chunks > 1 && c->side_stream && c->Xt_hi2 && c->timing_on < 2;
    if (overlap) {
      cudaStreamCaptureStatus cst = cudaStreamCaptureStatusNone;
      if (cudaStreamIsCapturing(s, &cst) != cudaSuccess || cst != cudaStreamCaptureStatusNone) overlap = false;
    }
    if (overlap) {
      // the side stream starts where the caller's stream is now: the inputs are ready and both buffers are free
      if (cudaEventRecord(c->ev_fork, s) != cudaSuccess || cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0) != cudaSuccess)
        return ARMOR_ERR_CUDA;
    }
    int64_t p = 0;
    for (int64_t r0 = 0; r0 < n_rows; r0 += c->gram_rows, ++p) {
      const int b = overlap ? (int)(p & 1) : 0;
      __half* thi = reinterpret_cast<__half*>(b ? c->Xt_hi2 : c->Xt_hi);
      __half* tlo = thi + d_in * c->gram_rows;
      float* gscale = b ? c->gscale2 : c->gscale;
      cudaStream_t ss = overlap ? c->side_stream : s;
      const int64_t n = n_rows - r0 < c->gram_rows ? n_rows - r0 : c->gram_rows;
      const int64_t kpad = (n + 63) / 64 * 64;
      // buffer b was last read by the contraction of chunk p - 2
      if (overlap && p >= 2 && cudaStreamWaitEvent(ss, c->ev_used[b], 0) != cudaSuccess) return ARMOR_ERR_CUDA;
      armor_status st = launch_f16_gram_stage(c, static_cast<const char*>(Xv) + (size_t)(r0 * ldx) * esz, x_dtype, ldx, n,
                                              d_in, thi, tlo, kpad, gscale, ss);
      if (st != ARMOR_OK) return st;
      if (overlap && (cudaEventRecord(c->ev_staged[b], ss) != cudaSuccess ||
                      cudaStreamWaitEvent(s, c->ev_staged[b], 0) != cudaSuccess))
        return ARMOR_ERR_CUDA;
      TcGemm g{};
      g.A = thi; g.Alo = tlo; g.lda = kpad;
      g.B = thi; g.Blo = tlo; g.ldb = kpad;
      g.C = H; g.ldc = d_in;
      g.M = d_in; g.N = d_in; g.K = kpad;
      g.passes = bf16 ? 0 : 6; g.fp16 = 1;
      g.row_scale = gscale; g.col_scale = gscale;
      g.accumulate = 1;
      g.symmetric_lower = 1;
      g.k_segment = K_SEGMENT;
      st = launch_tc_gemm(c, g, nullptr, s);
      if (st != ARMOR_OK) return st;
      if (overlap && cudaEventRecord(c->ev_used[b], s) != cudaSuccess) return ARMOR_ERR_CUDA;
    }
    launch_mirror_lower(c, H, d_in, s);
    return ARMOR_OK;
  }
  // bf16 values are exact in tf32: one tensor-core pass gives exact products
  const bool x3 = c->cfg.precision == ARMOR_PREC_FP32X3 && !bf16;
  const size_t esz = bf16 ? 2 : 4;
  for (int64_t r0 = 0; r0 < n_rows; r0 += c->gram_rows) {
    const int64_t n = n_rows - r0 < c->gram_rows ? n_rows - r0 : c->gram_rows;
    const int64_t kpad = (n + 31) / 32 * 32;     // staged row length (zero padded)
    launch_transpose_split(c, static_cast<const char*>(Xv) + (size_t)(r0 * ldx) * esz, x_dtype, ldx, n, d_in, c->Xt_hi,
                           x3 ? c->Xt_lo : nullptr, kpad, s);
    TcGemm g{};
    g.A = c->Xt_hi; g.Alo = c->Xt_lo; g.lda = kpad;
    g.B = c->Xt_hi; g.Blo = c->Xt_lo; g.ldb = kpad;
    g.C = H; g.ldc = d_in;
    g.M = d_in; g.N = d_in; g.K = kpad;
    g.passes = x3 ? 3 : 1;
    g.accumulate = 1;
    g.symmetric_lower = 1;
    g.k_segment = (c->cfg.precision == ARMOR_PREC_FP32X3) ? K_SEGMENT : 4 * K_SEGMENT;
    armor_status st = launch_tc_gemm(c, g, nullptr, s);
    if (st != ARMOR_OK) return st;
  }
  launch_mirror_lower(c, H, d_in, s);   // the product accumulates the lower triangle only
  return ARMOR_OK;
}

armor_status apply_core(armor_ctx* c, const float* z1, const float* S, const void* packed, float* z2, int64_t n,
                        bool bf16, cudaStream_t s) {
  const int64_t d_in = c->d_in, d_out = c->d_out;
  if (packed) {
    // bf16 deployment with the 2:4 core on the sparse tensor cores: kept values, then positions
    if (!bf16 || !tc_sparse_ok(c)) return ARMOR_ERR_UNSUPPORTED;
    const char* buf = static_cast<const char*>(packed);
    launch_f32_to_bf16(c, z1, nullptr, c->U, n, d_in, s);
    return launch_tc_sparse(c, buf, buf + tc_sparse_values_bytes(c), c->U, z2, false, n, s);
  }
  if (bf16 && c->cfg.precision != ARMOR_PREC_SIMT && d_out % 32 == 0 && d_in % 8 == 0) {
    // bf16 deployment: the core and the wrapped activations are rounded to bf16 and multiplied on the bf16
    // tensor-core path with fp32 accumulation
    launch_f32_to_bf16(c, z1, nullptr, c->U, n, d_in, s);
    launch_f32_to_bf16(c, S, nullptr, c->P, d_out, d_in, s);
    TcGemm g{};
    g.lda = d_in; g.ldb = d_in; g.ldc = d_out;
    g.M = n; g.N = d_out; g.K = d_in;
    g.C = z2;
    g.A = c->U; g.B = c->P; g.passes = 0;
    g.k_segment = 0;
    return launch_tc_gemm(c, g, nullptr, s);
  }
  if (c->cfg.precision == ARMOR_PREC_SIMT || (d_out % 32) || (d_in % 4)) {
    BGemm g{};
    g.A = z1; g.sAm = d_in; g.sAk = 1;
    g.B = S; g.sBk = 1; g.sBn = d_in;
    g.C = z2; g.sCm = d_out; g.sCn = 1;
    g.M = (int)n; g.N = (int)d_out; g.K = (int)d_in; g.batch = 1; g.alpha = 1.f;
    launch_bgemm(c, g, s);
    return ARMOR_OK;
  }
  TcGemm g{};
  g.lda = d_in; g.ldb = d_in; g.ldc = d_out;
  g.M = n; g.N = d_out; g.K = d_in;
  g.C = z2;
  if (c->cfg.precision == ARMOR_PREC_FP32X3) {
    launch_split_hilo(c, z1, nullptr, c->Lo, n * d_in, s);
    launch_split_hilo(c, S, nullptr, c->U, c->wn, s);
    g.A = z1; g.Alo = c->Lo; g.B = S; g.Blo = c->U; g.passes = 3;
  } else if (c->cfg.precision == ARMOR_PREC_FP16X3) {
    // rows of z1 (tokens) and rows of S (outputs) each scaled by their own power of two
    __half* ahi = reinterpret_cast<__half*>(c->Lo);
    __half* shi = reinterpret_cast<__half*>(c->U);
    launch_f16_split_rows(c, z1, d_in, n, d_in, nullptr, 1.f, ahi, ahi + n * d_in, c->rowscale, s);
    launch_f16_split_rows(c, S, d_in, d_out, d_in, nullptr, 1.f, shi, shi + c->wn, c->rowscale2, s);
    g.A = ahi; g.Alo = ahi + n * d_in; g.B = shi; g.Blo = shi + c->wn; g.passes = 6; g.fp16 = 1;
    g.row_scale = c->rowscale; g.col_scale = c->rowscale2;
  } else {
    g.A = z1; g.B = S; g.passes = 1;
  }
  g.k_segment = (g.passes >= 3) ? K_SEGMENT : 0;
  return launch_tc_gemm(c, g, nullptr, s);
}
