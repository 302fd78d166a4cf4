// C ABI entry points and the host-side orchestration of one ARMOR layer optimisation.
#include <new>

#include "armor_internal.cuh"

namespace {

constexpr int LOSS_REFRESH = 64;      // iterations of a call between two evaluations of the loss from the residual
constexpr int64_t GRAM_ROWS = 16384;  // rows of X staged (transposed, split) per tensor-core Gram pass

struct Layout {
  size_t total = 0;
  size_t take(size_t bytes) {
    size_t off = total;
    total += (bytes + 255) / 256 * 256;
    return off;
  }
};

armor_status check_config(const armor_config* cfg) {
  if (!cfg) return ARMOR_ERR_INVALID_ARG;
  if (cfg->d_out <= 0 || cfg->d_in <= 0 || cfg->d_block <= 0) return ARMOR_ERR_SHAPE;
  if (cfg->m_group <= 0 || cfg->n_keep <= 0 || cfg->n_keep > cfg->m_group) return ARMOR_ERR_SHAPE;
  if (cfg->d_out % cfg->d_block || cfg->d_in % cfg->d_block || cfg->d_block % cfg->m_group) return ARMOR_ERR_SHAPE;
  if (!((cfg->n_keep == 2 && cfg->m_group == 4) || (cfg->m_group == 8 && cfg->n_keep >= 4 && cfg->n_keep <= 6)))
    return ARMOR_ERR_UNSUPPORTED;   // 2:4, and the 4:8, 5:8, 6:8 patterns of Section 4.4
  if (cfg->d_block > 256 || cfg->d_block % 4) return ARMOR_ERR_UNSUPPORTED;
  if (cfg->d_block > 128 && cfg->d_block % 32) return ARMOR_ERR_UNSUPPORTED;   // large blocks use the panel solver
  if (cfg->h_mode != ARMOR_H_FULL && cfg->h_mode != ARMOR_H_DIAG) return ARMOR_ERR_INVALID_ARG;
  if (cfg->select_mode < ARMOR_SELECT_L1_RANDOM || cfg->select_mode > ARMOR_SELECT_L2_RANDOM) return ARMOR_ERR_INVALID_ARG;
  if (cfg->s_step != ARMOR_S_EXACT && cfg->s_step != ARMOR_S_BETA) return ARMOR_ERR_INVALID_ARG;
  if (cfg->ab_step < ARMOR_AB_EXACT || cfg->ab_step > ARMOR_AB_ADAM) return ARMOR_ERR_INVALID_ARG;
  if (cfg->mask_sweeps < 0 || cfg->mask_sweeps > 64) return ARMOR_ERR_INVALID_ARG;
  if (cfg->mask_groups < 0 || cfg->mask_groups > 8) return ARMOR_ERR_INVALID_ARG;
  if (cfg->adam_lr < 0.f || cfg->adam_beta1 < 0.f || cfg->adam_beta1 >= 1.f || cfg->adam_beta2 < 0.f ||
      cfg->adam_beta2 >= 1.f || cfg->adam_eps < 0.f)
    return ARMOR_ERR_INVALID_ARG;
  if (cfg->ab_step == ARMOR_AB_GD && cfg->h_mode != ARMOR_H_DIAG) return ARMOR_ERR_UNSUPPORTED;
  if (cfg->precision < ARMOR_PREC_FP32X3 || cfg->precision > ARMOR_PREC_FP16X3) return ARMOR_ERR_INVALID_ARG;
  if (cfg->precision != ARMOR_PREC_SIMT) {
    // the tensor-core GEMM works on whole 128 x 128 tiles with K in steps of 32
    if (cfg->h_mode == ARMOR_H_FULL && (cfg->d_out % 128 || cfg->d_in % 128)) return ARMOR_ERR_UNSUPPORTED;
  }
  if (!(cfg->ridge >= 0.f)) return ARMOR_ERR_INVALID_ARG;
  if (cfg->phases < 0 || cfg->phases > 15) return ARMOR_ERR_INVALID_ARG;
  return ARMOR_OK;
}

// Carves the workspace; with ctx == nullptr only the size is computed.
size_t carve(const armor_config& cfg, armor_ctx* c, char* base) {
  Layout L;
  const int64_t wn = cfg.d_out * cfg.d_in;
  const int db = cfg.d_block;
  const int64_t nbo = cfg.d_out / db, nbi = cfg.d_in / db;
  const size_t wbytes = (size_t)wn * sizeof(float);
  const size_t hbytes = (size_t)cfg.d_in * cfg.d_in * sizeof(float);
  const bool tc = cfg.precision != ARMOR_PREC_SIMT;
  const bool x3 = cfg.precision == ARMOR_PREC_FP32X3 || cfg.precision == ARMOR_PREC_FP16X3;   // split operands
#define TAKE(field, type, bytes)                         \
  do {                                                   \
    size_t off_ = L.take(bytes);                         \
    if (c) c->field = reinterpret_cast<type>(base + off_); \
  } while (0)
  TAKE(T, float*, wbytes);
  TAKE(E, float*, wbytes);
  TAKE(EH, float*, wbytes);
  TAKE(P, float*, wbytes);
  TAKE(U, float*, wbytes);
  TAKE(V, float*, wbytes);
  TAKE(VH, float*, wbytes);
  TAKE(Gam, float*, wbytes);
  TAKE(Tmp, float*, wbytes);
  TAKE(WH, float*, wbytes);
  if (x3) { TAKE(Lo, float*, wbytes); } else if (c) { c->Lo = nullptr; }
  if (x3) { TAKE(Hlo, float*, hbytes); } else if (c) { c->Hlo = nullptr; }
  const size_t ao = (size_t)nbo * db * db * sizeof(float), bo = (size_t)nbi * db * db * sizeof(float);
  TAKE(G, float*, ao);
  TAKE(GamA, float*, ao);
  TAKE(dA, float*, ao);
  TAKE(C, float*, bo);
  TAKE(GamB, float*, bo);
  TAKE(Delta, float*, bo);
  TAKE(Hjj, float*, bo);
  TAKE(Kfull, float*, bo);
  TAKE(Ktmp, float*, bo);
  TAKE(Hinv, float*, bo);
  TAKE(hinv_fail, int32_t*, (size_t)nbi * sizeof(int32_t));
  TAKE(alpha, float*, (size_t)cfg.d_out * sizeof(float));
  TAKE(hdiag, float*, (size_t)cfg.d_in * sizeof(float));
  const int64_t nbo_pad = (nbo + 31) / 32 * 32;
  const int64_t kg = cfg.mask_groups > 0 ? cfg.mask_groups : 1;   // draws per block: every per-draw table grows by kg
  TAKE(Zsel, float*, (size_t)nbo_pad * nbi * kg * db * sizeof(float));
  TAKE(Acol, float*, (size_t)nbo * nbi * kg * db * sizeof(float));
  TAKE(Ysel, float*, (size_t)nbo_pad * nbi * kg * cfg.d_in * sizeof(float));
  if (c) c->nbo_pad = (int)nbo_pad;
  TAKE(colpart, double*, (size_t)64 * cfg.d_in * sizeof(double));
  {
    const int64_t dmax = cfg.d_out > cfg.d_in ? cfg.d_out : cfg.d_in;
    TAKE(hpow, float*, (size_t)cfg.d_in * sizeof(float));
    TAKE(gscale, float*, (size_t)cfg.d_in * sizeof(float));
    TAKE(gscale2, float*, (size_t)cfg.d_in * sizeof(float));
    TAKE(gmax, unsigned*, (size_t)cfg.d_in * sizeof(unsigned));
    TAKE(rowscale, float*, (size_t)dmax * sizeof(float));
    TAKE(rowscale2, float*, (size_t)dmax * sizeof(float));
  }
  if (tc) {
    TAKE(gemm_slabs, float*, (size_t)160 * 128 * 256 * sizeof(float));
    if (c) c->gemm_slab_count = 160;
    TAKE(Xt_hi, float*, (size_t)cfg.d_in * GRAM_ROWS * sizeof(float));
    // (the fp16 mode keeps both 16-bit parts of the staged chunk in Xt_hi)
    if (cfg.precision == ARMOR_PREC_FP32X3) TAKE(Xt_lo, float*, (size_t)cfg.d_in * GRAM_ROWS * sizeof(float)); else if (c) c->Xt_lo = nullptr;
    if (cfg.precision == ARMOR_PREC_FP16X3) TAKE(Xt_hi2, float*, (size_t)cfg.d_in * GRAM_ROWS * sizeof(float)); else if (c) c->Xt_hi2 = nullptr;
  } else if (c) { c->Xt_hi = nullptr; c->Xt_lo = nullptr; c->Xt_hi2 = nullptr; c->gemm_slabs = nullptr; c->gemm_slab_count = 0; }
  const int64_t tiles = ((cfg.d_out + 127) / 128) * ((cfg.d_in + 127) / 128) + ((cfg.d_in + 127) / 128) * ((cfg.d_in + 127) / 128);
  const int64_t npart = tiles > ARMOR_DOT_BLOCKS ? tiles : ARMOR_DOT_BLOCKS;
  {
    const int64_t tiles = (int64_t)((db + 127) / 128) * ((db + 127) / 128);
    const int64_t g1 = 2 * nbo * pick_ksplit(2 * nbo, tiles, cfg.d_in) * (int64_t)db * db;
    const int64_t g2 = 2 * nbi * pick_ksplit(2 * nbi, tiles, cfg.d_out) * (int64_t)db * db;
    int64_t gp = g1 > g2 ? g1 : g2;
    const int64_t nbm = nbo > nbi ? nbo : nbi;
    if (gp < 16 * nbm * (int64_t)db * db) gp = 16 * nbm * (int64_t)db * db;   // up to 16 slabs of one Gram
    TAKE(gpart, float*, (size_t)gp * sizeof(float));
    if (c) c->gpart_floats = gp;
  }
  if (cfg.s_step == ARMOR_S_BETA && cfg.h_mode == ARMOR_H_FULL) {
    TAKE(Hq1, float*, hbytes);
    TAKE(Hq2, float*, hbytes);
  } else if (c) { c->Hq1 = nullptr; c->Hq2 = nullptr; }
  if (cfg.ab_step == ARMOR_AB_ADAM) {
    TAKE(mA, float*, ao); TAKE(vA, float*, ao);
    TAKE(mB, float*, bo); TAKE(vB, float*, bo);
    TAKE(mS, float*, wbytes); TAKE(vS, float*, wbytes);
  } else if (c) { c->mA = c->vA = c->mB = c->vB = c->mS = c->vS = nullptr; }
  TAKE(sc, double*, SC_COUNT * sizeof(double));
  TAKE(partials, double*, (size_t)16 * npart * sizeof(double));
  const int64_t nbmax = nbo > nbi ? nbo : nbi;
  TAKE(partblk, double*, (size_t)(4 * nbmax > nbo * nbi * kg ? 4 * nbmax : nbo * nbi * kg) * sizeof(double));
  TAKE(quadpart, double*, (size_t)nbo * nbi * kg * sizeof(double));
  TAKE(failflag, int32_t*, (size_t)nbmax * sizeof(int32_t));
  TAKE(sel, SelRec*, (size_t)nbo * nbi * kg * sizeof(SelRec));
  TAKE(tab_key, float*, (size_t)nbo * nbi * sizeof(float));
  TAKE(tab_g, unsigned long long*, (size_t)nbo * nbi * sizeof(unsigned long long));
  TAKE(status, int32_t*, ST_COUNT * sizeof(int32_t));
  TAKE(screen, int32_t*, 4 * sizeof(int32_t));
  TAKE(it_dev, int64_t*, sizeof(int64_t));
#undef TAKE
  if (c) {
    c->npart = npart;
    c->gram_rows = GRAM_ROWS;
  }
  return L.total;
}

inline cudaStream_t cs(armor_stream_t s) { return reinterpret_cast<cudaStream_t>(s); }

// per-block Gram-type products over a long contraction, two at a time (the second pair of operands is
// addressed through the distance between workspace buffers)
void rowblock_grams(armor_ctx* c, const float* P, const float* P2, const float* T, float* G, float* G2, cudaStream_t s) {
  // G_i = P_i T_i^T, G2_i = P2_i T_i^T  (contraction over d_in), batch over row-blocks i; P == nullptr: G2 only
  const int db = c->db;
  if (c->tc_blocks && tc_gram_ok(c)) {
    if (P && c->gram_pairs && tc_done(c, tc_rowblock_gram_pair(c, P, P2, T, G, G2, s))) return;
    armor_status st = P ? tc_rowblock_gram(c, P, T, G, s) : ARMOR_OK;
    if (st == ARMOR_OK) st = tc_rowblock_gram(c, P2, T, G2, s);
    if (tc_done(c, st)) return;
  }
  if (!P) { P = P2; G = G2; }   // fallback kernel: the same Gram twice into the same place
  BGemm g{};
  g.A = P; g.sAb = (int64_t)db * c->d_in; g.sAm = c->d_in; g.sAk = 1;
  g.B = T; g.sBb = (int64_t)db * c->d_in; g.sBk = 1; g.sBn = c->d_in;
  g.C = G; g.sCb = (int64_t)db * db; g.sCm = db; g.sCn = 1;
  g.M = db; g.N = db; g.K = (int)c->d_in; g.batch = 2 * c->nbo; g.alpha = 1.f;
  g.batch_inner = c->nbo; g.sAb2 = P2 - P; g.sBb2 = 0; g.sCb2 = G2 - G;
  g.ksplit = pick_ksplit(g.batch, (int64_t)((db + 127) / 128) * ((db + 127) / 128), g.K);
  launch_bgemm(c, g, s);
}
void colblock_grams(armor_ctx* c, const float* U, const float* Y, const float* Y2, float* Cm, float* Cm2, cudaStream_t s) {
  // C_j = U_j^T Y_j, C2_j = U_j^T Y2_j  (contraction over d_out), batch over column-blocks j; Y == nullptr: C2 only
  const int db = c->db;
  if (c->tc_blocks && tc_gram_ok(c)) {
    if (Y == U && c->gram_pairs && tc_done(c, tc_colblock_gram_self_pair(c, U, Y2, Cm, Cm2, s))) return;
    armor_status st = Y ? tc_colblock_gram(c, U, Y, Cm, s) : ARMOR_OK;
    if (st == ARMOR_OK) st = tc_colblock_gram(c, U, Y2, Cm2, s);
    if (tc_done(c, st)) return;
  }
  if (!Y) { Y = Y2; Cm = Cm2; }
  BGemm g{};
  g.A = U; g.sAb = db; g.sAm = 1; g.sAk = c->d_in;
  g.B = Y; g.sBb = db; g.sBk = c->d_in; g.sBn = 1;
  g.C = Cm; g.sCb = (int64_t)db * db; g.sCm = db; g.sCn = 1;
  g.M = db; g.N = db; g.K = (int)c->d_out; g.batch = 2 * c->nbi; g.alpha = 1.f;
  g.batch_inner = c->nbi; g.sAb2 = 0; g.sBb2 = Y2 - Y; g.sCb2 = Cm2 - Cm;
  g.ksplit = pick_ksplit(g.batch, (int64_t)((db + 127) / 128) * ((db + 127) / 128), g.K);
  launch_bgemm(c, g, s);
}
// Z_(i,j) = X_ij Y_ij^T (by_rows) or X_ij^T Y_ij for every d_block x d_block tile (i, j) of two W-shaped
// matrices: the terms of the paper's smoothness constants (Eq. lrA: T_ij D_j T_ij^T, Eq. lrB: U_ij^T U_ij).
void tile_grams(armor_ctx* c, const float* X, const float* Y, bool by_rows, float* Z, cudaStream_t s) {
  const int db = c->db;
  const int64_t d_in = c->d_in;
  BGemm g{};
  g.A = X; g.B = Y;
  if (by_rows) { g.sAm = d_in; g.sAk = 1; g.sBk = 1; g.sBn = d_in; }
  else         { g.sAm = 1; g.sAk = d_in; g.sBk = d_in; g.sBn = 1; }
  g.sAb = db; g.sAb2 = (int64_t)db * d_in; g.sBb = db; g.sBb2 = (int64_t)db * d_in;
  g.C = Z; g.sCb = (int64_t)db * db; g.sCb2 = (int64_t)c->nbi * db * db; g.sCm = db; g.sCn = 1;
  g.M = db; g.N = db; g.K = db; g.batch = c->nbo * c->nbi; g.batch_inner = c->nbi; g.alpha = 1.f;
  launch_bgemm(c, g, s);
}
void block_mm(armor_ctx* c, const float* X, bool tX, const float* Y, bool tY, float* Z, int nb, cudaStream_t s) {
  const int db = c->db;
  BGemm g{};
  g.A = X; g.sAb = (int64_t)db * db; g.sAm = tX ? 1 : db; g.sAk = tX ? db : 1;
  g.B = Y; g.sBb = (int64_t)db * db; g.sBk = tY ? 1 : db; g.sBn = tY ? db : 1;
  g.C = Z; g.sCb = (int64_t)db * db; g.sCm = db; g.sCn = 1;
  g.M = db; g.N = db; g.K = db; g.batch = nb; g.alpha = 1.f;
  launch_bgemm(c, g, s);
}

armor_status reset_adam(armor_ctx* c, cudaStream_t s) {
  if (c->cfg.ab_step != ARMOR_AB_ADAM) return ARMOR_OK;
  const size_t ao = (size_t)c->nbo * c->db * c->db * sizeof(float), bo = (size_t)c->nbi * c->db * c->db * sizeof(float);
  const size_t wb = (size_t)c->wn * sizeof(float);
  ARMOR_CUDA_OK(cudaMemsetAsync(c->mA, 0, ao, s)); ARMOR_CUDA_OK(cudaMemsetAsync(c->vA, 0, ao, s));
  ARMOR_CUDA_OK(cudaMemsetAsync(c->mB, 0, bo, s)); ARMOR_CUDA_OK(cudaMemsetAsync(c->vB, 0, bo, s));
  ARMOR_CUDA_OK(cudaMemsetAsync(c->mS, 0, wb, s)); ARMOR_CUDA_OK(cudaMemsetAsync(c->vS, 0, wb, s));
  return ARMOR_OK;
}

armor_status core_gradient(armor_ctx* c, const float* A, const float* B, cudaStream_t s) {
  // Gamma = A^T (E H_w) B^T  (minus half of the gradient display of Appendix D.3)
  bd_two_sided(c, A, true, c->EH, B, true, c->Tmp, c->Gam, c->d_out, c->d_in, 1.f, s);
  return ARMOR_OK;
}

armor_status residual_and_loss(armor_ctx* c, const float* W, const float* H, const float* A, const float* B,
                               const float* S, double* out, cudaStream_t s, bool exact_products = false) {
  // exact_products: the two wrapper products on the fp32 CUDA-core kernel, whose products with 0 and 1 are
  // exact, so that E vanishes exactly where W = A S B term by term (identity wrappers at the initialisation);
  // the three-pass tensor-core product carries 22 bits of each operand
  const int saved = c->tc_blocks;
  if (exact_products) c->tc_blocks = 0;
  bd_right(c, S, B, false, c->T, c->d_out, c->d_in, 1.f, nullptr, 0.f, s);      // T = S B
  if (c->cfg.h_mode == ARMOR_H_DIAG && c->tc_blocks && tc_block_ok(c, c->d_out, c->d_in)) {
    // diagonal weighting: E = W - A T, E H_w = E diag(h) and L = <E H_w, E> in one pass
    int nq = 0;
    if (tc_done(c, tc_bd_left_residual(c, A, c->T, W, c->hdiag, c->E, c->EH, c->d_out, c->d_in, c->partials, &nq, s))) {
      c->tc_blocks = saved;
      reduce_partials_to(c, c->partials, nq, out, s);
      return ARMOR_OK;
    }
  }
  bd_left(c, A, false, c->T, c->E, c->d_out, c->d_in, -1.f, W, 1.f, s);         // E = W - A T
  c->tc_blocks = saved;
  return rmul_H(c, c->E, H, c->EH, c->d_out, c->E, out, nullptr, nullptr, s);   // EH = E H_w, L = <EH, E>
}

}  // namespace

extern "C" {

const char* armor_status_string(armor_status st) {
  switch (st) {
    case ARMOR_OK: return "ok";
    case ARMOR_ERR_INVALID_ARG: return "invalid argument";
    case ARMOR_ERR_SHAPE: return "shape error: d_block must divide d_out and d_in, m_group must divide d_block";
    case ARMOR_ERR_WORKSPACE: return "workspace too small or misaligned";
    case ARMOR_ERR_CUDA: return "CUDA runtime error";
    case ARMOR_ERR_NOT_SPD: return "block not positive definite";
    case ARMOR_ERR_TIMEOUT: return "bounded device wait ran out";
    case ARMOR_ERR_UNSUPPORTED: return "configuration not supported";
    case ARMOR_ERR_TOO_LARGE: return "size exceeds the built-in scratch of the no-allocation entry point";
  }
  return "unknown status";
}

armor_status armor_workspace_bytes(const armor_config* cfg, size_t* bytes) {
  if (!bytes) return ARMOR_ERR_INVALID_ARG;
  armor_status st = check_config(cfg);
  if (st != ARMOR_OK) return st;
  *bytes = carve(*cfg, nullptr, nullptr);
  return ARMOR_OK;
}

armor_status armor_create(armor_ctx** out, const armor_config* cfg, void* d_workspace, size_t bytes) {
  if (!out) return ARMOR_ERR_INVALID_ARG;
  *out = nullptr;
  armor_status st = check_config(cfg);
  if (st != ARMOR_OK) return st;
  if (!d_workspace) return ARMOR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_workspace) % 256) return ARMOR_ERR_WORKSPACE;
  if (bytes < carve(*cfg, nullptr, nullptr)) return ARMOR_ERR_WORKSPACE;
  armor_ctx* c = new (std::nothrow) armor_ctx();
  if (!c) return ARMOR_ERR_INVALID_ARG;
  c->cfg = *cfg;
  if (c->cfg.phases == 0) c->cfg.phases = 15;
  c->d_out = cfg->d_out; c->d_in = cfg->d_in; c->wn = cfg->d_out * cfg->d_in;
  c->db = cfg->d_block; c->nbo = (int)(cfg->d_out / cfg->d_block); c->nbi = (int)(cfg->d_in / cfg->d_block);
  c->ws = static_cast<char*>(d_workspace); c->ws_bytes = bytes;
  c->launches = 0;
  c->tc_blocks = 3;
  c->gram_pairs = 1;
  c->host_err = ARMOR_OK;
  if (cudaGetDevice(&c->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess || c->n_sm < 1) {
    delete c;
    return ARMOR_ERR_CUDA;
  }
  c->use_graphs = 1;
  c->cap_split = 0; c->cap_n = 0; c->cap_failed = 0;
  c->cap_stream = nullptr;
  if (cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) != cudaSuccess) c->cap_stream = nullptr;
  // a second stream of the context's own and five events: the Gram stages chunk p + 1 there while chunk p is contracted
  c->side_stream = nullptr;
  c->ev_fork = nullptr;
  for (int k = 0; k < 2; ++k) { c->ev_staged[k] = nullptr; c->ev_used[k] = nullptr; }
  {
    bool ok = cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    for (int k = 0; k < 2 && ok; ++k)
      ok = cudaEventCreateWithFlags(&c->ev_staged[k], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->ev_used[k], cudaEventDisableTiming) == cudaSuccess;
    if (!ok && c->side_stream) { cudaStreamDestroy(c->side_stream); c->side_stream = nullptr; }   // the Gram then runs in one stream
  }
  c->kg = cfg->mask_groups > 0 ? cfg->mask_groups : 1;
  c->h_cached = nullptr;
  c->timing_on = 0; c->timing_n = 0; c->ev_beg = nullptr; c->ev_end = nullptr; c->ev_cls = nullptr; c->ev_work = nullptr;
  c->ev_created = 0;
  carve(*cfg, c, c->ws);
  if (cudaMemset(c->status, 0, ST_COUNT * sizeof(int32_t)) != cudaSuccess) { delete c; return ARMOR_ERR_CUDA; }
  if (cudaMemset(c->sc, 0, SC_COUNT * sizeof(double)) != cudaSuccess) { delete c; return ARMOR_ERR_CUDA; }
  *out = c;
  return ARMOR_OK;
}

armor_status armor_destroy(armor_ctx* c) {
  if (!c) return ARMOR_ERR_INVALID_ARG;
  for (int i = 0; i < c->ev_created; ++i) { cudaEventDestroy(c->ev_beg[i]); cudaEventDestroy(c->ev_end[i]); }
  delete[] c->ev_beg;
  delete[] c->ev_end;
  delete[] c->ev_cls;
  delete[] c->ev_work;
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  if (c->side_stream) cudaStreamDestroy(c->side_stream);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  for (int k = 0; k < 2; ++k) {
    if (c->ev_staged[k]) cudaEventDestroy(c->ev_staged[k]);
    if (c->ev_used[k]) cudaEventDestroy(c->ev_used[k]);
  }
  delete c;
  return ARMOR_OK;
}

int64_t armor_launch_count(const armor_ctx* c) { return c ? c->launches : -1; }

armor_status armor_kernel_timing_enable(armor_ctx* c, int32_t level) {
  if (!c || level < 0 || level > 2) return ARMOR_ERR_INVALID_ARG;
  if (level && c->ev_created < ARMOR_MAX_TIMED) {
    if (!c->ev_beg) c->ev_beg = new (std::nothrow) cudaEvent_t[ARMOR_MAX_TIMED];
    if (!c->ev_end) c->ev_end = new (std::nothrow) cudaEvent_t[ARMOR_MAX_TIMED];
    if (!c->ev_cls) c->ev_cls = new (std::nothrow) int32_t[ARMOR_MAX_TIMED];
    if (!c->ev_work) c->ev_work = new (std::nothrow) double[ARMOR_MAX_TIMED];
    if (!c->ev_beg || !c->ev_end || !c->ev_cls || !c->ev_work) return ARMOR_ERR_INVALID_ARG;
    // (an earlier call may have stopped part of the way: continue from the pairs that exist)
    for (int i = c->ev_created; i < ARMOR_MAX_TIMED; ++i) {
      if (cudaEventCreate(&c->ev_beg[i]) != cudaSuccess) return ARMOR_ERR_CUDA;
      if (cudaEventCreate(&c->ev_end[i]) != cudaSuccess) { cudaEventDestroy(c->ev_beg[i]); return ARMOR_ERR_CUDA; }
      c->ev_created = i + 1;
    }
  }
  c->timing_on = level;
  return ARMOR_OK;
}

armor_status armor_kernel_timing(armor_ctx* c, int32_t n_classes, int64_t* launches, double* total_ms, double* total_work) {
  if (!c || !launches || !total_ms || !total_work || n_classes < 1) return ARMOR_ERR_INVALID_ARG;
  for (int k = 0; k < n_classes; ++k) { launches[k] = 0; total_ms[k] = 0.0; total_work[k] = 0.0; }
  for (int i = 0; i < c->timing_n; ++i) {
    ARMOR_CUDA_OK(cudaEventSynchronize(c->ev_end[i]));
    float t = 0.f;
    ARMOR_CUDA_OK(cudaEventElapsedTime(&t, c->ev_beg[i], c->ev_end[i]));
    const int k = c->ev_cls[i];
    if (k < 0 || k >= n_classes) continue;
    launches[k] += 1;
    total_ms[k] += (double)t;
    total_work[k] += c->ev_work[i];
  }
  c->timing_n = 0;
  return ARMOR_OK;
}

armor_status armor_use_graphs(armor_ctx* c, int32_t enable) {
  if (!c) return ARMOR_ERR_INVALID_ARG;
  c->use_graphs = enable ? 1 : 0;
  return ARMOR_OK;
}

armor_status armor_fuse_grams(armor_ctx* c, int32_t enable) {
  if (!c) return ARMOR_ERR_INVALID_ARG;
  c->gram_pairs = enable ? 1 : 0;
  return ARMOR_OK;
}

armor_status armor_gemm_timing_enable(armor_ctx* c, int32_t enable) { return armor_kernel_timing_enable(c, enable ? 1 : 0); }

armor_status armor_gemm_timing(armor_ctx* c, int64_t* n_launches, double* total_ms, double* total_flops) {
  if (!c || !n_launches || !total_ms || !total_flops) return ARMOR_ERR_INVALID_ARG;
  return armor_kernel_timing(c, 1, n_launches, total_ms, total_flops);
}

armor_status armor_get_device_status(armor_ctx* c, int32_t* h_codes, int32_t n) {
  if (!c || !h_codes || n < 0) return ARMOR_ERR_INVALID_ARG;
  if (n > ST_COUNT) n = ST_COUNT;
  ARMOR_CUDA_OK(cudaMemcpy(h_codes, c->status, (size_t)n * sizeof(int32_t), cudaMemcpyDeviceToHost));
  return ARMOR_OK;
}

armor_status armor_gram(armor_ctx* c, const void* d_X, int32_t x_dtype, int64_t n_rows, int64_t ldx, float* d_H,
                        armor_stream_t stream) {
  if (!c || !d_H || n_rows < 0) return ARMOR_ERR_INVALID_ARG;
  if (n_rows == 0) return ARMOR_OK;
  if (!d_X || ldx < c->d_in) return ARMOR_ERR_INVALID_ARG;
  if (x_dtype != ARMOR_DTYPE_F32 && x_dtype != ARMOR_DTYPE_BF16) return ARMOR_ERR_UNSUPPORTED;
  return gram_accumulate(c, d_X, x_dtype, n_rows, ldx, d_H, cs(stream));
}

armor_status armor_init(armor_ctx* c, const float* d_W, const float* d_H, float* d_Wbar, float* d_r1, float* d_r2,
                        float* d_A, float* d_B, float* d_S, uint8_t* d_M, armor_stream_t stream) {
  if (!c || !d_W || !d_H || !d_Wbar || !d_A || !d_B || !d_S || !d_M) return ARMOR_ERR_INVALID_ARG;
  if (c->cfg.normalize && (!d_r1 || !d_r2)) return ARMOR_ERR_INVALID_ARG;
  if (launch_screen_inputs(c, d_W, d_H, cs(stream)) != ARMOR_OK) return ARMOR_ERR_CUDA;
  launch_init(c, d_W, d_H, d_Wbar, d_r1, d_r2, d_A, d_B, d_S, d_M, cs(stream));
  if (reset_adam(c, cs(stream)) != ARMOR_OK) return ARMOR_ERR_CUDA;
  return finish_call(c);
}

armor_status armor_proxy_loss(armor_ctx* c, const float* W, const float* H, const float* A, const float* B,
                              const float* S, double* d_loss, armor_stream_t stream) {
  if (!c || !W || !H || !A || !B || !S || !d_loss) return ARMOR_ERR_INVALID_ARG;
  cudaStream_t s = cs(stream);
  armor_status st = prepare_H(c, H, s);
  if (st != ARMOR_OK) return st;
  st = residual_and_loss(c, W, H, A, B, S, d_loss, s);
  if (st != ARMOR_OK) return st;
  return finish_call(c);
}

armor_status armor_bcd_step(armor_ctx* c, const float* W, const float* H, float* A, float* B, float* S, uint8_t* M,
                            int64_t t_first, int32_t n_iters, armor_iter_stats* d_stats, armor_stream_t stream) {
  if (!c || !W || !H || !A || !B || !S || !M || n_iters < 0 || t_first < 0) return ARMOR_ERR_INVALID_ARG;
  cudaStream_t s = cs(stream);
  const int db = c->db, nbo = c->nbo, nbi = c->nbi;
  const int64_t d_out = c->d_out, d_in = c->d_in;
  const int ph = c->cfg.phases;
  if (launch_screen_inputs(c, W, H, s) != ARMOR_OK) return ARMOR_ERR_CUDA;
  armor_status st = prepare_H(c, H, s);
  if (st != ARMOR_OK) return st;
  // W H_w is the same for every iteration of the call: E H_w = W H_w - A (T H_w)
  if (c->cfg.ab_step != ARMOR_AB_ADAM) {
    st = rmul_H(c, W, H, c->WH, d_out, nullptr, nullptr, nullptr, nullptr, s);
    if (st != ARMOR_OK) return st;
  }
  // P = T H_w = S B H_w is formed by a dense product in the first iteration of a call only.  Afterwards it
  // follows the state: the B-step and the S-step each form R H_w for their own direction R (S Delta, resp.
  // Gamma_M B) to get the step length, and P moves by tau R H_w; the group updates add the rows
  // z H_w[block row] that their guard has formed already.  With a diagonal H_w the product is a column
  // scale and P is simply recomputed.
  const bool adam = (c->cfg.ab_step == ARMOR_AB_ADAM);
  const int sweeps = c->cfg.mask_sweeps > 0 ? c->cfg.mask_sweeps : 1;
  const bool carry_P = (c->cfg.h_mode == ARMOR_H_FULL) && !adam;
  if (!adam && c->cfg.ab_step == ARMOR_AB_EXACT && (ph & ARMOR_PHASE_B) && n_iters > 0) {
    st = launch_hjj_inverse(c, s);
    if (st != ARMOR_OK) return st;
  }
  if (adam && t_first == 0 && reset_adam(c, s) != ARMOR_OK) return ARMOR_ERR_CUDA;
  // One iteration, enqueued on stream s.  Which iteration it is reaches the kernels through the device counter
  // c->it_dev (record d_stats[it], selection counter, Adam's step number), so that the same sequence of launches
  // serves every iteration but the first of a call and can be replayed from a CUDA graph.
  //   first:      the first iteration of the call (T H_w is formed by a dense product);
  //   fresh_loss: the loss at the start is evaluated from the residual (first iteration, every LOSS_REFRESH-th, and
  //               always with Adam); otherwise it is the loss the previous iteration ended with, which follows from
  //               the evaluated one by the exact decreases of the quadratic sub-steps;
  //   t_zero:     iteration 0 of the whole run (Adam: exact products, see below).
  armor_iter_stats* const is = d_stats;   // base of the records; the kernels add the device counter
  auto body = [&](bool first, bool fresh_loss, bool t_zero, cudaStream_t s) -> armor_status {
    armor_status st = ARMOR_OK;
    launch_zero_scalars(c, !fresh_loss, is, s);      // with a carried loss this also opens the iteration's record
    if (adam) {
      // Adam normalises every entry's move, so a gradient that is exactly zero (the kept entries of the core at
      // the initialisation, where E vanishes on them) must come out as zero: E H_w is formed from E itself, not
      // as the difference W H_w - A P, and at t = 0 (identity wrappers) with the exact fp32 products
      st = residual_and_loss(c, W, H, A, B, S, c->sc + SC_L0, s, t_zero);
      if (st != ARMOR_OK) return st;
      launch_stage(c, is, 0, nullptr, 0, 0, s);
    } else {
    bd_right(c, S, B, false, c->T, d_out, d_in, 1.f, nullptr, 0.f, s);              // T = S B
    if (first || !carry_P) {
      st = rmul_H(c, c->T, H, c->P, d_out, nullptr, nullptr, nullptr, nullptr, s);   // P = T H_w
      if (st != ARMOR_OK) return st;
    }
    bd_left(c, A, false, c->P, c->EH, d_out, d_in, -1.f, c->WH, 1.f, s);             // E H_w = W H_w - A P
    if (fresh_loss) {
      bd_left(c, A, false, c->T, c->E, d_out, d_in, -1.f, W, 1.f, s);                // E = W - A T
      dot_partials(c, c->EH, c->E, c->wn, c->partials, s);                           // L = <E H_w, E>
      launch_stage(c, is, 0, nullptr, 0, 0, s, c->partials, ARMOR_DOT_BLOCKS, SC_L0);
    }
    }

    if (adam) {
      // ---- joint Adam step on A, B and the core from gradients at one point (Section 3.3.1) --------------
      const int64_t na = (int64_t)nbo * db * db, nbl = (int64_t)nbi * db * db;
      rowblock_grams(c, nullptr, c->EH, c->T, nullptr, c->GamA, s);                  // Gamma^A_i = E_i H_w T_i^T
      bd_left(c, A, false, S, c->U, d_out, d_in, 1.f, nullptr, 0.f, s);              // U = A S
      colblock_grams(c, c->U, nullptr, c->EH, nullptr, c->GamB, s);                  // Gamma^B_j = U_j^T (E H_w)_j
      core_gradient(c, A, B, s);                                                     // Gamma = A^T E H_w B^T
      launch_adam(c, A, c->GamA, c->mA, c->vA, na, nullptr, t_first + 1, s);      // step number: t_first + 1 + counter
      launch_adam(c, B, c->GamB, c->mB, c->vB, nbl, nullptr, t_first + 1, s);
      launch_adam(c, S, c->Gam, c->mS, c->vS, c->wn, M, t_first + 1, s);
      // the new state: residual, E H_w and the loss afresh
      st = residual_and_loss(c, W, H, A, B, S, c->sc + SC_L0, s);
      if (st != ARMOR_OK) return st;
      launch_stage(c, is, 9, nullptr, 0, 0, s);
    }

    // ---- A-step: A_i += Gamma_i (G_i + lam I)^-1 -------------------------------------------
    if (!adam && (ph & ARMOR_PHASE_A)) {
      rowblock_grams(c, c->P, c->EH, c->T, c->G, c->GamA, s);   // G_i = T_i H_w T_i^T, Gamma_i = E_i H_w T_i^T
      if (c->cfg.ab_step == ARMOR_AB_GD) {
        // the paper's gradient step (Algorithm 2): A_i += Gamma_i / (beta_A / 2), beta_A / 2 = sum_ij |T_ij D_j T_ij^T|_F
        // (Eq. lrA; P = T D with the diagonal weighting)
        const int64_t na = (int64_t)nbo * db * db;
        tile_grams(c, c->P, c->T, true, c->V, s);
        launch_block_fro_sum(c, c->V, nbo * nbi, nullptr, c->sc + SC_HB_A, s);
        dot_to_ptr(c, c->GamA, c->GamA, na, c->sc + SC_TMP0, s);                     // |Gamma|^2
        block_mm(c, c->GamA, false, c->G, false, c->dA, nbo, s);                     // Gamma_i G_i
        dot_to_ptr(c, c->dA, c->GamA, na, c->sc + SC_TMP1, s);                       // sum_i <Gamma_i G_i, Gamma_i>
        launch_stage(c, is, 7, nullptr, 0, 0, s);
        if (cudaMemsetAsync(c->dA, 0, (size_t)na * sizeof(float), s) != cudaSuccess) return ARMOR_ERR_CUDA;
        launch_axpy_slot(c, c->dA, c->GamA, na, SC_TAU_A, 1.f, s);                   // dA = tau Gamma
        launch_axpy_slot(c, A, c->GamA, na, SC_TAU_A, 1.f, s);                       // A += tau Gamma
      } else {
        st = launch_chol(c, 0, c->G, c->GamA, c->dA, nullptr, A, nbo, c->partblk, s);
        if (st != ARMOR_OK) return st;
        launch_stage(c, is, 1, c->partblk, nbo * chol_parts_per_block(db, nbo), nbo, s);
      }
      bd_left(c, c->dA, false, c->P, c->EH, d_out, d_in, -1.f, c->EH, 1.f, s);       // EH -= dA P
    } else if (!adam) {
      launch_stage(c, is, 1, nullptr, 0, 0, s);
    }

    // ---- B-step: block-Newton directions, one exact step --------------------------------------
    if (!adam && (ph & ARMOR_PHASE_B)) {
      launch_zero_flags(c, s);
      bd_left(c, A, false, S, c->U, d_out, d_in, 1.f, nullptr, 0.f, s);              // U = A S
      colblock_grams(c, c->U, c->U, c->EH, c->C, c->GamB, s);   // C_j = U_j^T U_j, Gamma_j = U_j^T (E H_w)_j
      const bool b_gd = (c->cfg.ab_step == ARMOR_AB_GD);
      if (b_gd) {
        // the paper's gradient step: the direction is Gamma itself, the step 1 / (beta_B / 2) with
        // beta_B / 2 = sum_ij |U_ij^T U_ij|_F |D_j|_F  (Eq. lrB)
        const int64_t nbl = (int64_t)nbi * db * db;
        if (cudaMemcpyAsync(c->Delta, c->GamB, (size_t)nbl * sizeof(float), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
          return ARMOR_ERR_CUDA;
        tile_grams(c, c->U, c->U, false, c->V, s);
        launch_block_fro_sum(c, c->V, nbo * nbi, c->hdiag, c->sc + SC_HB_B, s);
        dot_to_ptr(c, c->GamB, c->GamB, nbl, c->sc + SC_GD_B, s);                    // <Gamma, Delta>
      } else {
        // Delta_j = (C_j + lam I)^-1 Gamma_j (H_jj + mu I)^-1: a solve with C_j, then a product with the inverse
        // that was formed once for the call (as accurate here as a second solve: both are good to a few 1e-7 on
        // these blocks, and it replaces a latency-bound factorisation by a small product)
        st = launch_chol(c, 1, c->C, c->GamB, c->Ktmp, nullptr, nullptr, nbi, nullptr, s);
        if (st != ARMOR_OK) return st;
        block_mm(c, c->Ktmp, false, c->Hinv, false, c->Delta, nbi, s);
        launch_delta_finish(c, c->Delta, c->GamB, c->partblk, s);                    // part_j = <Gamma_j, Delta_j>
      }
      // direction in B: V = A R with R = S Delta; R H_w serves both V H_w = A (R H_w) and the carried P
      bd_right(c, S, c->Delta, false, c->Tmp, d_out, d_in, 1.f, nullptr, 0.f, s);    // R = S Delta
      st = rmul_H(c, c->Tmp, H, c->E, d_out, nullptr, nullptr, nullptr, nullptr, s); // R H_w
      if (st != ARMOR_OK) return st;
      // V H_w = A (R H_w) and q = <V H_w, V> with V = A R (summed by the stage; V itself is needed nowhere else)
      int nq = 0;
      bd_left_dual(c, A, c->Tmp, c->E, c->V, c->VH, d_out, d_in, c->partials, &nq, s);
      if (b_gd) launch_stage(c, is, 8, nullptr, 0, 0, s, c->partials, nq, SC_Q_B);
      else launch_stage(c, is, 2, c->partblk, nbi, nbi, s, c->partials, nq, SC_Q_B);
      launch_axpy_slot(c, B, c->Delta, (int64_t)nbi * db * db, SC_TAU_B, 1.f, s);    // B += tau Delta
      // EH -= tau V H_w and, where T H_w is carried, P += tau R H_w: one launch
      launch_axpy_multi(c, c->EH, c->VH, -1.f, carry_P ? c->P : nullptr, c->E, 1.f, nullptr, nullptr, 0.f, c->wn, SC_TAU_B, s);
    } else if (!adam) {
      launch_stage(c, is, 2, nullptr, 0, 0, s);
    }

    // ---- S-step: exact line search along Gamma (.) M ------------------------------------------
    if (!adam && (ph & ARMOR_PHASE_S)) {
      core_gradient(c, A, B, s);
      double* nrm_part = c->partials + 8 * c->npart;                                 // kept until the stage below
      launch_masked_copy(c, c->Gam, M, c->U, nrm_part, s);                           // U = Gamma (.) M, |U|^2
      bd_right(c, c->U, B, false, c->Tmp, d_out, d_in, 1.f, nullptr, 0.f, s);        // R = Gamma_M B
      st = rmul_H(c, c->Tmp, H, c->E, d_out, nullptr, nullptr, nullptr, nullptr, s); // R H_w
      if (st != ARMOR_OK) return st;
      // V H_w = A (R H_w) and q = <V H_w, V> with V = A Gamma_M B
      int nq = 0;
      bd_left_dual(c, A, c->Tmp, c->E, c->V, c->VH, d_out, d_in, c->partials, &nq, s);
      const bool beta_step = (c->cfg.s_step == ARMOR_S_BETA);
      if (beta_step) {
        // the paper's step size (Eq. lrWprime): |A^T A|_F and |B H_w B^T|_F  (these dot products reuse the
        // partial-sum buffer, so q is summed first)
        reduce_partials_to(c, c->partials, nq, c->sc + SC_Q_S, s);
        block_mm(c, A, true, A, false, c->G, nbo, s);
        dot_to_ptr(c, c->G, c->G, (int64_t)nbo * db * db, c->sc + SC_BETA_A, s);
        if (c->cfg.h_mode == ARMOR_H_FULL) {
          bd_left(c, B, false, H, c->Hq1, d_in, d_in, 1.f, nullptr, 0.f, s);
          bd_right(c, c->Hq1, B, true, c->Hq2, d_in, d_in, 1.f, nullptr, 0.f, s);
          dot_to_ptr(c, c->Hq2, c->Hq2, d_in * d_in, c->sc + SC_BETA_K, s);
        } else {
          block_mm(c, B, false, c->Hjj, false, c->Ktmp, nbi, s);
          block_mm(c, c->Ktmp, false, B, true, c->Kfull, nbi, s);
          dot_to_ptr(c, c->Kfull, c->Kfull, (int64_t)nbi * db * db, c->sc + SC_BETA_K, s);
        }
      }
      launch_stage(c, is, beta_step ? 6 : 3, nullptr, 0, 0, s, beta_step ? nullptr : c->partials, nq, SC_Q_S,
                   nrm_part, ARMOR_DOT_BLOCKS, SC_NRM_S);
      // S += tau Gamma_M, EH -= tau V H_w and, where T H_w is carried, P += tau R H_w: one launch
      launch_axpy_multi(c, S, c->U, 1.f, c->EH, c->VH, -1.f, carry_P ? c->P : nullptr, c->E, 1.f, c->wn, SC_TAU_S, s);
    } else if (!adam) {
      launch_stage(c, is, 3, nullptr, 0, 0, s);
    }

    // ---- sparse-core update (Algorithm 3), mask_sweeps times ------------------------------------
    if (ph & ARMOR_PHASE_MASK) {
      block_mm(c, B, false, c->Hjj, false, c->Ktmp, nbi, s);                         // B_j H_jj
      launch_mask_prep(c, A, B, c->Ktmp, s);               // alpha_r and the m x m diagonal blocks of K_j = B_j H_jj B_j^T
      for (int sw = 0; sw < sweeps; ++sw) {
        if (sw > 0) {
          // E H_w for the state the previous run left
          if (adam) {
            st = residual_and_loss(c, W, H, A, B, S, c->sc + SC_TMP0, s);
            if (st != ARMOR_OK) return st;
          } else {
            if (carry_P) {
              launch_mask_carry_P(c, c->P, s);                                       // P += dS B H_w (if accepted)
            } else {
              bd_right(c, S, B, false, c->T, d_out, d_in, 1.f, nullptr, 0.f, s);     // T = S B
              st = rmul_H(c, c->T, H, c->P, d_out, nullptr, nullptr, nullptr, nullptr, s);
              if (st != ARMOR_OK) return st;
            }
            bd_left(c, A, false, c->P, c->EH, d_out, d_in, -1.f, c->WH, 1.f, s);     // E H_w = W H_w - A P
          }
        }
        core_gradient(c, A, B, s);
        launch_mask_select(c, c->Gam, S, M, (uint64_t)(t_first * sweeps + sw), (uint64_t)sweeps, s);   // counter (t_first + it) K + k
        launch_mask_quadratic(c, A, B, H, s);
        launch_stage(c, is, 4, c->partblk, nbo * nbi * c->kg, 0, s, c->quadpart, nbo * nbi * c->kg, SC_Q_M);
        launch_mask_commit(c, S, M, is, s);
      }
      if (carry_P) launch_mask_carry_P(c, c->P, s);                                  // P += dS B H_w (if accepted)
    } else {
      launch_stage(c, is, 5, nullptr, 0, 0, s);
    }
    launch_advance_iteration(c, s);
    return ARMOR_OK;
  };

  if (cudaMemsetAsync(c->it_dev, 0, sizeof(int64_t), s) != cudaSuccess) return ARMOR_ERR_CUDA;
  // Iterations other than the first of the call (and the ones that re-evaluate the loss) enqueue the same launches:
  // they are captured once, on a stream of the context's own, and replayed from a CUDA graph on the caller's stream
  // (the gaps between the 50-odd small launches of an iteration are 3 - 4 % of its time otherwise).
  auto is_generic = [&](int it) { return it > 0 && t_first + it != 0 && (adam || it % LOSS_REFRESH != 0); };
  int n_generic = 0;
  for (int it = 0; it < n_iters; ++it) n_generic += is_generic(it) ? 1 : 0;
  // With events around the dense products (timing level 1) the iteration is captured in pieces around them and the
  // products themselves are launched directly; with every launch timed (level 2) nothing is captured.
  bool use_graph = c->use_graphs && c->cap_stream && c->timing_on <= 1 && n_generic >= 3;
  const bool split = c->timing_on == 1 && c->cfg.h_mode == ARMOR_H_FULL;
  if (use_graph) {
    cudaStreamCaptureStatus cst = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cst) != cudaSuccess || cst != cudaStreamCaptureStatusNone) use_graph = false;
  }
  cudaGraphExec_t exec[ARMOR_MAX_PIECES] = {};
  int n_pieces = 0;                 // graph pieces; piece k < n_pieces - 1 is followed by the remembered product k
  int64_t body_launches = 0;
  armor_status result = ARMOR_OK;
  for (int it = 0; it < n_iters && result == ARMOR_OK; ++it) {
    if (use_graph && is_generic(it)) {
      if (n_pieces == 0) {
        const int64_t l0 = c->launches;
        armor_status bst = ARMOR_ERR_CUDA;
        c->cap_n = 0; c->cap_failed = 0;
        for (int k = 0; k < ARMOR_MAX_PIECES; ++k) c->cap_graph[k] = nullptr;
        if (cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
          c->cap_split = split ? 1 : 0;
          bst = body(false, adam, false, c->cap_stream);
          c->cap_split = 0;
          if (cudaStreamEndCapture(c->cap_stream, &c->cap_graph[c->cap_n]) != cudaSuccess || c->cap_failed) bst = ARMOR_ERR_CUDA;
        }
        bool ok = (bst == ARMOR_OK && c->host_err == ARMOR_OK);
        for (int k = 0; ok && k <= c->cap_n; ++k)
          ok = c->cap_graph[k] && cudaGraphInstantiate(&exec[k], c->cap_graph[k], 0) == cudaSuccess;
        if (ok) {
          n_pieces = c->cap_n + 1;
          body_launches = c->launches - l0;
        } else {
          for (int k = 0; k < ARMOR_MAX_PIECES; ++k)
            if (exec[k]) { cudaGraphExecDestroy(exec[k]); exec[k] = nullptr; }
          use_graph = false;              // this call goes on with direct launches
          c->host_err = ARMOR_OK;
          (void)cudaGetLastError();
        }
        for (int k = 0; k < ARMOR_MAX_PIECES; ++k)
          if (c->cap_graph[k]) { cudaGraphDestroy(c->cap_graph[k]); c->cap_graph[k] = nullptr; }
        c->launches = l0;
      }
      if (n_pieces > 0) {
        for (int k = 0; k < n_pieces && result == ARMOR_OK; ++k) {
          if (cudaGraphLaunch(exec[k], s) != cudaSuccess) result = ARMOR_ERR_CUDA;
          if (k + 1 < n_pieces && result == ARMOR_OK) {
            const armor_ctx::RmulCall& r = c->cap_call[k];
            result = rmul_H(c, r.in, r.H, r.out, r.rows, r.d1, r.out1, r.d2, r.out2, s);
          }
        }
        c->launches += body_launches;
        continue;
      }
    }
    result = body(it == 0, adam || (it % LOSS_REFRESH == 0), t_first + it == 0, s);
  }
  for (int k = 0; k < ARMOR_MAX_PIECES; ++k)
    if (exec[k]) cudaGraphExecDestroy(exec[k]);   // a graph still executing is released when it has finished
  if (result != ARMOR_OK) { c->host_err = ARMOR_OK; return result; }
  return finish_call(c);
}

// x -> y = A (S (B x)) in chunks of tokens; `packed` non-null: the core comes packed for the sparse tensor cores
static armor_status apply_impl(armor_ctx* c, const float* A, const float* B, const float* S, const void* packed,
                               const float* r1, const float* r2, const void* d_x, void* d_y, bool bf16, int64_t n_tokens,
                               cudaStream_t s) {
  const size_t esz = bf16 ? 2 : 4;
  const int64_t d_out = c->d_out, d_in = c->d_in;
  const int64_t chunk = d_out < d_in ? d_out : d_in;   // z1 [chunk, d_in] and z2 [chunk, d_out] fit W-shaped scratch
  for (int64_t t0 = 0; t0 < n_tokens; t0 += chunk) {
    const int64_t n = (n_tokens - t0 < chunk) ? n_tokens - t0 : chunk;
    const float* xc;
    float* yc;
    if (bf16) {
      // bf16 activations are widened on the way in and rounded once on the way out; the three products run in
      // the context's precision
      launch_bf16_to_f32(c, static_cast<const char*>(d_x) + (size_t)(t0 * d_in) * esz, r1, c->Tmp, n, d_in, s);
      xc = c->Tmp;
      yc = c->V;
    } else {
      xc = static_cast<const float*>(d_x) + t0 * d_in;
      yc = static_cast<float*>(d_y) + t0 * d_out;
      if (r1) {
        launch_scale_rows_cols(c, xc, r1, nullptr, c->Tmp, n, d_in, s);
        xc = c->Tmp;
      }
    }
    // the bf16 forward rounds z1, S and y to 8 bits: its wrapper products take one tf32 pass (11 bits)
    c->block_one_pass = bf16 ? 1 : 0;
    bd_right(c, xc, B, true, c->T, n, d_in, 1.f, nullptr, 0.f, s);                   // z1 = x B^T
    c->block_one_pass = 0;
    armor_status st = apply_core(c, c->T, S, packed, c->E, n, bf16, s);              // z2 = z1 S^T
    if (st != ARMOR_OK) return st;
    c->block_one_pass = bf16 ? 1 : 0;
    bd_right(c, c->E, A, true, yc, n, d_out, 1.f, nullptr, 0.f, s);                  // y = z2 A^T
    c->block_one_pass = 0;
    if (bf16) launch_f32_to_bf16(c, yc, r2, static_cast<char*>(d_y) + (size_t)(t0 * d_out) * esz, n, d_out, s);
    else if (r2) launch_scale_rows_cols(c, yc, r2, nullptr, yc, n, d_out, s);
  }
  return finish_call(c);
}

armor_status armor_apply(armor_ctx* c, const float* A, const float* B, const float* S, const uint8_t* M,
                         const float* r1, const float* r2, const void* d_x, void* d_y, int32_t xy_dtype,
                         int64_t n_tokens, armor_stream_t stream) {
  if (!c || !A || !B || !S || n_tokens < 0) return ARMOR_ERR_INVALID_ARG;
  if (n_tokens == 0) return ARMOR_OK;
  if (!d_x || !d_y) return ARMOR_ERR_INVALID_ARG;
  if (xy_dtype != ARMOR_DTYPE_F32 && xy_dtype != ARMOR_DTYPE_BF16 && xy_dtype != ARMOR_DTYPE_BF16_SPARSE)
    return ARMOR_ERR_UNSUPPORTED;
  const bool sparse = (xy_dtype == ARMOR_DTYPE_BF16_SPARSE);
  if (sparse && !M) return ARMOR_ERR_INVALID_ARG;
  if (sparse && !tc_sparse_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  if ((r1 == nullptr) != (r2 == nullptr)) return ARMOR_ERR_INVALID_ARG;
  cudaStream_t s = cs(stream);
  const void* packed = nullptr;
  if (sparse) {
    char* buf = reinterpret_cast<char*>(c->P);          // workspace: values wn bytes, positions wn / 8 bytes
    launch_compress_24(c, S, M, buf, buf + tc_sparse_values_bytes(c), s);
    packed = buf;
  }
  return apply_impl(c, A, B, S, packed, r1, r2, d_x, d_y, xy_dtype != ARMOR_DTYPE_F32, n_tokens, s);
}

armor_status armor_packed_core_bytes(const armor_config* cfg, size_t* out_bytes) {
  if (!cfg || !out_bytes) return ARMOR_ERR_INVALID_ARG;
  armor_status st = check_config(cfg);
  if (st != ARMOR_OK) return st;
  if (cfg->n_keep != 2 || cfg->m_group != 4 || cfg->d_out % 128 || cfg->d_in % 128) return ARMOR_ERR_UNSUPPORTED;
  const size_t wn = (size_t)cfg->d_out * (size_t)cfg->d_in;
  *out_bytes = wn + wn / 8;
  return ARMOR_OK;
}

armor_status armor_pack_core(armor_ctx* c, const float* S, const uint8_t* M, void* d_packed, armor_stream_t stream) {
  if (!c || !S || !M || !d_packed) return ARMOR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_packed) % 128) return ARMOR_ERR_INVALID_ARG;
  if (!tc_sparse_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  char* buf = static_cast<char*>(d_packed);
  launch_compress_24(c, S, M, buf, buf + tc_sparse_values_bytes(c), cs(stream));
  return finish_call(c);
}

armor_status armor_apply_packed(armor_ctx* c, const float* A, const float* B, const void* d_packed, const float* r1,
                                const float* r2, const void* d_x, void* d_y, int64_t n_tokens, armor_stream_t stream) {
  if (!c || !A || !B || !d_packed || n_tokens < 0) return ARMOR_ERR_INVALID_ARG;
  if (n_tokens == 0) return ARMOR_OK;
  if (!d_x || !d_y || reinterpret_cast<uintptr_t>(d_packed) % 128) return ARMOR_ERR_INVALID_ARG;
  if (!tc_sparse_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  if ((r1 == nullptr) != (r2 == nullptr)) return ARMOR_ERR_INVALID_ARG;
  return apply_impl(c, A, B, nullptr, d_packed, r1, r2, d_x, d_y, true, n_tokens, cs(stream));
}

// ---- the whole layer packed for the bf16 forward: core values, core positions, B blocks, A blocks -------------
static size_t layer_off_B(const armor_ctx* c) { return (size_t)c->wn + (size_t)c->wn / 8; }
static size_t layer_off_A(const armor_ctx* c) { return layer_off_B(c) + (size_t)c->nbi * c->db * c->db * 2; }

armor_status armor_packed_layer_bytes(const armor_config* cfg, size_t* out_bytes) {
  if (!cfg || !out_bytes) return ARMOR_ERR_INVALID_ARG;
  armor_status st = check_config(cfg);
  if (st != ARMOR_OK) return st;
  if (cfg->n_keep != 2 || cfg->m_group != 4 || cfg->d_out % 128 || cfg->d_in % 128 || cfg->d_block % 128)
    return ARMOR_ERR_UNSUPPORTED;
  const size_t wn = (size_t)cfg->d_out * (size_t)cfg->d_in;
  *out_bytes = wn + wn / 8 + ((size_t)cfg->d_out + (size_t)cfg->d_in) * (size_t)cfg->d_block * 2;
  return ARMOR_OK;
}

armor_status armor_pack_layer(armor_ctx* c, const float* A, const float* B, const float* S, const uint8_t* M,
                              const float* r1, const float* r2, void* d_packed, armor_stream_t stream) {
  if (!c || !A || !B || !S || !M || !d_packed) return ARMOR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_packed) % 128 || (r1 == nullptr) != (r2 == nullptr)) return ARMOR_ERR_INVALID_ARG;
  if (!tc_sparse_ok(c) || !fwd_block_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  cudaStream_t s = cs(stream);
  char* buf = static_cast<char*>(d_packed);
  launch_compress_24(c, S, M, buf, buf + tc_sparse_values_bytes(c), s);
  launch_pack_blocks(c, B, nullptr, r1, buf + layer_off_B(c), c->nbi, s);   // B's columns carry r1
  launch_pack_blocks(c, A, r2, nullptr, buf + layer_off_A(c), c->nbo, s);   // A's rows carry r2
  return finish_call(c);
}

armor_status armor_apply_layer(armor_ctx* c, const void* d_packed, const void* d_x, void* d_y, int64_t n_tokens,
                               armor_stream_t stream) {
  if (!c || !d_packed || n_tokens < 0) return ARMOR_ERR_INVALID_ARG;
  if (n_tokens == 0) return ARMOR_OK;
  if (!d_x || !d_y || reinterpret_cast<uintptr_t>(d_packed) % 128) return ARMOR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_x) % 16 || reinterpret_cast<uintptr_t>(d_y) % 16) return ARMOR_ERR_INVALID_ARG;
  if (!tc_sparse_ok(c) || !fwd_block_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  cudaStream_t s = cs(stream);
  const char* buf = static_cast<const char*>(d_packed);
  const int64_t d_out = c->d_out, d_in = c->d_in;
  const int64_t chunk = d_out < d_in ? d_out : d_in;   // bf16 z1 [chunk, d_in] and z2 [chunk, d_out] fit W-shaped scratch
  for (int64_t t0 = 0; t0 < n_tokens; t0 += chunk) {
    const int64_t n = (n_tokens - t0 < chunk) ? n_tokens - t0 : chunk;
    const char* xc = static_cast<const char*>(d_x) + (size_t)(t0 * d_in) * 2;
    char* yc = static_cast<char*>(d_y) + (size_t)(t0 * d_out) * 2;
    armor_status st = launch_fwd_block(c, xc, buf + layer_off_B(c), c->T, n, d_in, s);        // z1 = (r1 . x) B^T
    if (st != ARMOR_OK) return st;
    st = launch_tc_sparse(c, buf, buf + tc_sparse_values_bytes(c), c->T, c->E, true, n, s);   // z2 = z1 S^T
    if (st != ARMOR_OK) return st;
    st = launch_fwd_block(c, c->E, buf + layer_off_A(c), yc, n, d_out, s);                    // y = r2 . (z2 A^T)
    if (st != ARMOR_OK) return st;
  }
  return finish_call(c);
}

}  // extern "C"
