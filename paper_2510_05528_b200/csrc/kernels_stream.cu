// Streaming (HBM-bound) kernels over W-shaped tensors, reductions and small bookkeeping kernels.
#include <cuda_bf16.h>

#include "armor_internal.cuh"

namespace {

constexpr int NT = 256;

__device__ __forceinline__ double block_reduce_sum(double v) {
  __shared__ double sm[32];
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) sm[w] = v;
  __syncthreads();
  const int nw = (blockDim.x + 31) >> 5;
  v = (threadIdx.x < nw) ? sm[threadIdx.x] : 0.0;
  if (w == 0) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  }
  __syncthreads();
  return v;  // valid in thread 0
}

// ---- deterministic two-stage dot product: fixed grid, fixed order --------------------------------
__global__ void __launch_bounds__(NT) dot_partial_kernel(const float4* __restrict__ x,
                                                         const float4* __restrict__ y, int64_t n4,
                                                         double* __restrict__ part) {
  double acc = 0.0;
  const int64_t stride = (int64_t)gridDim.x * NT;
  // four independent pairs of loads in flight per thread; the order of the additions is fixed by the grid
  for (int64_t i0 = (int64_t)blockIdx.x * NT + threadIdx.x; i0 < n4; i0 += 4 * stride) {
    float4 a[4], b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t i = i0 + u * stride;
      a[u] = b[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i < n4) { a[u] = x[i]; b[u] = y[i]; }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float s = a[u].x * b[u].x;
      s = fmaf(a[u].y, b[u].y, s);
      s = fmaf(a[u].z, b[u].z, s);
      s = fmaf(a[u].w, b[u].w, s);
      acc += (double)s;
    }
  }
  acc = block_reduce_sum(acc);
  if (threadIdx.x == 0) part[blockIdx.x] = acc;
}

__global__ void __launch_bounds__(NT) reduce_final_kernel(const double* __restrict__ part, int n,
                                                          double* __restrict__ out) {
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += NT) acc += part[i];
  acc = block_reduce_sum(acc);
  if (threadIdx.x == 0) *out = acc;
}

// ---- column scale: out = in * diag(h) -----------------------------------------------------------
__global__ void __launch_bounds__(NT) colscale_kernel(const float4* __restrict__ in, const float4* __restrict__ h,
                                                      float4* __restrict__ out, int64_t n4, int cols4) {
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) {
    float4 a = in[i], s = h[i % cols4];
    out[i] = make_float4(a.x * s.x, a.y * s.y, a.z * s.z, a.w * s.w);
  }
}

__global__ void __launch_bounds__(NT) rowcolscale_kernel(const float* __restrict__ in, const float* __restrict__ cs,
                                                         const float* __restrict__ rs, float* __restrict__ out,
                                                         int64_t rows, int64_t cols) {
  const int64_t n = rows * cols;
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n; i += (int64_t)gridDim.x * NT) {
    float v = in[i];
    if (cs) v *= cs[i % cols];
    if (rs) v *= rs[i / cols];
    out[i] = v;
  }
}

// ---- H diagonal and diagonal blocks -------------------------------------------------------------
__global__ void extract_hblocks_kernel(const float* __restrict__ H, float* __restrict__ hdiag,
                                       float* __restrict__ Hjj, int64_t d_in, int db, int diag_only) {
  const int j = blockIdx.x;
  for (int e = threadIdx.x; e < db * db; e += blockDim.x) {
    int a = e / db, b = e % db;
    float v = H[(int64_t)(j * db + a) * d_in + (j * db + b)];
    if (diag_only && a != b) v = 0.f;
    Hjj[(int64_t)j * db * db + e] = v;
    if (a == b) hdiag[j * db + a] = v;
  }
}

// ---- Gamma_M = Gamma (.) M and its squared norm -------------------------------------------------
// One float4 per thread step; a mask byte covers m_group / 4 consecutive float4 (q4 = 1 or 2).
__global__ void __launch_bounds__(NT) masked_copy_kernel(const float4* __restrict__ gam, const uint8_t* __restrict__ M,
                                                         float4* __restrict__ out, int64_t n4, int q4,
                                                         double* __restrict__ part) {
  double acc = 0.0;
  for (int64_t g = (int64_t)blockIdx.x * NT + threadIdx.x; g < n4; g += (int64_t)gridDim.x * NT) {
    float4 v = gam[g];
    const unsigned m = (q4 == 1) ? M[g] : ((unsigned)M[g >> 1] >> (4 * (int)(g & 1)));
    v.x = (m & 1u) ? v.x : 0.f;
    v.y = (m & 2u) ? v.y : 0.f;
    v.z = (m & 4u) ? v.z : 0.f;
    v.w = (m & 8u) ? v.w : 0.f;
    out[g] = v;
    float s = v.x * v.x;
    s = fmaf(v.y, v.y, s);
    s = fmaf(v.z, v.z, s);
    s = fmaf(v.w, v.w, s);
    acc += (double)s;
  }
  acc = block_reduce_sum(acc);
  if (threadIdx.x == 0) part[blockIdx.x] = acc;
}

// ---- y += sign * sc[slot] * x -------------------------------------------------------------------
__global__ void __launch_bounds__(NT) axpy_slot_kernel(float4* __restrict__ y, const float4* __restrict__ x,
                                                       int64_t n4, const double* __restrict__ sc, int slot,
                                                       float sign) {
  const float a = sign * (float)sc[slot];
  if (a == 0.f) return;                 // a zero step (also what withheld updates look like): y stays bit for bit
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) {
    float4 u = y[i], v = x[i];
    y[i] = make_float4(fmaf(a, v.x, u.x), fmaf(a, v.y, u.y), fmaf(a, v.z, u.z), fmaf(a, v.w, u.w));
  }
}

// the same for up to three arrays of one length that move by the same step: one launch
struct AxpyTerm { float4* y; const float4* x; float sign; };
__global__ void __launch_bounds__(NT) axpy_multi_slot_kernel(AxpyTerm t0, AxpyTerm t1, AxpyTerm t2, int n_terms, int64_t n4,
                                                             const double* __restrict__ sc, int slot) {
  const float a = (float)sc[slot];
  if (a == 0.f) return;
  const AxpyTerm t[3] = {t0, t1, t2};
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) {
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      if (k >= n_terms) break;
      const float ak = t[k].sign * a;
      const float4 u = t[k].y[i], v = t[k].x[i];
      t[k].y[i] = make_float4(fmaf(ak, v.x, u.x), fmaf(ak, v.y, u.y), fmaf(ak, v.z, u.z), fmaf(ak, v.w, u.w));
    }
  }
}

// ---- normalisation (Section 3.2): r1 = column norms, r2 = row norms of W / r1 -------------------
constexpr int COLSUM_CHUNKS = 64;
__global__ void __launch_bounds__(NT) colsumsq_partial_kernel(const float* __restrict__ W, int64_t rows, int64_t cols,
                                                              double* __restrict__ part) {
  const int64_t col = (int64_t)blockIdx.x * NT + threadIdx.x;
  if (col >= cols) return;
  const int64_t per = (rows + COLSUM_CHUNKS - 1) / COLSUM_CHUNKS;
  const int64_t r0 = blockIdx.y * per, r1 = min(rows, r0 + per);
  double acc = 0.0;
  for (int64_t r = r0; r < r1; ++r) {
    double w = W[r * cols + col];
    acc += w * w;
  }
  part[(int64_t)blockIdx.y * cols + col] = acc;
}
__global__ void __launch_bounds__(NT) colnorm_final_kernel(const double* __restrict__ part, int64_t cols,
                                                           float* __restrict__ r1) {
  const int64_t col = (int64_t)blockIdx.x * NT + threadIdx.x;
  if (col >= cols) return;
  double acc = 0.0;
  for (int ch = 0; ch < COLSUM_CHUNKS; ++ch) acc += part[(int64_t)ch * cols + col];
  float r = (float)sqrt(acc);
  r1[col] = (r == 0.f) ? 1.f : r;
}
__global__ void __launch_bounds__(NT) rownorm_scale_kernel(const float* __restrict__ W, const float* __restrict__ r1,
                                                           float* __restrict__ r2, float* __restrict__ Wbar,
                                                           int64_t cols) {
  const int64_t row = blockIdx.x;
  const float* w = W + row * cols;
  double acc = 0.0;
  for (int64_t c = threadIdx.x; c < cols; c += NT) {
    double v = (double)w[c] / (double)r1[c];
    acc += v * v;
  }
  __shared__ float r2s;
  acc = block_reduce_sum(acc);
  if (threadIdx.x == 0) {
    float r = (float)sqrt(acc);
    r = (r == 0.f) ? 1.f : r;
    r2[row] = r;
    r2s = r;
  }
  __syncthreads();
  const float rr = r2s;
  for (int64_t c = threadIdx.x; c < cols; c += NT) Wbar[row * cols + c] = (w[c] / r1[c]) / rr;
}

// ---- initialisation (Eq. init): top-n_keep of each group of MG by W^2 * H_jj ---------------------
// Position p is kept iff fewer than n_keep positions beat it; q beats p if its score is larger, or equal
// with q < p (ties keep the lower column).
template <int MG>
__global__ void __launch_bounds__(NT) init_core_kernel(const float* __restrict__ W, const float* __restrict__ H,
                                                       int64_t d_in, float* __restrict__ S, uint8_t* __restrict__ M,
                                                       int64_t ngroups, int groups_per_row, int n_keep) {
  for (int64_t g = (int64_t)blockIdx.x * NT + threadIdx.x; g < ngroups; g += (int64_t)gridDim.x * NT) {
    const int64_t c0 = (g % groups_per_row) * MG;
    float wv[MG];
#pragma unroll
    for (int h = 0; h < MG / 4; ++h) {
      const float4 w = *reinterpret_cast<const float4*>(W + g * MG + 4 * h);
      wv[4 * h] = w.x; wv[4 * h + 1] = w.y; wv[4 * h + 2] = w.z; wv[4 * h + 3] = w.w;
    }
    double sc[MG];
#pragma unroll
    for (int p = 0; p < MG; ++p) {
      const double h = (double)H[(c0 + p) * d_in + (c0 + p)];
      sc[p] = (double)wv[p] * (double)wv[p] * h;
    }
    unsigned m = 0;
#pragma unroll
    for (int p = 0; p < MG; ++p) {
      int beaten = 0;
#pragma unroll
      for (int q = 0; q < MG; ++q) beaten += (q != p) && (sc[q] > sc[p] || (sc[q] == sc[p] && q < p));
      if (beaten < n_keep) m |= 1u << p;
    }
    M[g] = (uint8_t)m;
#pragma unroll
    for (int h = 0; h < MG / 4; ++h)
      *reinterpret_cast<float4*>(S + g * MG + 4 * h) =
          make_float4((m >> (4 * h) & 1u) ? wv[4 * h] : 0.f, (m >> (4 * h + 1) & 1u) ? wv[4 * h + 1] : 0.f,
                      (m >> (4 * h + 2) & 1u) ? wv[4 * h + 2] : 0.f, (m >> (4 * h + 3) & 1u) ? wv[4 * h + 3] : 0.f);
  }
}

__global__ void identity_blocks_kernel(float* __restrict__ A, int db) {
  const int64_t off = (int64_t)blockIdx.x * db * db;
  for (int e = threadIdx.x; e < db * db; e += blockDim.x) A[off + e] = (e / db == e % db) ? 1.f : 0.f;
}

__global__ void copy_kernel(const float4* __restrict__ in, float4* __restrict__ out, int64_t n4) {
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) out[i] = in[i];
}

// ---- scalars and per-iteration bookkeeping ------------------------------------------------------
__device__ __forceinline__ void start_record(armor_iter_stats* st, double loss) {
  st->loss_start = loss;
  st->chol_failed = 0;
  st->groups_changed = 0;
  st->mask_accepted = 0;
  st->delta_L_mask = 0.0;
  st->tau_B = 0.f;
  st->tau_S = 0.f;
  st->reserved = 0;
}

// carry_loss: the running loss of the previous iteration becomes this iteration's starting loss, and the
// iteration's record is opened here (no loss evaluation follows)
__global__ void zero_scalars_kernel(double* sc, int32_t* failflag, int nflag, int carry_loss, armor_iter_stats* st_base,
                                    const int64_t* __restrict__ it_dev) {
  armor_iter_stats* st = st_base ? st_base + *it_dev : nullptr;
  const double carried = sc[SC_LOSS];
  __syncthreads();
  for (int i = threadIdx.x; i < SC_COUNT; i += blockDim.x)
    sc[i] = (carry_loss && (i == SC_L0 || i == SC_LOSS)) ? carried : 0.0;
  for (int i = threadIdx.x; i < nflag; i += blockDim.x) failflag[i] = 0;
  if (carry_loss && st && threadIdx.x == 0) start_record(st, carried);
}

// Fixed-order sums by the CTA of the bookkeeping kernel (STAGE_NT threads): thread t adds entries t, t + STAGE_NT, ...
// (eight loads in flight), a shuffle tree per warp, then the warps in order.  All threads get the sum.  The line
// searches hand over thousands of partial sums (four or eight per tile); one warp took 14 us over them.
constexpr int STAGE_NT = 256;
__device__ __forceinline__ double stage_sum_f64(const double* __restrict__ p, int n, double* scratch) {
  double v = 0.0;
  int i = threadIdx.x;
  for (; i + 7 * STAGE_NT < n; i += 8 * STAGE_NT) {
    double t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) t[u] = p[i + STAGE_NT * u];
#pragma unroll
    for (int u = 0; u < 8; ++u) v += t[u];
  }
  for (; i < n; i += STAGE_NT) v += p[i];
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < STAGE_NT / 32; ++w) t += scratch[w];
  __syncthreads();
  return t;
}
__device__ __forceinline__ int stage_count_flags(const int32_t* __restrict__ f, int n, double* scratch) {
  int v = 0;
  for (int i = threadIdx.x; i < n; i += STAGE_NT) v += f[i] ? 1 : 0;
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = (double)v;
  __syncthreads();
  int t = 0;
  for (int w = 0; w < STAGE_NT / 32; ++w) t += (int)scratch[w];
  __syncthreads();
  return t;
}

// stage 0: start, 1: after A, 2: after B, 3 / 6: after S, 4: mask accept, 5: mask phase off.  One CTA of STAGE_NT threads.
// Up to two arrays of partial sums (p1, p2) are first added, in a fixed order, into the scalars slot1 / slot2: the
// reductions of the dot products that precede the stage need no launch of their own.
__global__ void advance_iteration_kernel(int64_t* it_dev) { *it_dev += 1; }

__global__ void stage_kernel(double* sc, armor_iter_stats* st_base, const int64_t* __restrict__ it_dev, int stage,
                             const int32_t* failflag, int nflag,
                             const double* partA, int nA, int32_t* status, const double* p1, int n1, int slot1,
                             const double* p2, int n2, int slot2) {
  armor_iter_stats* st = st_base ? st_base + *it_dev : nullptr;
  __shared__ double scratch[STAGE_NT / 32];
  if (p1) { const double v = stage_sum_f64(p1, n1, scratch); if (threadIdx.x == 0) sc[slot1] = v; }
  if (p2) { const double v = stage_sum_f64(p2, n2, scratch); if (threadIdx.x == 0) sc[slot2] = v; }
  double psum = 0.0;
  int nf = 0;
  if (stage == 1 || stage == 2 || stage == 4) psum = stage_sum_f64(partA, nA, scratch);
  if (stage == 1 || stage == 2) nf = stage_count_flags(failflag, nflag, scratch);
  if (threadIdx.x != 0) return;
  const bool poisoned = status[ST_POISON] != 0;   // unusable inputs: every step length is zero, nothing is accepted
  if (stage == 0) {
    sc[SC_LOSS] = sc[SC_L0];
    if (st) start_record(st, sc[SC_L0]);
  } else if (stage == 1) {
    sc[SC_DEC_A] = psum;
    sc[SC_LOSS] -= psum;
    if (st) { st->loss_A = sc[SC_LOSS]; st->chol_failed += nf; }
    if (nf) atomicAdd(&status[ST_CHOL_FAILS], nf);
  } else if (stage == 2) {
    const double gd = psum;
    sc[SC_GD_B] = gd;
    const double q = sc[SC_Q_B];
    const double tau = (q > 0.0 && !poisoned) ? gd / q : 0.0;
    sc[SC_TAU_B] = tau;
    sc[SC_LOSS] -= 2.0 * tau * gd - tau * tau * q;
    if (st) { st->loss_B = sc[SC_LOSS]; st->tau_B = (float)tau; st->chol_failed += nf; }
    if (nf) atomicAdd(&status[ST_CHOL_FAILS], nf);
  } else if (stage == 3 || stage == 6) {
    const double nrm = sc[SC_NRM_S], q = sc[SC_Q_S];
    double tau = (q > 0.0) ? nrm / q : 0.0;
    if (stage == 6) {  // the paper's step 1 / beta_W' (Eq. lrWprime): the move is Gamma_M / (|A^T A|_F |B H_w B^T|_F)
      const double bh = sqrt(sc[SC_BETA_A]) * sqrt(sc[SC_BETA_K]);
      tau = (bh > 0.0) ? 1.0 / bh : 0.0;
    }
    if (poisoned) tau = 0.0;
    sc[SC_TAU_S] = tau;
    sc[SC_LOSS] -= 2.0 * tau * nrm - tau * tau * q;
    if (st) { st->loss_S = sc[SC_LOSS]; st->tau_S = (float)tau; }
  } else if (stage == 4) {
    sc[SC_EHV_M] = psum;   // <Gamma, dS> = <E H_w, V>, one term per block
    const double dl = -2.0 * sc[SC_EHV_M] + sc[SC_Q_M];
    const bool acc = (dl <= 0.0) && !poisoned;
    sc[SC_DL_M] = dl;
    sc[SC_ACCEPT] = acc ? 1.0 : 0.0;
    if (acc) sc[SC_LOSS] += dl;
    if (st) { st->delta_L_mask += dl; st->mask_accepted += acc ? 1 : 0; st->loss_mask = sc[SC_LOSS]; }   // summed over the sweeps
  } else if (stage == 7) {   // A gradient step with the step of Eq. lrA: tau = 1 / (beta_A / 2)
    const double hb = sc[SC_HB_A], nrm = sc[SC_TMP0], q = sc[SC_TMP1];
    const double tau = (hb > 0.0 && !poisoned) ? 1.0 / hb : 0.0;
    sc[SC_TAU_A] = tau;
    sc[SC_DEC_A] = 2.0 * tau * nrm - tau * tau * q;   // exact decrease of the quadratic in A along Gamma
    sc[SC_LOSS] -= sc[SC_DEC_A];
    if (st) st->loss_A = sc[SC_LOSS];
  } else if (stage == 8) {   // B gradient step with the step of Eq. lrB
    const double hb = sc[SC_HB_B], gd = sc[SC_GD_B], q = sc[SC_Q_B];
    const double tau = (hb > 0.0 && !poisoned) ? 1.0 / hb : 0.0;
    sc[SC_TAU_B] = tau;
    sc[SC_LOSS] -= 2.0 * tau * gd - tau * tau * q;
    if (st) { st->loss_B = sc[SC_LOSS]; st->tau_B = (float)tau; }
  } else if (stage == 9) {   // joint Adam step: the loss was evaluated afresh from the new state
    sc[SC_LOSS] = sc[SC_L0];
    if (st) st->loss_A = st->loss_B = st->loss_S = sc[SC_LOSS];
  } else if (stage == 5) {  // sparse-core update switched off: nothing was evaluated, nothing accepted
    sc[SC_ACCEPT] = 0.0;
    sc[SC_DL_M] = 0.0;
    if (st) st->loss_mask = sc[SC_LOSS];
  }
}

// ---- input screening -----------------------------------------------------------------------------
__device__ __forceinline__ int bad4(const float4 v) {
  return (isfinite(v.x) ? 0 : 1) + (isfinite(v.y) ? 0 : 1) + (isfinite(v.z) ? 0 : 1) + (isfinite(v.w) ? 0 : 1);
}
__global__ void __launch_bounds__(NT) screen_count_kernel(const float4* __restrict__ W, int64_t wn4,
                                                          const float4* __restrict__ H, int64_t hn4,
                                                          const float* __restrict__ Hs, int64_t d_in,
                                                          int32_t* __restrict__ scr) {
  int bw = 0, bh = 0, neg = 0, zero = 0;
  const int64_t stride = (int64_t)gridDim.x * NT, i0 = (int64_t)blockIdx.x * NT + threadIdx.x;
  for (int64_t i = i0; i < wn4; i += stride) bw += bad4(W[i]);
  for (int64_t i = i0; i < hn4; i += stride) bh += bad4(H[i]);
  for (int64_t i = i0; i < d_in; i += stride) {
    const float d = Hs[i * d_in + i];
    neg += (d < 0.f) ? 1 : 0;
    zero += (d == 0.f) ? 1 : 0;
  }
  for (int o = 16; o > 0; o >>= 1) {
    bw += __shfl_xor_sync(0xffffffffu, bw, o); bh += __shfl_xor_sync(0xffffffffu, bh, o);
    neg += __shfl_xor_sync(0xffffffffu, neg, o); zero += __shfl_xor_sync(0xffffffffu, zero, o);
  }
  if ((threadIdx.x & 31) == 0) {        // integer sums: the order does not matter
    if (bw) atomicAdd(&scr[0], bw);
    if (bh) atomicAdd(&scr[1], bh);
    if (neg) atomicAdd(&scr[2], neg);
    if (zero) atomicAdd(&scr[3], zero);
  }
}
__global__ void screen_final_kernel(const int32_t* __restrict__ scr, int32_t* __restrict__ status) {
  status[ST_NONFINITE_W] += scr[0];
  status[ST_NONFINITE_H] += scr[1];
  status[ST_NEG_DIAG_H] += scr[2];
  status[ST_DEAD_CHANNELS] = scr[3];
  const bool bad = scr[0] || scr[1] || scr[2];
  status[ST_POISON] = bad ? 1 : 0;
  if (bad) status[ST_LAST_ERR] = ARMOR_ERR_INVALID_ARG;
}

// ---- operand split for the three-pass tensor-core mode ------------------------------------------
__global__ void __launch_bounds__(NT) split_hilo_kernel(const float4* __restrict__ in, float4* __restrict__ hi,
                                                        float4* __restrict__ lo, int64_t n4) {
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) {
    float4 v = in[i];
    float4 h;
    h.x = __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
    h.y = __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
    h.z = __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
    h.w = __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
    if (hi) hi[i] = h;
    lo[i] = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
  }
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// X [rows, cols] (ld ldx) -> Thi/Tlo [cols, rows] (ld ldt): transposed and split.  bf16 input is exact in
// tf32, so its low part is zero and Tlo is not needed.
template <typename TIn>
__global__ void transpose_split_kernel(const TIn* __restrict__ X, int64_t ldx, int64_t rows, int64_t cols,
                                       float* __restrict__ Thi, float* __restrict__ Tlo, int64_t ldt) {
  __shared__ float tile[32][33];
  const int64_t c0 = (int64_t)blockIdx.x * 32, r0 = (int64_t)blockIdx.y * 32;
  for (int j = threadIdx.y; j < 32; j += blockDim.y) {
    int64_t r = r0 + j, cidx = c0 + threadIdx.x;
    tile[j][threadIdx.x] = (r < rows && cidx < cols) ? to_f32(X[r * ldx + cidx]) : 0.f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += blockDim.y) {
    int64_t cidx = c0 + j, r = r0 + threadIdx.x;
    if (cidx < cols && r < ldt) {
      float v = tile[threadIdx.x][j];
      float h = __uint_as_float(__float_as_uint(v) & 0xffffe000u);
      Thi[cidx * ldt + r] = h;
      if (Tlo) Tlo[cidx * ldt + r] = v - h;
    }
  }
}

// bf16 <-> fp32 with an optional per-column scale (the denormalisation of the deployment form)
__global__ void __launch_bounds__(NT) bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ in,
                                                         const float* __restrict__ cs, float* __restrict__ out,
                                                         int64_t n, int64_t cols) {
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n; i += (int64_t)gridDim.x * NT) {
    float v = __bfloat162float(in[i]);
    if (cs) v *= cs[i % cols];
    out[i] = v;
  }
}
__global__ void __launch_bounds__(NT) f32_to_bf16_kernel(const float* __restrict__ in, const float* __restrict__ cs,
                                                         __nv_bfloat16* __restrict__ out, int64_t n, int64_t cols) {
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n; i += (int64_t)gridDim.x * NT) {
    float v = in[i];
    if (cs) v *= cs[i % cols];
    out[i] = __float2bfloat16_rn(v);
  }
}

// H[r][c] = H[c][r] for c > r: the upper triangle from the lower one, 32 x 32 tiles through shared memory
__global__ void mirror_lower_kernel(float* __restrict__ H, int64_t n) {
  if (blockIdx.x < blockIdx.y) return;   // blockIdx.x: tile column of the destination, blockIdx.y: its tile row
  __shared__ float tile[32][33];
  const int64_t c0 = (int64_t)blockIdx.x * 32, r0 = (int64_t)blockIdx.y * 32;
  // source tile: rows c0.., columns r0..
  for (int j = threadIdx.y; j < 32; j += blockDim.y) {
    const int64_t sr = c0 + j, sc = r0 + threadIdx.x;
    tile[j][threadIdx.x] = (sr < n && sc < n) ? H[sr * n + sc] : 0.f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += blockDim.y) {
    const int64_t dr = r0 + j, dc = c0 + threadIdx.x;
    if (dr < n && dc < n && dc > dr) H[dr * n + dc] = tile[threadIdx.x][j];
  }
}

// part[b] = weight * || X_b ||_F for block b of db x db floats (the terms of beta_A and beta_B, Eq. lrA / lrB)
__global__ void __launch_bounds__(NT) block_fro_kernel(const float4* __restrict__ X, int n4_per_block,
                                                       const float* __restrict__ hdiag, int db, int nbi,
                                                       double* __restrict__ part) {
  const float4* xb = X + (int64_t)blockIdx.x * n4_per_block;
  double acc = 0.0;
  for (int i = threadIdx.x; i < n4_per_block; i += NT) {
    const float4 v = xb[i];
    float s = v.x * v.x;
    s = fmaf(v.y, v.y, s);
    s = fmaf(v.z, v.z, s);
    s = fmaf(v.w, v.w, s);
    acc += (double)s;
  }
  acc = block_reduce_sum(acc);
  double wsum = 0.0;
  if (hdiag) {
    const float* h = hdiag + (int64_t)(blockIdx.x % nbi) * db;
    for (int k = threadIdx.x; k < db; k += NT) wsum += (double)h[k] * (double)h[k];
    wsum = block_reduce_sum(wsum);
  }
  if (threadIdx.x == 0) part[blockIdx.x] = sqrt(acc) * (hdiag ? sqrt(wsum) : 1.0);
}

// ---- Adam (Kingma & Ba, Algorithm 1, with bias correction) ----------------------------------------------
__global__ void __launch_bounds__(NT) adam_kernel(float4* __restrict__ theta, const float4* __restrict__ gamma,
                                                  float4* __restrict__ m, float4* __restrict__ v, int64_t n4,
                                                  const uint8_t* __restrict__ M, int q4, float lr, float b1, float b2,
                                                  float eps, int64_t step_base, const int64_t* __restrict__ it_dev,
                                                  const int32_t* __restrict__ status) {
  if (status[ST_POISON] != 0) return;   // unusable inputs: parameters and moments stay as they are
  // bias corrections 1 / (1 - beta^step), step = step_base + the iteration counter: once per block
  __shared__ float s_bc[2];
  if (threadIdx.x == 0) {
    const double step = (double)(step_base + *it_dev);
    s_bc[0] = (float)(1.0 / (1.0 - pow((double)b1, step)));
    s_bc[1] = (float)(1.0 / (1.0 - pow((double)b2, step)));
  }
  __syncthreads();
  const float inv_bc1 = s_bc[0], inv_bc2 = s_bc[1];
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) {
    const float4 ga = gamma[i];
    float4 mm = m[i], vv = v[i], th = theta[i];
    unsigned keep = 0xFu;
    if (M) keep = (q4 == 1) ? M[i] : ((unsigned)M[i >> 1] >> (4 * (int)(i & 1)));
    const float g[4] = {-2.f * ga.x, -2.f * ga.y, -2.f * ga.z, -2.f * ga.w};
    float mo[4] = {mm.x, mm.y, mm.z, mm.w}, vo[4] = {vv.x, vv.y, vv.z, vv.w}, t[4] = {th.x, th.y, th.z, th.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float gk = ((keep >> k) & 1u) ? g[k] : 0.f;      // the core's gradient is masked
      mo[k] = fmaf(b1, mo[k], (1.f - b1) * gk);
      vo[k] = fmaf(b2, vo[k], (1.f - b2) * gk * gk);
      const float upd = lr * (mo[k] * inv_bc1) / (sqrtf(vo[k] * inv_bc2) + eps);
      t[k] = ((keep >> k) & 1u) ? t[k] - upd : 0.f;
    }
    m[i] = make_float4(mo[0], mo[1], mo[2], mo[3]);
    v[i] = make_float4(vo[0], vo[1], vo[2], vo[3]);
    theta[i] = make_float4(t[0], t[1], t[2], t[3]);
  }
}

inline int grid_for(int64_t n) {
  int64_t b = (n + NT - 1) / NT;
  return (int)(b < 1 ? 1 : (b > 148 * 16 ? 148 * 16 : b));
}

}  // namespace

void dot_to_ptr(armor_ctx* c, const float* x, const float* y, int64_t n, double* out, cudaStream_t s) {
  KTimer kt(c, n >= (1 << 22) ? ARMOR_KC_DOT : ARMOR_KC_SMALL, 8.0 * (double)n, s);
  dot_partial_kernel<<<ARMOR_DOT_BLOCKS, NT, 0, s>>>((const float4*)x, (const float4*)y, n / 4, c->partials);
  reduce_final_kernel<<<1, NT, 0, s>>>(c->partials, ARMOR_DOT_BLOCKS, out);
  c->launches += 2;
}

// partial sums of <x, y> only (ARMOR_DOT_BLOCKS entries at `part`); the consumer adds them up
void dot_partials(armor_ctx* c, const float* x, const float* y, int64_t n, double* part, cudaStream_t s) {
  KTimer kt(c, n >= (1 << 22) ? ARMOR_KC_DOT : ARMOR_KC_SMALL, 8.0 * (double)n, s);
  dot_partial_kernel<<<ARMOR_DOT_BLOCKS, NT, 0, s>>>((const float4*)x, (const float4*)y, n / 4, part);
  c->launches++;
}

void reduce_partials_to(armor_ctx* c, const double* part, int n, double* out, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  reduce_final_kernel<<<1, NT, 0, s>>>(part, n, out);
  c->launches++;
}

void launch_zero_flags(armor_ctx* c, cudaStream_t s) {
  const int nflag = c->nbo > c->nbi ? c->nbo : c->nbi;
  cudaMemsetAsync(c->failflag, 0, (size_t)nflag * sizeof(int32_t), s);
}

void launch_colscale(armor_ctx* c, const float* in, const float* h, float* out, int64_t rows, int64_t cols,
                     cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_AXPY, 8.0 * (double)rows * (double)cols, s);
  colscale_kernel<<<grid_for(rows * cols / 4), NT, 0, s>>>((const float4*)in, (const float4*)h, (float4*)out,
                                                          rows * cols / 4, (int)(cols / 4));
  c->launches++;
}

void launch_scale_rows_cols(armor_ctx* c, const float* in, const float* colscale, const float* rowscale, float* out,
                            int64_t rows, int64_t cols, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_FORWARD, 8.0 * (double)rows * (double)cols, s);
  rowcolscale_kernel<<<grid_for(rows * cols), NT, 0, s>>>(in, colscale, rowscale, out, rows, cols);
  c->launches++;
}

void launch_extract_hblocks(armor_ctx* c, const float* H, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  extract_hblocks_kernel<<<c->nbi, NT, 0, s>>>(H, c->hdiag, c->Hjj, c->d_in, c->db, c->cfg.h_mode == ARMOR_H_DIAG);
  c->launches++;
}

void launch_masked_copy(armor_ctx* c, const float* Gam, const uint8_t* M, float* out, double* part, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_MASKED_COPY, (8.0 + 1.0 / c->cfg.m_group) * (double)c->wn, s);
  masked_copy_kernel<<<ARMOR_DOT_BLOCKS, NT, 0, s>>>((const float4*)Gam, M, (float4*)out, c->wn / 4,
                                                    c->cfg.m_group / 4, part);
  c->launches++;
}

void launch_axpy_slot(armor_ctx* c, float* y, const float* x, int64_t n, int slot, float sign, cudaStream_t s) {
  KTimer kt(c, n >= (1 << 22) ? ARMOR_KC_AXPY : ARMOR_KC_SMALL, 12.0 * (double)n, s);
  axpy_slot_kernel<<<grid_for(n / 4), NT, 0, s>>>((float4*)y, (const float4*)x, n / 4, c->sc, slot, sign);
  c->launches++;
}

// y_k += sign_k * sc[slot] * x_k for up to three pairs of length n (a pair with y == nullptr is skipped)
void launch_axpy_multi(armor_ctx* c, float* y0, const float* x0, float s0, float* y1, const float* x1, float s1, float* y2,
                       const float* x2, float s2, int64_t n, int slot, cudaStream_t s) {
  AxpyTerm t[3];
  int k = 0;
  if (y0) t[k++] = {(float4*)y0, (const float4*)x0, s0};
  if (y1) t[k++] = {(float4*)y1, (const float4*)x1, s1};
  if (y2) t[k++] = {(float4*)y2, (const float4*)x2, s2};
  if (k == 0) return;
  for (int j = k; j < 3; ++j) t[j] = t[0];
  KTimer kt(c, n >= (1 << 22) ? ARMOR_KC_AXPY : ARMOR_KC_SMALL, 12.0 * (double)n * k, s);
  axpy_multi_slot_kernel<<<grid_for(n / 4), NT, 0, s>>>(t[0], t[1], t[2], k, n / 4, c->sc, slot);
  c->launches++;
}

void launch_init(armor_ctx* c, const float* W, const float* H, float* Wbar, float* r1, float* r2, float* A, float* B,
                 float* S, uint8_t* M, cudaStream_t s) {
  const int64_t rows = c->d_out, cols = c->d_in;
  // W read (twice more with the normalisation), Wbar, S and the mask bytes written
  KTimer kt(c, ARMOR_KC_INIT, (double)c->wn * (c->cfg.normalize ? 20.0 : 12.0 + (Wbar != W ? 4.0 : 0.0)) +
                                  (double)c->wn / c->cfg.m_group, s);
  if (c->cfg.normalize) {
    double* part = c->colpart;
    dim3 g1((unsigned)((cols + NT - 1) / NT), COLSUM_CHUNKS);
    colsumsq_partial_kernel<<<g1, NT, 0, s>>>(W, rows, cols, part);
    colnorm_final_kernel<<<(unsigned)((cols + NT - 1) / NT), NT, 0, s>>>(part, cols, r1);
    rownorm_scale_kernel<<<(unsigned)rows, NT, 0, s>>>(W, r1, r2, Wbar, cols);
    c->launches += 3;
  } else if (Wbar != W) {
    copy_kernel<<<grid_for(c->wn / 4), NT, 0, s>>>((const float4*)W, (float4*)Wbar, c->wn / 4);
    c->launches++;
  }
  const int mg = c->cfg.m_group;
  if (mg == 8)
    init_core_kernel<8><<<grid_for(c->wn / 8), NT, 0, s>>>(Wbar, H, cols, S, M, c->wn / 8, (int)(cols / 8),
                                                          c->cfg.n_keep);
  else
    init_core_kernel<4><<<grid_for(c->wn / 4), NT, 0, s>>>(Wbar, H, cols, S, M, c->wn / 4, (int)(cols / 4),
                                                          c->cfg.n_keep);
  identity_blocks_kernel<<<c->nbo, NT, 0, s>>>(A, c->db);
  identity_blocks_kernel<<<c->nbi, NT, 0, s>>>(B, c->db);
  c->launches += 3;
}

armor_status launch_screen_inputs(armor_ctx* c, const float* W, const float* H, cudaStream_t s) {
  if (cudaMemsetAsync(c->screen, 0, 4 * sizeof(int32_t), s) != cudaSuccess) return ARMOR_ERR_CUDA;
  const int64_t wn4 = c->wn / 4, hn4 = c->d_in * c->d_in / 4;
  KTimer kt(c, ARMOR_KC_INIT, 4.0 * ((double)c->wn + (double)c->d_in * (double)c->d_in), s);
  screen_count_kernel<<<grid_for(wn4 > hn4 ? wn4 : hn4), NT, 0, s>>>(reinterpret_cast<const float4*>(W), wn4,
                                                                     reinterpret_cast<const float4*>(H), hn4, H, c->d_in,
                                                                     c->screen);
  screen_final_kernel<<<1, 1, 0, s>>>(c->screen, c->status);
  c->launches += 2;
  return ARMOR_OK;
}

void launch_zero_scalars(armor_ctx* c, bool carry_loss, armor_iter_stats* st, cudaStream_t s) {
  const int nflag = c->nbo > c->nbi ? c->nbo : c->nbi;
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  zero_scalars_kernel<<<1, NT, 0, s>>>(c->sc, c->failflag, nflag, carry_loss ? 1 : 0, st, c->it_dev);
  c->launches++;
}

void launch_advance_iteration(armor_ctx* c, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  advance_iteration_kernel<<<1, 1, 0, s>>>(c->it_dev);
  c->launches++;
}

void launch_stage(armor_ctx* c, armor_iter_stats* st, int stage, const double* part, int npart, int nflag,
                  cudaStream_t s, const double* p1, int n1, int slot1, const double* p2, int n2, int slot2) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  stage_kernel<<<1, STAGE_NT, 0, s>>>(c->sc, st, c->it_dev, stage, c->failflag, nflag, part, npart, c->status, p1, n1, slot1,
                               p2, n2, slot2);
  c->launches++;
}

void launch_split_hilo(armor_ctx* c, const float* in, float* hi, float* lo, int64_t n, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_OPERAND_SPLIT, 8.0 * (double)n, s);
  split_hilo_kernel<<<grid_for(n / 4), NT, 0, s>>>((const float4*)in, (float4*)hi, (float4*)lo, n / 4);
  c->launches++;
}

void launch_transpose_split(armor_ctx* c, const void* X, int x_dtype, int64_t ldx, int64_t rows, int64_t cols,
                            float* Thi, float* Tlo, int64_t ldt, cudaStream_t s) {
  dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((ldt + 31) / 32));
  KTimer kt(c, ARMOR_KC_GRAM_STAGING, (double)rows * (double)cols * (x_dtype == ARMOR_DTYPE_BF16 ? 6.0 : (Tlo ? 12.0 : 8.0)), s);
  if (x_dtype == ARMOR_DTYPE_BF16)
    transpose_split_kernel<<<grid, dim3(32, 8), 0, s>>>(static_cast<const __nv_bfloat16*>(X), ldx, rows, cols, Thi,
                                                       (float*)nullptr, ldt);
  else
    transpose_split_kernel<<<grid, dim3(32, 8), 0, s>>>(static_cast<const float*>(X), ldx, rows, cols, Thi, Tlo, ldt);
  c->launches++;
}

void launch_mirror_lower(armor_ctx* c, float* H, int64_t n, cudaStream_t s) {
  const unsigned t = (unsigned)((n + 31) / 32);
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  mirror_lower_kernel<<<dim3(t, t), dim3(32, 8), 0, s>>>(H, n);
  c->launches++;
}

void launch_block_fro_sum(armor_ctx* c, const float* X, int nblk, const float* hdiag, double* out, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  block_fro_kernel<<<nblk, NT, 0, s>>>((const float4*)X, c->db * c->db / 4, hdiag, c->db, c->nbi, c->quadpart);
  reduce_final_kernel<<<1, NT, 0, s>>>(c->quadpart, nblk, out);
  c->launches += 2;
}

void launch_adam(armor_ctx* c, float* theta, const float* gamma, float* m, float* v, int64_t n, const uint8_t* M,
                 int64_t step_base, cudaStream_t s) {
  const float lr = c->cfg.adam_lr > 0.f ? c->cfg.adam_lr : 1e-4f;
  const float b1 = c->cfg.adam_beta1 > 0.f ? c->cfg.adam_beta1 : 0.9f;
  const float b2 = c->cfg.adam_beta2 > 0.f ? c->cfg.adam_beta2 : 0.999f;
  const float eps = c->cfg.adam_eps > 0.f ? c->cfg.adam_eps : 1e-8f;
  KTimer kt(c, n >= (1 << 22) ? ARMOR_KC_AXPY : ARMOR_KC_SMALL, 28.0 * (double)n, s);
  adam_kernel<<<grid_for(n / 4), NT, 0, s>>>((float4*)theta, (const float4*)gamma, (float4*)m, (float4*)v, n / 4, M,
                                            c->cfg.m_group / 4, lr, b1, b2, eps, step_base, c->it_dev, c->status);
  c->launches++;
}

void launch_bf16_to_f32(armor_ctx* c, const void* in, const float* colscale, float* out, int64_t rows, int64_t cols,
                        cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_FORWARD, 6.0 * (double)rows * (double)cols, s);
  bf16_to_f32_kernel<<<grid_for(rows * cols), NT, 0, s>>>(static_cast<const __nv_bfloat16*>(in), colscale, out,
                                                         rows * cols, cols);
  c->launches++;
}

void launch_f32_to_bf16(armor_ctx* c, const float* in, const float* colscale, void* out, int64_t rows, int64_t cols,
                        cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_FORWARD, 6.0 * (double)rows * (double)cols, s);
  f32_to_bf16_kernel<<<grid_for(rows * cols), NT, 0, s>>>(in, colscale, static_cast<__nv_bfloat16*>(out), rows * cols,
                                                         cols);
  c->launches++;
}
