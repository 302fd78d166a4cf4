// Greedy sparse-core update (Algorithm 3 and Appendix B.1 of the paper): every 2:4 group of every
// (i, j) block is scored by the L1 norm of the core gradient, one group per block is drawn with
// probability proportional to its score, and that group is re-solved in closed form over all six
// masks (Eq. mask_loss_opt / mask_loss_opt_sol).
#include "armor_internal.cuh"

namespace {

constexpr int NT = 256;

__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// -ln(u) for u = (k + 1/2) / 2^24, k the top 24 bits of the hash.  Both branches feed the logarithm an
// argument that is exact in fp32, so the result is good to a few ulp even for u next to 1, where the
// winners of the exponential race live.
__device__ __forceinline__ float neg_log_uniform(uint32_t k24) {
  if (k24 < (1u << 23)) return -logf((float)(2u * k24 + 1u) * 2.98023223876953125e-8f);        // * 2^-25
  return -log1pf(-(float)(2u * ((1u << 24) - k24) - 1u) * 2.98023223876953125e-8f);
}

// alpha[r] = || A[:, r] ||^2 : column r of the block that owns row r of the core.
// blockDim = (32 columns, 8 row slices); grid = (nbo, db / 32).
__global__ void alpha_kernel(const float* __restrict__ A, float* __restrict__ alpha, int db) {
  const int i = blockIdx.x;
  const int r = blockIdx.y * 32 + threadIdx.x;
  const float* Ai = A + (int64_t)i * db * db;
  double acc = 0.0;
  if (r < db)
    for (int o = threadIdx.y; o < db; o += 8) {
      const double v = Ai[(int64_t)o * db + r];
      acc += v * v;
    }
  __shared__ double part[8][33];
  part[threadIdx.y][threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.y == 0 && r < db) {
    double t = 0.0;
    for (int k = 0; k < 8; ++k) t += part[k][threadIdx.x];
    alpha[i * db + r] = (float)t;
  }
}

// 2x2 PSD solve with the pseudo-inverse rule: w = K^+ z, red = z^T K^+ z.
__device__ __forceinline__ void pinv2(double k11, double k12, double k22, double z1, double z2, double& w1,
                                      double& w2, double& red) {
  const double det = k11 * k22 - k12 * k12;
  if (det <= 1e-12 * k11 * k22) {
    const double tr = k11 + k22;
    if (tr <= 0.0) { w1 = w2 = 0.0; red = 0.0; return; }
    const double inv = 1.0 / (tr * tr);
    w1 = (k11 * z1 + k12 * z2) * inv;
    w2 = (k12 * z1 + k22 * z2) * inv;
  } else {
    w1 = (k22 * z1 - k12 * z2) / det;
    w2 = (k11 * z2 - k12 * z1) / det;
  }
  red = z1 * w1 + z2 * w2;
}

// n x n SPD solve (n <= NKM) by unpivoted Cholesky; false if a pivot is not positive (that mask is skipped).
template <int NKM>
__device__ __forceinline__ bool chol_small(int n, const double (&Kin)[NKM][NKM], const double (&z)[NKM],
                                           double (&w)[NKM],
                                           double& red) {
  double L[NKM][NKM];
#pragma unroll
  for (int i = 0; i < NKM; ++i) {
#pragma unroll
    for (int j = 0; j < NKM; ++j) {
      if (i >= n || j > i) continue;
      double sacc = Kin[i][j];
#pragma unroll
      for (int p = 0; p < NKM; ++p)
        if (p < j) sacc -= L[i][p] * L[j][p];
      if (i == j) {
        if (!(sacc > 0.0) || !isfinite(sacc)) return false;
        L[i][i] = sqrt(sacc);
      } else {
        L[i][j] = sacc / L[j][j];
      }
    }
  }
  double y[NKM];
#pragma unroll
  for (int i = 0; i < NKM; ++i) {
    if (i >= n) continue;
    double sacc = z[i];
#pragma unroll
    for (int p = 0; p < NKM; ++p)
      if (p < i) sacc -= L[i][p] * y[p];
    y[i] = sacc / L[i][i];
  }
#pragma unroll
  for (int i = NKM - 1; i >= 0; --i) {
    if (i >= n) continue;
    double sacc = y[i];
#pragma unroll
    for (int p = 0; p < NKM; ++p)
      if (p > i && p < n) sacc -= L[p][i] * w[p];
    w[i] = sacc / L[i][i];
  }
  red = 0.0;
#pragma unroll
  for (int i = 0; i < NKM; ++i)
    if (i < n) red += z[i] * w[i];
  return true;
}

// One CTA per (i, j) block of the core, N:M groups with M = MG (4 or 8) and N = n_keep (<= NKM: 4 for 2:4 and 4:8, 6 for 5:8 and 6:8).
// Pass 1: every group of the block is scored, keyed and the arg-min found by warp shuffles.
// Pass 2: thread b < 2^MG evaluates the mask with bit pattern b (if it keeps exactly n_keep positions);
// the best one is found in this order: larger reduction first; among equal reductions the
// incumbent, then the lexicographically first index tuple.
// PHASE 0: both passes in one launch (several draws per block).  A single draw runs as two launches, so that the
// streaming pass keeps few registers and the per-block solves, which are chains of dependent loads, all run
// side by side: PHASE 1 is pass 1 alone (the block's winner goes to best_key / best_g), PHASE 2 is pass 2
// alone (one warp per block for groups of four, 256 threads for groups of eight).
template <int MG, int NKM, bool MULTI, int PHASE>
__global__ void __launch_bounds__(NT) mask_select_kernel(const float* __restrict__ Gam, const float* __restrict__ S,
                                                         const uint8_t* __restrict__ M, const float* __restrict__ alpha,
                                                         const float* __restrict__ Kfull, SelRec* __restrict__ sel,
                                                         double* __restrict__ part, int64_t d_in, int db, int nbi,
                                                         int n_keep, int select_mode, uint64_t seed, uint64_t t_base,
                                                         uint64_t t_mul, const int64_t* __restrict__ it_dev,
                                                         uint64_t n_groups_total, int kg_arg,
                                                         float* __restrict__ tab_key,
                                                         unsigned long long* __restrict__ tab_g) {
  const uint64_t t = t_base + t_mul * (uint64_t)(*it_dev);   // selection counter of this run of Algorithm 3
  const int kg = MULTI ? kg_arg : 1;                       // one draw: the loop and the key cache compile away
  const int bi = blockIdx.x / nbi, bj = blockIdx.x % nbi;
  extern __shared__ float s_keys[];         // kg > 1: the keys of the block's groups, kept for the later draws
  const int gpb = db / MG;                // groups per block row
  const int64_t ng_row = d_in / MG;       // groups per matrix row
  const int n_in_block = db * gpb;
  // kg draws: the kg smallest keys of the block, one after the other; the record of draw kk of block (i, j) is
  // entry (i, kk * nbi + j) of a [nbo][kg * nbi] table (kk * nbi + j acts as a column block of its own downstream)
  for (int kk = 0; kk < kg; ++kk) {
  const int blk = bi * (kg * nbi) + kk * nbi + bj;
  float best_key = INFINITY;
  uint64_t best_g = ~0ull;
  if (PHASE == 2) {
    best_key = tab_key[blk];
    best_g = tab_g[blk];
  } else {
  if (MULTI && kk > 0) {
    // later draws: keys from the first pass, drawn ones at +inf
    for (int idx = threadIdx.x; idx < n_in_block; idx += NT) {
      const int rl = idx / gpb, cl = idx % gpb;
      const float key = s_keys[idx];
      const uint64_t g = (uint64_t)((int64_t)bi * db + rl) * (uint64_t)ng_row + (uint64_t)((int64_t)bj * gpb + cl);
      if (key < best_key || (key == best_key && g < best_g)) { best_key = key; best_g = g; }
    }
  } else {
    // A thread keeps one group column of the block and walks down its rows, NT / gpb rows apart (threads beyond
    // the last whole row of groups idle), so the group index, the hash counter and the addresses advance by
    // additions.  Four groups per thread and step: the loads are issued together, then scores and hashes.
    // With a single draw most logarithms are skipped: -ln(u) >= 1 - u, so a group whose (1 - u) / score
    // exceeds the best key its warp has seen cannot win (the bound is tight exactly where winners live, u next
    // to 1; the warp-wide bound, refreshed after every step, makes whole warps skip the logarithm, which a
    // per-thread bound would not: among 32 lanes one almost always passes its own).
    constexpr int U = 4;
    const int rstep = NT / gpb;                                  // rows of the block covered per step (gpb <= 64)
    const int cl = (int)threadIdx.x % gpb, rl0 = (int)threadIdx.x / gpb;
    {
      const bool lane_on = rl0 < rstep;
      float wbound = INFINITY;                                   // warp-uniform: the smallest key any lane holds
      const int n_steps = (db + U * rstep - 1) / (U * rstep);    // the same for every lane: the shuffles below need all 32
      const int64_t row0 = (int64_t)bi * db + (lane_on ? rl0 : 0);
      const int64_t cg = (int64_t)bj * gpb + cl;
      const float* gp = Gam + row0 * d_in + cg * MG;
      const float* ap = alpha + row0;
      uint64_t g = (uint64_t)row0 * (uint64_t)ng_row + (uint64_t)cg;
      uint64_t ctr = t * n_groups_total + g;
      const uint64_t gstep = (uint64_t)rstep * (uint64_t)ng_row;
      const int64_t pstep = (int64_t)rstep * d_in;
      for (int step = 0, rl = rl0; step < n_steps; ++step, rl += U * rstep) {
        float4 g4[U][MG / 4];
        float al[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          al[u] = 0.f;
#pragma unroll
          for (int h = 0; h < MG / 4; ++h) g4[u][h] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (lane_on && rl + u * rstep < db) {
            al[u] = ap[u * rstep];
#pragma unroll
            for (int h = 0; h < MG / 4; ++h) g4[u][h] = *reinterpret_cast<const float4*>(gp + u * pstep + 4 * h);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (lane_on && rl + u * rstep < db) {
            float score = 0.f, sq = 0.f;
#pragma unroll
            for (int h = 0; h < MG / 4; ++h) {
              score += fabsf(g4[u][h].x);
              score += fabsf(g4[u][h].y);
              score += fabsf(g4[u][h].z);
              score += fabsf(g4[u][h].w);
              if (select_mode == ARMOR_SELECT_L2_RANDOM) {
                sq = fmaf(g4[u][h].x, g4[u][h].x, sq);
                sq = fmaf(g4[u][h].y, g4[u][h].y, sq);
                sq = fmaf(g4[u][h].z, g4[u][h].z, sq);
                sq = fmaf(g4[u][h].w, g4[u][h].w, sq);
              }
            }
            // the ablation's weights (Appendix E.1): L2 norm of the group's gradient, or equal weights
            if (select_mode == ARMOR_SELECT_L2_RANDOM) score = sqrtf(sq);
            else if (select_mode == ARMOR_SELECT_UNIFORM_RANDOM) score = 1.f;
            if (!(al[u] > 0.f)) score = 0.f;
            const uint64_t gu = g + (uint64_t)u * gstep;
            float key = INFINITY;
            if (score > 0.f) {
              if (select_mode != ARMOR_SELECT_L1_GREEDY) {
                const uint64_t bits = splitmix64(seed ^ splitmix64(ctr + (uint64_t)u * gstep));
                const uint32_t k24 = (uint32_t)(bits >> 40);
                // 1 - u = (2^24 - k24 - 1/2) 2^-24, exact in fp32; the factor 1 - 1e-5 covers the few ulp by
                // which the computed key can fall below (1 - u) / score
                const float one_minus_u = (float)(2u * ((1u << 24) - k24) - 1u) * 2.98023223876953125e-8f;
                if (MULTI || !(one_minus_u * 0.99999f >= wbound * score))
                  key = neg_log_uniform(k24) / score;
              } else {
                key = -score;
              }
              if (key < best_key || (key == best_key && gu < best_g)) { best_key = key; best_g = gu; }
            }
            if (MULTI) s_keys[(rl + u * rstep) * gpb + cl] = key;
          }
        }
        gp += U * pstep;
        ap += U * rstep;
        g += U * gstep;
        ctr += U * gstep;
        if (!MULTI) {
          wbound = best_key;
          for (int o = 16; o > 0; o >>= 1) wbound = fminf(wbound, __shfl_xor_sync(0xffffffffu, wbound, o));
        }
      }
    }
  }
  // arg-min over the CTA; ties go to the lower group index
  for (int o = 16; o > 0; o >>= 1) {
    const float ok = __shfl_down_sync(0xffffffffu, best_key, o);
    const uint64_t og = __shfl_down_sync(0xffffffffu, best_g, o);
    if (ok < best_key || (ok == best_key && og < best_g)) { best_key = ok; best_g = og; }
  }
  __shared__ float skey[NT / 32];
  __shared__ uint64_t sg[NT / 32];
  __shared__ float s_key;
  __shared__ uint64_t s_g;
  if ((threadIdx.x & 31) == 0) { skey[threadIdx.x >> 5] = best_key; sg[threadIdx.x >> 5] = best_g; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < NT / 32; ++w)
      if (skey[w] < best_key || (skey[w] == best_key && sg[w] < best_g)) { best_key = skey[w]; best_g = sg[w]; }
    s_key = best_key;
    s_g = best_g;
  }
  __syncthreads();
  best_key = s_key;
  best_g = s_g;
  if (PHASE == 1) {
    if (threadIdx.x == 0) { tab_key[blk] = best_key; tab_g[blk] = best_g; }
    return;
  }
  }
  if (!(best_key < INFINITY)) {                               // nothing left to draw in this block (uniform)
    if (threadIdx.x == 0) {
      SelRec rec;
      rec.valid = 0; rec.row = 0; rec.cgrp = 0; rec.new_mask = 0; rec.old_mask = 0;
      for (int p = 0; p < 8; ++p) { rec.new_val[p] = 0.f; rec.old_val[p] = 0.f; }
      for (int k2 = kk; k2 < kg; ++k2) {
        sel[bi * (kg * nbi) + k2 * nbi + bj] = rec;
        part[bi * (kg * nbi) + k2 * nbi + bj] = 0.0;
      }
    }
    return;
  }
  if (MULTI && threadIdx.x == 0) {                          // out of the race for the later draws
    const int rl0 = (int)(best_g / (uint64_t)ng_row) - bi * db, cl0 = (int)(best_g % (uint64_t)ng_row) - bj * gpb;
    s_keys[rl0 * gpb + cl0] = INFINITY;
  }

  // ---- the selected group: z = Gamma_g + alpha K_c s_g, one candidate mask per thread
  const int64_t row = (int64_t)(best_g / (uint64_t)ng_row);
  const int64_t cg = (int64_t)(best_g % (uint64_t)ng_row);
  const int lc = (int)(cg % gpb) * MG;   // first row of the group inside B_j
  const float* Kj = Kfull + (int64_t)bj * db * db;
  const double a_r = (double)alpha[row];
  const unsigned om = M[row * ng_row + cg];
  double z[MG], sg_old[MG];
#pragma unroll
  for (int p = 0; p < MG; ++p) sg_old[p] = (double)S[row * d_in + cg * MG + p];
#pragma unroll
  for (int p = 0; p < MG; ++p) {
    double kz = 0.0;
#pragma unroll
    for (int q = 0; q < MG; ++q) kz += (double)Kj[(int64_t)(lc + p) * db + (lc + q)] * sg_old[q];
    z[p] = (double)Gam[row * d_in + cg * MG + p] + a_r * kz;
  }
  const unsigned cand = threadIdx.x;
  bool ok = cand < (1u << MG) && __popc(cand) == n_keep;
  double red = 0.0, wv[NKM];
  int pos[NKM];
#pragma unroll
  for (int i = 0; i < NKM; ++i) { wv[i] = 0.0; pos[i] = 0; }
  if (ok) {
    int cnt = 0;
#pragma unroll
    for (int p = 0; p < MG; ++p)
      if ((cand >> p) & 1u) { if (cnt < NKM) pos[cnt] = p; ++cnt; }
    if (n_keep == 2) {
      pinv2((double)Kj[(int64_t)(lc + pos[0]) * db + lc + pos[0]], (double)Kj[(int64_t)(lc + pos[0]) * db + lc + pos[1]],
            (double)Kj[(int64_t)(lc + pos[1]) * db + lc + pos[1]], z[pos[0]], z[pos[1]], wv[0], wv[1], red);
    } else {
      double Ks[NKM][NKM], zs[NKM];
#pragma unroll
      for (int i = 0; i < NKM; ++i) {
        zs[i] = 0.0;
#pragma unroll
        for (int j = 0; j < NKM; ++j) Ks[i][j] = 0.0;
      }
#pragma unroll
      for (int i = 0; i < NKM; ++i) {
        if (i >= n_keep) continue;
#pragma unroll
        for (int p = 0; p < MG; ++p)
          if (p == pos[i]) zs[i] = z[p];
#pragma unroll
        for (int j = 0; j < NKM; ++j)
          if (j < n_keep) Ks[i][j] = (double)Kj[(int64_t)(lc + pos[i]) * db + lc + pos[j]];
      }
      ok = chol_small<NKM>(n_keep, Ks, zs, wv, red);
    }
    red /= a_r;
  }
  // order: larger reduction; then the incumbent; then the lexicographically first tuple (= larger
  // bit-reversed pattern)
  const unsigned rev = __brev(cand) >> (32 - MG);
  double b_red = ok ? red : -INFINITY;
  unsigned b_tie = ok ? (((cand == om) ? (1u << MG) : 0u) | rev) : 0u;
  unsigned b_cand = ok ? cand : 0xffffffffu;
  for (int o = 16; o > 0; o >>= 1) {
    const double o_red = __shfl_down_sync(0xffffffffu, b_red, o);
    const unsigned o_tie = __shfl_down_sync(0xffffffffu, b_tie, o);
    const unsigned o_cand = __shfl_down_sync(0xffffffffu, b_cand, o);
    const bool take = (o_cand != 0xffffffffu) &&
                      (b_cand == 0xffffffffu || o_red > b_red || (o_red == b_red && o_tie > b_tie));
    if (take) { b_red = o_red; b_tie = o_tie; b_cand = o_cand; }
  }
  __shared__ double sred[NT / 32];
  __shared__ unsigned stie[NT / 32], scand[NT / 32];
  __shared__ unsigned s_win;
  if ((threadIdx.x & 31) == 0) { sred[threadIdx.x >> 5] = b_red; stie[threadIdx.x >> 5] = b_tie; scand[threadIdx.x >> 5] = b_cand; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) {
      const bool take = (scand[w] != 0xffffffffu) &&
                        (b_cand == 0xffffffffu || sred[w] > b_red || (sred[w] == b_red && stie[w] > b_tie));
      if (take) { b_red = sred[w]; b_tie = stie[w]; b_cand = scand[w]; }
    }
    s_win = b_cand;
    if (b_cand == 0xffffffffu) {   // every mask failed its factorisation: nothing happens in this block
      SelRec rec;
      rec.valid = 0; rec.row = 0; rec.cgrp = 0; rec.new_mask = 0; rec.old_mask = 0;
      for (int p = 0; p < 8; ++p) { rec.new_val[p] = 0.f; rec.old_val[p] = 0.f; }
      sel[blk] = rec;
      part[blk] = 0.0;
    }
  }
  __syncthreads();
  if (s_win != 0xffffffffu && cand == s_win) {
  // the winning thread writes the record
  SelRec rec;
  rec.valid = 1;
  rec.row = (int32_t)row;
  rec.cgrp = (int32_t)cg;
  rec.old_mask = (int32_t)om;
  rec.new_mask = (int32_t)cand;
  for (int p = 0; p < 8; ++p) { rec.new_val[p] = 0.f; rec.old_val[p] = 0.f; }
#pragma unroll
  for (int p = 0; p < MG; ++p) rec.old_val[p] = (float)sg_old[p];
#pragma unroll
  for (int i = 0; i < NKM; ++i)
    if (i < n_keep) rec.new_val[pos[i]] = (float)(wv[i] / a_r);
  // <Gamma, dS> restricted to this group: this block's share of <E H_w, V>
  double ehv = 0.0;
#pragma unroll
  for (int p = 0; p < MG; ++p)
    ehv += (double)Gam[row * d_in + cg * MG + p] * ((double)rec.new_val[p] - (double)rec.old_val[p]);
  part[blk] = ehv;
  sel[blk] = rec;
  }
  __syncthreads();                                          // the shared scratch is reused by the next draw
  }
}

// The group updates of one iteration change the core by dS (one group per (i, j) block) and the
// reconstruction by V = A dS B.  Block (i, j) of dS has a single non-zero row r, so
//   tr(V H_w V^T) = sum_i sum_{j, j'} (a_ij . a_ij') * (z_ij H_w[j, j'] z_ij'^T)
// with a_ij = A_i[:, r_ij] and z_ij = delta_ij^T B_j[rows of the group, :]: row-blocks decouple because A is
// block diagonal.  mask_vectors_kernel gathers a and z, a batched product forms y_ij = z_ij H_w[j-th block
// row, :], and mask_quad_kernel sums the pairs in a fixed order.
__global__ void __launch_bounds__(NT) mask_vectors_kernel(const float* __restrict__ A, const float* __restrict__ B,
                                                          const SelRec* __restrict__ sel, float* __restrict__ Zsel,
                                                          float* __restrict__ Acol, int db, int nbo_pad, int nbi, int mg,
                                                          int nbv) {
  const int blk = blockIdx.x;                  // (row block, virtual column block v = draw * nbi + column block)
  const int bi = blk / nbv, v = blk % nbv, bj = v % nbi;
  const SelRec rec = sel[blk];
  for (int k = threadIdx.x; k < db; k += NT) {
    float a = 0.f, z = 0.f;
    if (rec.valid) {
      const int rl = rec.row - bi * db;
      const int lc = (rec.cgrp % (db / mg)) * mg;
      a = A[(int64_t)bi * db * db + (int64_t)k * db + rl];
      const float* Bj = B + (int64_t)bj * db * db;
      for (int p = 0; p < mg; ++p) z = fmaf(rec.new_val[p] - rec.old_val[p], Bj[(int64_t)(lc + p) * db + k], z);
    }
    Acol[((int64_t)bi * nbv + v) * db + k] = a;
    Zsel[((int64_t)v * nbo_pad + bi) * db + k] = z;
  }
}

// One CTA per block (i, j), one warp per pair (j, j') at a time.  Y == nullptr: diagonal weighting, only the
// j == j' pair contributes and y = z (.) hdiag.
__global__ void __launch_bounds__(NT) mask_quad_kernel(const float* __restrict__ Zsel, const float* __restrict__ Acol,
                                                       const float* __restrict__ Y, const float* __restrict__ hdiag,
                                                       double* __restrict__ part, int64_t d_in, int db, int nbo_pad,
                                                       int nbi, int nbv) {
  const int bi = blockIdx.x / nbv, j = blockIdx.x % nbv;      // j, j2: virtual column blocks (draw * nbi + column block)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = NT / 32;
  double acc = 0.0;
  const float* a1 = Acol + ((int64_t)bi * nbv + j) * db;
  const float* z1 = Zsel + ((int64_t)j * nbo_pad + bi) * db;
  for (int j2 = warp; j2 < nbv; j2 += nw) {
    if (!Y && (j2 % nbi) != (j % nbi)) continue;              // diagonal weighting: other column blocks do not interact
    const float* a2 = Acol + ((int64_t)bi * nbv + j2) * db;
    const float* z2 = Zsel + ((int64_t)j2 * nbo_pad + bi) * db;
    float w = 0.f, m = 0.f;
    if (Y) {
      const float* y = Y + ((int64_t)j * nbo_pad + bi) * d_in + (int64_t)(j2 % nbi) * db;
      for (int k = lane; k < db; k += 32) { w = fmaf(a1[k], a2[k], w); m = fmaf(y[k], z2[k], m); }
    } else {
      const float* h = hdiag + (int64_t)(j % nbi) * db;
      for (int k = lane; k < db; k += 32) { w = fmaf(a1[k], a2[k], w); m = fmaf(z1[k] * h[k], z2[k], m); }
    }
    for (int o = 16; o > 0; o >>= 1) {
      w += __shfl_xor_sync(0xffffffffu, w, o);
      m += __shfl_xor_sync(0xffffffffu, m, o);
    }
    acc += (double)w * (double)m;
  }
  __shared__ double red[NT / 32];
  if (lane == 0) red[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w2 = 0; w2 < nw; ++w2) t += red[w2];
    part[blockIdx.x] = t;
  }
}

__global__ void mask_commit_kernel(const SelRec* __restrict__ sel, int nblocks, float* __restrict__ S,
                                   uint8_t* __restrict__ M, int64_t d_in, int mg, const double* __restrict__ sc,
                                   armor_iter_stats* st_base, const int64_t* __restrict__ it_dev) {
  armor_iter_stats* st = st_base ? st_base + *it_dev : nullptr;
  __shared__ int changed;
  if (threadIdx.x == 0) changed = 0;
  __syncthreads();
  const bool accept = sc[SC_ACCEPT] != 0.0;
  int mine = 0;
  if (accept) {
    for (int b = threadIdx.x; b < nblocks; b += blockDim.x) {
      const SelRec rec = sel[b];
      if (!rec.valid) continue;
      float* sp = S + (int64_t)rec.row * d_in + (int64_t)rec.cgrp * mg;
      for (int h = 0; h < mg / 4; ++h)
        *reinterpret_cast<float4*>(sp + 4 * h) =
            make_float4(rec.new_val[4 * h], rec.new_val[4 * h + 1], rec.new_val[4 * h + 2], rec.new_val[4 * h + 3]);
      M[(int64_t)rec.row * (d_in / mg) + rec.cgrp] = (uint8_t)rec.new_mask;
      mine += (rec.new_mask != rec.old_mask) ? 1 : 0;
    }
  }
  atomicAdd(&changed, mine);
  __syncthreads();
  if (threadIdx.x == 0 && st) st->groups_changed += changed;   // summed over the sweeps of the iteration
}

// The accepted group updates change T H_w = S B H_w by the rows (delta^T B_j[group rows, :]) H_w[j-th block
// row, :] = y_ij, added to row r_ij.  Groups of one row-block may share a row, so one CTA walks the column
// blocks j in order (deterministic sums); the grid is (row-block, chunk of 1024 columns).
__global__ void __launch_bounds__(NT) mask_carry_kernel(const SelRec* __restrict__ sel, const float* __restrict__ Y,
                                                        float* __restrict__ P, const double* __restrict__ sc,
                                                        int64_t d_in, int nbo_pad, int nbv) {
  if (sc[SC_ACCEPT] == 0.0) return;
  const int bi = blockIdx.x;
  const int64_t c4 = (int64_t)blockIdx.y * 1024 + 4 * threadIdx.x;
  if (c4 >= d_in) return;
  // Virtual column blocks in order, eight at a time.  The eight rows are almost always distinct: then their loads are
  // independent and issued together (a chain of 32 dependent read-modify-writes was the whole cost of this kernel);
  // a batch in which two groups share a row is walked one by one, so that every element of P sees its additions in
  // the order of the column blocks (deterministic sums).
  for (int j0 = 0; j0 < nbv; j0 += 8) {
    int row[8];
    bool val[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      val[u] = false; row[u] = 0;
      if (j0 + u < nbv) {
        const SelRec* rec = sel + (bi * nbv + j0 + u);
        val[u] = rec->valid != 0;
        row[u] = rec->row;
      }
    }
    bool shared_row = false;
#pragma unroll
    for (int u = 1; u < 8; ++u)
#pragma unroll
      for (int w = 0; w < u; ++w) shared_row |= val[u] && val[w] && row[u] == row[w];
    if (!shared_row) {
      float4 y[8], v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (val[u]) {
          y[u] = *reinterpret_cast<const float4*>(Y + ((int64_t)(j0 + u) * nbo_pad + bi) * d_in + c4);
          v[u] = *reinterpret_cast<const float4*>(P + (int64_t)row[u] * d_in + c4);
        }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (val[u]) {
          v[u].x += y[u].x; v[u].y += y[u].y; v[u].z += y[u].z; v[u].w += y[u].w;
          *reinterpret_cast<float4*>(P + (int64_t)row[u] * d_in + c4) = v[u];
        }
    } else {
      for (int u = 0; u < 8; ++u) {
        if (!val[u]) continue;
        const float4 y = *reinterpret_cast<const float4*>(Y + ((int64_t)(j0 + u) * nbo_pad + bi) * d_in + c4);
        float4* dst = reinterpret_cast<float4*>(P + (int64_t)row[u] * d_in + c4);
        float4 v = *dst;
        v.x += y.x; v.y += y.y; v.z += y.z; v.w += y.w;
        *dst = v;
      }
    }
  }
}

}  // namespace

void launch_mask_carry_P(armor_ctx* c, float* P, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_MASK_GUARD, 0.0, s);
  mask_carry_kernel<<<dim3(c->nbo, (unsigned)((c->d_in + 1023) / 1024)), NT, 0, s>>>(c->sel, c->Ysel, P, c->sc, c->d_in,
                                                                                   c->nbo_pad, c->nbi * c->kg);
  c->launches++;
}

void launch_alpha(armor_ctx* c, const float* A, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_MASK_GUARD, 0.0, s);
  alpha_kernel<<<dim3(c->nbo, (c->db + 31) / 32), dim3(32, 8), 0, s>>>(A, c->alpha, c->db);
  c->launches++;
}

// alpha (column norms of the blocks of A) and the m x m diagonal blocks of K_j = (B_j H_jj) B_j^T, the only entries
// of K_j the group solves read (Appendix B.1: B' D B'^T for the m rows of one group), in one launch.
// Y = B_j H_jj comes from a block product.  CTAs [0, n_kc): one warp per group, lane l takes columns l, l + 32, ..;
// the remaining CTAs compute alpha.
template <int MG>
__global__ void __launch_bounds__(NT) mask_prep_kernel(const float* __restrict__ A, const float* __restrict__ B,
                                                       const float* __restrict__ Y, float* __restrict__ Kfull,
                                                       float* __restrict__ alpha, int db, int nbi, int n_kc) {
  if ((int)blockIdx.x < n_kc) {
    const int gpb = db / MG;
    const int wg = blockIdx.x * (NT / 32) + (threadIdx.x >> 5);       // (column block, group)
    const int lane = threadIdx.x & 31;
    if (wg >= nbi * gpb) return;
    const int j = wg / gpb, lc = (wg % gpb) * MG;
    const float* Yj = Y + (int64_t)j * db * db;
    const float* Bj = B + (int64_t)j * db * db;
    float acc[MG][MG];
#pragma unroll
    for (int p = 0; p < MG; ++p)
#pragma unroll
      for (int q = 0; q < MG; ++q) acc[p][q] = 0.f;
    for (int k = lane; k < db; k += 32) {
      float y[MG], b[MG];
#pragma unroll
      for (int p = 0; p < MG; ++p) { y[p] = Yj[(int64_t)(lc + p) * db + k]; b[p] = Bj[(int64_t)(lc + p) * db + k]; }
#pragma unroll
      for (int p = 0; p < MG; ++p)
#pragma unroll
        for (int q = 0; q < MG; ++q) acc[p][q] = fmaf(y[p], b[q], acc[p][q]);
    }
#pragma unroll
    for (int p = 0; p < MG; ++p)
#pragma unroll
      for (int q = 0; q < MG; ++q) {
        float v = acc[p][q];
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) Kfull[(int64_t)j * db * db + (int64_t)(lc + p) * db + (lc + q)] = v;
      }
    return;
  }
  // alpha[r] = || A_i[:, r] ||^2: 256 threads = 32 columns x 8 row slices
  const int ab = blockIdx.x - n_kc;
  const int per = (db + 31) / 32;
  const int i = ab / per;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int r = (ab % per) * 32 + tx;
  const float* Ai = A + (int64_t)i * db * db;
  double acc = 0.0;
  if (r < db)
    for (int o = ty; o < db; o += 8) {
      const double v = Ai[(int64_t)o * db + r];
      acc += v * v;
    }
  __shared__ double part[8][33];
  part[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && r < db) {
    double t = 0.0;
    for (int k = 0; k < 8; ++k) t += part[k][tx];
    alpha[i * db + r] = (float)t;
  }
}

void launch_mask_prep(armor_ctx* c, const float* A, const float* B, const float* Y, cudaStream_t s) {
  const int db = c->db, mg = c->cfg.m_group;
  const int n_kc = (c->nbi * (db / mg) + NT / 32 - 1) / (NT / 32);
  const int n_al = c->nbo * ((db + 31) / 32);
  KTimer kt(c, ARMOR_KC_MASK_GUARD, 0.0, s);
  if (mg == 8) mask_prep_kernel<8><<<n_kc + n_al, NT, 0, s>>>(A, B, Y, c->Kfull, c->alpha, db, c->nbi, n_kc);
  else mask_prep_kernel<4><<<n_kc + n_al, NT, 0, s>>>(A, B, Y, c->Kfull, c->alpha, db, c->nbi, n_kc);
  c->launches++;
}

void launch_mask_select(armor_ctx* c, const float* Gam, const float* S, const uint8_t* M, uint64_t t_base, uint64_t t_mul,
                        cudaStream_t s) {
  const int mg = c->cfg.m_group;
  const uint64_t n_groups = (uint64_t)(c->d_out * (c->d_in / mg));
#define ARMOR_SELECT_ARGS Gam, S, M, c->alpha, c->Kfull, c->sel, c->partblk, c->d_in, c->db, c->nbi, c->cfg.n_keep, \
                          c->cfg.select_mode, c->cfg.seed, t_base, t_mul, c->it_dev, n_groups, c->kg, c->tab_key, c->tab_g
  // kg > 1: the block's keys stay in shared memory between the draws (up to 64 KiB: d_block 256, groups of four)
  const size_t smem = c->kg > 1 ? (size_t)c->db * (c->db / mg) * sizeof(float) : 0;
#define ARMOR_SELECT_LAUNCH(MGV, NKV, MULTIV)                                                                           \
  do {                                                                                                                  \
    if (MULTIV) {                                                                                                       \
      if (smem > 48 * 1024)                                                                                             \
        cudaFuncSetAttribute(mask_select_kernel<MGV, NKV, MULTIV, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize,      \
                             (int)smem);                                                                                \
      mask_select_kernel<MGV, NKV, MULTIV, 0><<<c->nbo * c->nbi, NT, smem, s>>>(ARMOR_SELECT_ARGS);                     \
    } else {                                                                                                            \
      mask_select_kernel<MGV, NKV, false, 1><<<c->nbo * c->nbi, NT, 0, s>>>(ARMOR_SELECT_ARGS);                         \
      mask_select_kernel<MGV, NKV, false, 2><<<c->nbo * c->nbi, MGV == 4 ? 32 : NT, 0, s>>>(ARMOR_SELECT_ARGS);         \
      c->launches++;                                                                                                    \
    }                                                                                                                   \
  } while (0)
  const bool multi = c->kg > 1;
  KTimer kt(c, ARMOR_KC_MASK_SELECT, 4.0 * (double)c->wn, s);   // one read of the core gradient
  if (mg == 8 && c->cfg.n_keep > 4) { if (multi) ARMOR_SELECT_LAUNCH(8, 6, true); else ARMOR_SELECT_LAUNCH(8, 6, false); }
  else if (mg == 8) { if (multi) ARMOR_SELECT_LAUNCH(8, 4, true); else ARMOR_SELECT_LAUNCH(8, 4, false); }
  else { if (multi) ARMOR_SELECT_LAUNCH(4, 4, true); else ARMOR_SELECT_LAUNCH(4, 4, false); }
#undef ARMOR_SELECT_LAUNCH
#undef ARMOR_SELECT_ARGS
  c->launches++;
}

void launch_mask_quadratic(armor_ctx* c, const float* A, const float* B, const float* H, cudaStream_t s) {
  const int db = c->db, nbo = c->nbo, nbi = c->nbi, nbo_pad = c->nbo_pad, kg = c->kg, nbv = nbi * kg;
  {
    KTimer kt(c, ARMOR_KC_MASK_GUARD, 0.0, s);
    mask_vectors_kernel<<<nbo * nbv, NT, 0, s>>>(A, B, c->sel, c->Zsel, c->Acol, db, nbo_pad, nbi, c->cfg.m_group, nbv);
  }
  c->launches++;
  const float* Y = nullptr;
  if (c->cfg.h_mode == ARMOR_H_FULL) {
    // y_v = z_v H[j-th block row, :], batched over the column blocks j, one launch per draw:  [nbo, db] x [db, d_in]
    for (int kk = 0; kk < kg; ++kk) {
      const float* Zk = c->Zsel + (int64_t)kk * nbi * nbo_pad * db;
      float* Yk = c->Ysel + (int64_t)kk * nbi * nbo_pad * c->d_in;
      if (!(c->tc_blocks && tc_gram_ok(c) && tc_done(c, tc_select_rows_times_H(c, Zk, H, Yk, nbo_pad, s)))) {
        BGemm g{};
        g.A = Zk; g.sAb = (int64_t)nbo_pad * db; g.sAm = db; g.sAk = 1;
        g.B = H; g.sBb = (int64_t)db * c->d_in; g.sBk = c->d_in; g.sBn = 1;
        g.C = Yk; g.sCb = (int64_t)nbo_pad * c->d_in; g.sCm = c->d_in; g.sCn = 1;
        g.M = nbo; g.N = (int)c->d_in; g.K = db; g.batch = nbi; g.alpha = 1.f;
        launch_bgemm(c, g, s);
      }
    }
    Y = c->Ysel;
  }
  double* part = c->quadpart;
  {
    KTimer kt(c, ARMOR_KC_MASK_GUARD, 0.0, s);
    mask_quad_kernel<<<nbo * nbv, NT, 0, s>>>(c->Zsel, c->Acol, Y, c->hdiag, part, c->d_in, db, nbo_pad, nbi, nbv);
  }
  c->launches++;
  // (the caller's stage kernel adds the nbo * nbv terms up into sc[SC_Q_M])
}

void launch_mask_commit(armor_ctx* c, float* S, uint8_t* M, armor_iter_stats* st, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_MASK_GUARD, 0.0, s);
  mask_commit_kernel<<<1, 256, 0, s>>>(c->sel, c->nbo * c->nbi * c->kg, S, M, c->d_in, c->cfg.m_group, c->sc, st,
                                       c->it_dev);
  c->launches++;
}
