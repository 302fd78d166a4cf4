// Per-block SPD solves for the wrapper updates.  The block systems are the zeros of the paper's
// gradients with respect to A and B (Appendix D.1 and D.2) made proximal by a relative ridge:
//   mode 0 (A update): X = Gamma (G + lam I)^-1;  A += X;  dA = X;  part = <Gamma, X> + lam |X|^2
//   mode 1 (left)    : out = (G + lam I)^-1 rhs
//   mode 2 (right+gd): out = rhs (G + lam I)^-1;  part = <dotw, out>
// A failed factorisation leaves A unchanged / writes zeros and raises failflag[block].
//
// One CTA factorises one d_block x d_block matrix in shared memory and solves for a slice of the
// right-hand sides (all of them for d_block <= 128; d_block = 256 is split over four CTAs that each
// repeat the factorisation, because factor and right-hand sides do not fit one CTA's shared memory).
// Blocked left-looking Cholesky with panels of 32 columns: a panel first receives the contributions of
// all earlier panels as one small matrix product (every element is accumulated in fp64 and rounded to
// fp32 once), then its 32 columns are eliminated with dot products of at most 31 terms.  The
// triangular solves are blocked the same way; the 32 x 32 diagonal solves keep one right-hand side per
// thread in registers and eliminate column by column, so the dependent chain is one multiply-add per
// unknown.
#include "armor_internal.cuh"

namespace {

constexpr int NT = 256;
constexpr int NB = 32;       // panel width
constexpr int LDP = NB + 1;  // padded row length of a panel

struct PanelMap {
  int db;
  // offset (floats) of panel kb: rows NB*kb .. db-1, LDP floats each
  __device__ __forceinline__ int off(int kb) const { return LDP * (kb * db - NB * kb * (kb - 1) / 2); }
  // element (i, k), i >= NB * (k / NB)
  __device__ __forceinline__ int at(int i, int k) const {
    const int kb = k / NB;
    return off(kb) + (i - NB * kb) * LDP + (k - NB * kb);
  }
};

__host__ __device__ inline size_t panel_floats(int db) {
  const int np = db / NB;
  return (size_t)LDP * ((size_t)np * db - (size_t)NB * np * (np - 1) / 2);
}

// y -= sum over the 32 columns of one earlier panel, fp32 products; the caller adds the chunk to an fp64 sum
#define ARMOR_TILE_ZERO(acc)                                   \
  _Pragma("unroll") for (int a_ = 0; a_ < 4; ++a_)             \
  _Pragma("unroll") for (int b_ = 0; b_ < 4; ++b_) acc[a_][b_] = 0.f;

__global__ void __launch_bounds__(NT, 1)
chol_blocked_kernel(int mode, const float* __restrict__ Gmat, const float* __restrict__ rhs, float* __restrict__ out,
                    const float* __restrict__ dotw, float* __restrict__ A, float ridge, int db,
                    int w, double* __restrict__ part, int32_t* __restrict__ failflag, int32_t* __restrict__ status) {
  extern __shared__ float smem[];
  const PanelMap pm{db};
  const int np = db / NB;
  const int ldr = w + 1;
  float* Lp = smem;
  float* Rs = smem + panel_floats(db);                  // [db][w + 1]: row = unknown index, column = right-hand side
  __shared__ float Df[NB][NB + 1];                      // diagonal block of the current panel
  __shared__ float invd[NB];                            // reciprocals of its diagonal
  __shared__ double red[NT / 32];
  __shared__ int s_fail;
  __shared__ double s_lam;
  const int b = blockIdx.x, q = blockIdx.y, tid = threadIdx.x, lane = threadIdx.x & 31;
  const int64_t off = (int64_t)b * db * db;
  const bool right = (mode != 1);
  const int v0 = q * w;  // first right-hand side of this CTA

  // ---- load: lower triangle of G, the slice of right-hand sides.  float4 loads, eight in flight per
  // thread, so that the global-memory latency is paid a few times and not once per element.
  {
    const int q4 = db / 4;                      // float4 per row
    const int n4 = db * q4;
    for (int e0 = tid; e0 < n4; e0 += 8 * NT) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = e0 + u * NT;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < n4 && (e % q4) * 4 <= e / q4) v[u] = reinterpret_cast<const float4*>(Gmat + off)[e];
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = e0 + u * NT;
        if (e >= n4) continue;
        const int r = e / q4, c4 = (e % q4) * 4;
        if (c4 > r) continue;
        float* dst = Lp + pm.at(r, c4);         // c4 .. c4 + 3 lie in one panel
        const float vv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (c4 + j <= r) dst[j] = vv[j];
      }
    }
    // right-hand sides: vector id x unknown index
    const int m4 = right ? w * q4 : db * (w / 4);
    for (int e0 = tid; e0 < m4; e0 += 8 * NT) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = e0 + u * NT;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < m4) {
          if (right) v[u] = *reinterpret_cast<const float4*>(rhs + off + (int64_t)(v0 + e / q4) * db + (e % q4) * 4);
          else v[u] = *reinterpret_cast<const float4*>(rhs + off + (int64_t)(e / (w / 4)) * db + v0 + (e % (w / 4)) * 4);
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = e0 + u * NT;
        if (e >= m4) continue;
        const float vv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
        if (right) {
          // right-hand side vid is row v0 + vid of rhs; the unknown index runs along the row
          const int vid = e / q4, r4 = (e % q4) * 4;
#pragma unroll
          for (int j = 0; j < 4; ++j) Rs[(r4 + j) * ldr + vid] = vv[j];
        } else {
          const int r = e / (w / 4), vid4 = (e % (w / 4)) * 4;
#pragma unroll
          for (int j = 0; j < 4; ++j) Rs[r * ldr + vid4 + j] = vv[j];
        }
      }
    }
  }
  if (tid == 0) s_fail = 0;
  __syncthreads();
  if (tid < 32) {
    double tr = 0.0;
    for (int i = tid; i < db; i += 32) tr += (double)Lp[pm.at(i, i)];
    for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
    if (tid == 0) s_lam = (double)ridge * tr / (double)db;
  }
  __syncthreads();
  const double lam = s_lam;
  for (int i = tid; i < db; i += NT) Lp[pm.at(i, i)] = (float)((double)Lp[pm.at(i, i)] + lam);
  __syncthreads();

  // ---- blocked Cholesky
  for (int kb = 0; kb < np; ++kb) {
    const int c0 = NB * kb;
    float* P = Lp + pm.off(kb);
    if (kb > 0) {
      // panel(i, k) -= sum_{p < c0} L(i, p) L(k, p): 4 x 4 tiles, rows c0 + 4*tr.., columns c0 + 4*tc..
      const int ntiles = ((db - c0) / 4) * (NB / 4);
      for (int tix = tid; tix < ntiles; tix += NT) {
        const int tr = tix / (NB / 4), tc = tix % (NB / 4);
        double acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int bb = 0; bb < 4; ++bb) acc[a][bb] = 0.0;
        for (int pb = 0; pb < kb; ++pb) {
          const float* Li = Lp + pm.off(pb) + (c0 + 4 * tr - NB * pb) * LDP;   // rows i of panel pb
          const float* Lk = Lp + pm.off(pb) + (c0 + 4 * tc - NB * pb) * LDP;   // rows k of panel pb
          float a32[4][4];
          ARMOR_TILE_ZERO(a32)
#pragma unroll 8
          for (int p = 0; p < NB; ++p) {
            float li[4], lk[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) { li[a] = Li[a * LDP + p]; lk[a] = Lk[a * LDP + p]; }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
              for (int bb = 0; bb < 4; ++bb) a32[a][bb] = fmaf(li[a], lk[bb], a32[a][bb]);
          }
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) acc[a][bb] += (double)a32[a][bb];
        }
        float* dst = P + (4 * tr) * LDP + 4 * tc;
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int bb = 0; bb < 4; ++bb) dst[a * LDP + bb] = (float)((double)dst[a * LDP + bb] - acc[a][bb]);
      }
      __syncthreads();
    }
    // diagonal block: warp 0, lane i keeps row i in registers and the warp eliminates column by column
    // (right-looking); the entries of the pivot column come from the other lanes by shuffle, so nothing in the
    // chain goes through memory
    if (tid < 32) {
      float arow[NB];
#pragma unroll
      for (int j = 0; j < NB; ++j) arow[j] = (j <= lane) ? P[lane * LDP + j] : 0.f;
      bool bad = false;
#pragma unroll
      for (int k = 0; k < NB; ++k) {
        const float akk = __shfl_sync(0xffffffffu, arow[k], k);
        bad |= !(akk > 0.f) | !isfinite(akk);
        // 1 / sqrt(a): hardware estimate refined by one Newton step
        float inv = rsqrtf(akk);
        inv = inv * fmaf(-0.5f * akk * inv, inv, 1.5f);
        const float lik = (lane == k) ? akk * inv : arow[k] * inv;
        arow[k] = lik;
        if (lane == k) invd[k] = inv;
#pragma unroll
        for (int j = k + 1; j < NB; ++j) {
          const float ljk = __shfl_sync(0xffffffffu, lik, j);
          arow[j] = fmaf(-lik, ljk, arow[j]);      // entries above the diagonal (j > lane) are never used
        }
      }
      if (bad) {
        if (lane == 0) s_fail = 1;
      } else {
#pragma unroll
        for (int j = 0; j < NB; ++j) {
          Df[lane][j] = (j <= lane) ? arow[j] : 0.f;
          if (j <= lane) P[lane * LDP + j] = arow[j];
        }
      }
    }
    __syncthreads();
    if (s_fail) break;
    // rows below the diagonal block: l_ik = (a_ik - sum_{p<k} l_ip l_kp) / l_kk, row i in registers
    const int nrow = db - c0;
    if (tid >= NB && tid < nrow) {   // nrow <= d_block <= 256 = NT
      const int i = tid;
      // column-oriented elimination: once l_ik is final it leaves the later entries of the row at once, so the
      // dependent chain is one multiply-add per column
      float arow[NB];
#pragma unroll
      for (int j = 0; j < NB; ++j) arow[j] = P[i * LDP + j];
#pragma unroll
      for (int k = 0; k < NB; ++k) {
        const float lik = arow[k] * invd[k];
        arow[k] = lik;
#pragma unroll
        for (int j = k + 1; j < NB; ++j) arow[j] = fmaf(-lik, Df[j][k], arow[j]);
      }
#pragma unroll
      for (int j = 0; j < NB; ++j) P[i * LDP + j] = arow[j];
    }
    __syncthreads();
  }
  __syncthreads();
  const bool fail = (s_fail != 0);
  const bool hold = (mode == 0) && status[ST_POISON] != 0;   // unusable inputs: the A-step is withheld (X = 0)

  if (!fail) {
    const int wq = w / 4;          // column c of tile column tc: tc + wq * j  (conflict-free shared-memory rows)
    // ---- forward substitution  L y = r, then backward substitution  L^T x = y
    for (int pass = 0; pass < 2; ++pass) {
      for (int step = 0; step < np; ++step) {
        const int kb = pass == 0 ? step : np - 1 - step;
        const int c0 = NB * kb;
        const float* P = Lp + pm.off(kb);
        // the diagonal block and the reciprocals of its diagonal
        for (int e = tid; e < NB * NB; e += NT) {
          const int r = e / NB, cc = e % NB;
          const float v = (cc <= r) ? P[r * LDP + cc] : 0.f;
          Df[r][cc] = v;
          if (r == cc) invd[r] = 1.f / v;
        }
        if (step > 0) {
          const int ntiles = (NB / 4) * wq;
          for (int tix = tid; tix < ntiles; tix += NT) {
            const int ta = tix / wq, tc = tix % wq;
            double acc[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
              for (int j = 0; j < 4; ++j) acc[a][j] = 0.0;
            if (pass == 0) {
              for (int pb = 0; pb < kb; ++pb) {
                const float* Li = Lp + pm.off(pb) + (c0 + 4 * ta - NB * pb) * LDP;
                const float* Xp = Rs + (NB * pb) * ldr + tc;
                float a32[4][4];
                ARMOR_TILE_ZERO(a32)
#pragma unroll 8
                for (int p = 0; p < NB; ++p) {
                  float li[4], x[4];
#pragma unroll
                  for (int a = 0; a < 4; ++a) { li[a] = Li[a * LDP + p]; x[a] = Xp[p * ldr + wq * a]; }
#pragma unroll
                  for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int j = 0; j < 4; ++j) a32[a][j] = fmaf(li[a], x[j], a32[a][j]);
                }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                  for (int j = 0; j < 4; ++j) acc[a][j] += (double)a32[a][j];
              }
            } else {
              // sum over p >= c0 + NB of L(p, c0 + 4 ta + a) x[p]: column c0 + 4 ta + a lives in panel kb
              const float* Lcol = P + 4 * ta;
              const float* Xp = Rs + tc;
              for (int p0 = c0 + NB; p0 < db; p0 += NB) {
                float a32[4][4];
                ARMOR_TILE_ZERO(a32)
#pragma unroll 8
                for (int p = p0; p < p0 + NB; ++p) {
                  float lc[4], x[4];
#pragma unroll
                  for (int a = 0; a < 4; ++a) { lc[a] = Lcol[(p - c0) * LDP + a]; x[a] = Xp[p * ldr + wq * a]; }
#pragma unroll
                  for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int j = 0; j < 4; ++j) a32[a][j] = fmaf(lc[a], x[j], a32[a][j]);
                }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                  for (int j = 0; j < 4; ++j) acc[a][j] += (double)a32[a][j];
              }
            }
            float* dst = Rs + (c0 + 4 * ta) * ldr + tc;
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
              for (int j = 0; j < 4; ++j) dst[a * ldr + wq * j] = (float)((double)dst[a * ldr + wq * j] - acc[a][j]);
          }
        }
        __syncthreads();
        if (tid < w) {
          float sreg[NB];
#pragma unroll
          for (int r = 0; r < NB; ++r) sreg[r] = Rs[(c0 + r) * ldr + tid];
          if (pass == 0) {
#pragma unroll
            for (int r = 0; r < NB; ++r) {
              const float x = sreg[r] * invd[r];
              sreg[r] = x;
#pragma unroll
              for (int r2 = r + 1; r2 < NB; ++r2) sreg[r2] = fmaf(-Df[r2][r], x, sreg[r2]);
            }
          } else {
#pragma unroll
            for (int r = NB - 1; r >= 0; --r) {
              const float x = sreg[r] * invd[r];
              sreg[r] = x;
#pragma unroll
              for (int r2 = 0; r2 < r; ++r2) sreg[r2] = fmaf(-Df[r][r2], x, sreg[r2]);
            }
          }
#pragma unroll
          for (int r = 0; r < NB; ++r) Rs[(c0 + r) * ldr + tid] = sreg[r];
        }
        __syncthreads();
      }
    }
  }

  // ---- write back.  Right solves: solution vid is row v0 + vid of the result; left solves: column v0 + vid.
  double acc = 0.0;
  {
    const int q4 = db / 4;
    const int m4 = right ? w * q4 : db * (w / 4);
    for (int e0 = tid; e0 < m4; e0 += 4 * NT) {
      float4 x[4], aold[4], gin[4];
      int64_t gidx[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * NT;
        x[u] = aold[u] = gin[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        gidx[u] = -1;
        if (e >= m4) continue;
        if (right) {
          const int vid = e / q4, r4 = (e % q4) * 4;
          gidx[u] = (int64_t)(v0 + vid) * db + r4;
          if (!fail && !hold) x[u] = make_float4(Rs[r4 * ldr + vid], Rs[(r4 + 1) * ldr + vid], Rs[(r4 + 2) * ldr + vid],
                                                 Rs[(r4 + 3) * ldr + vid]);
        } else {
          const int r = e / (w / 4), vid4 = (e % (w / 4)) * 4;
          gidx[u] = (int64_t)r * db + v0 + vid4;
          if (!fail && !hold) x[u] = make_float4(Rs[r * ldr + vid4], Rs[r * ldr + vid4 + 1], Rs[r * ldr + vid4 + 2],
                                                 Rs[r * ldr + vid4 + 3]);
        }
        if (mode == 0) {
          aold[u] = *reinterpret_cast<const float4*>(A + off + gidx[u]);
          gin[u] = *reinterpret_cast<const float4*>(rhs + off + gidx[u]);
        } else if (mode == 2) {
          gin[u] = *reinterpret_cast<const float4*>(dotw + off + gidx[u]);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (gidx[u] < 0) continue;
        *reinterpret_cast<float4*>(out + off + gidx[u]) = x[u];
        if (mode == 0) {
          *reinterpret_cast<float4*>(A + off + gidx[u]) =
              make_float4(aold[u].x + x[u].x, aold[u].y + x[u].y, aold[u].z + x[u].z, aold[u].w + x[u].w);
          acc += (double)gin[u].x * (double)x[u].x + lam * (double)x[u].x * (double)x[u].x;
          acc += (double)gin[u].y * (double)x[u].y + lam * (double)x[u].y * (double)x[u].y;
          acc += (double)gin[u].z * (double)x[u].z + lam * (double)x[u].z * (double)x[u].z;
          acc += (double)gin[u].w * (double)x[u].w + lam * (double)x[u].w * (double)x[u].w;
        } else if (mode == 2) {
          acc += (double)gin[u].x * (double)x[u].x + (double)gin[u].y * (double)x[u].y +
                 (double)gin[u].z * (double)x[u].z + (double)gin[u].w * (double)x[u].w;
        }
      }
    }
  }
  if (mode != 1) {
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) red[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      for (int wp = 0; wp < NT / 32; ++wp) t += red[wp];
      part[(int64_t)b * gridDim.y + q] = t;
    }
  }
  if (tid == 0 && q == 0 && fail) {
    failflag[b] = 1;
    atomicCAS(&status[ST_FIRST_FAIL], 0, b + 1);
  }
}

// Unblocked variant for block sizes that are not a multiple of 32: thread i owns row i.
__global__ void chol_kernel(int mode, const float* __restrict__ Gmat, const float* __restrict__ rhs,
                            float* __restrict__ out, const float* __restrict__ dotw, float* __restrict__ A,
                            float ridge, int db, double* __restrict__ part,
                            int32_t* __restrict__ failflag, int32_t* __restrict__ status) {
  extern __shared__ float smem[];
  const int ld = db + 1;
  float* L = smem;
  float* Rs = smem + (size_t)db * ld;
  __shared__ double red[8];
  __shared__ float s_diag;
  __shared__ int s_fail;
  __shared__ double s_lam;
  const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const int64_t off = (int64_t)b * db * db;
  const bool right = (mode != 1);
  for (int e = tid; e < db * db; e += nt) {
    const int r = e / db, cidx = e % db;
    L[r * ld + cidx] = Gmat[off + e];
    const float v = rhs[off + e];
    if (right) Rs[cidx * ld + r] = v; else Rs[r * ld + cidx] = v;
  }
  if (tid == 0) s_fail = 0;
  __syncthreads();
  if (tid == 0) {
    double tr = 0.0;
    for (int i = 0; i < db; ++i) tr += (double)L[i * ld + i];
    s_lam = (double)ridge * tr / (double)db;
  }
  __syncthreads();
  const double lam = s_lam;
  if (tid < db) L[tid * ld + tid] = (float)((double)L[tid * ld + tid] + lam);
  __syncthreads();

  const int i = tid;
  for (int k = 0; k < db; ++k) {
    double s = 0.0;
    if (i >= k && i < db) {
      s = (double)L[i * ld + k];
      for (int p = 0; p < k; ++p) s -= (double)L[i * ld + p] * (double)L[k * ld + p];
      if (i == k) {
        if (!(s > 0.0) || !isfinite(s)) s_fail = 1; else s_diag = (float)sqrt(s);
      }
    }
    __syncthreads();
    if (s_fail) break;
    if (i >= k && i < db) L[i * ld + k] = (i == k) ? s_diag : (float)(s / (double)s_diag);
    __syncthreads();
  }
  const bool fail = (s_fail != 0);
  const bool hold = (mode == 0) && status[ST_POISON] != 0;   // unusable inputs: the A-step is withheld (X = 0)

  double acc = 0.0;
  if (!fail) {
    const int cidx = tid;
    if (cidx < db) {
      for (int r = 0; r < db; ++r) {
        double s = (double)Rs[r * ld + cidx];
        for (int p = 0; p < r; ++p) s -= (double)L[r * ld + p] * (double)Rs[p * ld + cidx];
        Rs[r * ld + cidx] = (float)(s / (double)L[r * ld + r]);
      }
      for (int r = db - 1; r >= 0; --r) {
        double s = (double)Rs[r * ld + cidx];
        for (int p = r + 1; p < db; ++p) s -= (double)L[p * ld + r] * (double)Rs[p * ld + cidx];
        Rs[r * ld + cidx] = (float)(s / (double)L[r * ld + r]);
      }
    }
  }
  __syncthreads();
  for (int e = tid; e < db * db; e += nt) {
    const int r = e / db, cidx = e % db;
    float x = 0.f;
    if (!fail && !hold) x = right ? Rs[cidx * ld + r] : Rs[r * ld + cidx];
    if (mode == 0) {
      const float a = A[off + e] + x;
      A[off + e] = a;
      out[off + e] = x;
      acc += (double)rhs[off + e] * (double)x + lam * (double)x * (double)x;
    } else {
      out[off + e] = x;
      if (mode == 2) acc += (double)dotw[off + e] * (double)x;
    }
  }
  if (mode != 1) {
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) red[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      for (int w = 0; w < (nt + 31) / 32; ++w) t += red[w];
      part[b] = t;
    }
  }
  if (tid == 0 && fail) {
    failflag[b] = 1;
    atomicCAS(&status[ST_FIRST_FAIL], 0, b + 1);
  }
}

}  // namespace

// Right-hand sides of one block are split over this many CTAs (each repeats the factorisation).  d_block 256
// needs 4 for its shared memory; smaller blocks are split while that still fits one wave of CTAs.
int chol_parts_per_block(int db, int nb) {
  if (db % NB) return 1;
  if (db > 128) return db / 64;
  int parts = 1;
  while (parts < 4 && 2 * parts * nb <= 148 && db / (2 * parts) >= 32) parts *= 2;
  return parts;
}

armor_status launch_chol(armor_ctx* c, int mode, const float* Gmat, const float* rhs, float* out, const float* dotw,
                         float* A, int nb, double* part, cudaStream_t s) {
  const int db = c->db;
  KTimer kt(c, ARMOR_KC_CHOLESKY, (double)nb * (7.0 / 3.0) * (double)db * (double)db * (double)db, s);   // flops
  if (db % NB == 0) {
    const int slices = chol_parts_per_block(db, nb);
    const int w = db / slices;
    const size_t smem = (panel_floats(db) + (size_t)db * (w + 1)) * sizeof(float);
    static size_t attr_bytes[64] = {};   // per device: the limit set so far
    const int dv = (c->device >= 0 && c->device < 64) ? c->device : 0;
    if (smem > attr_bytes[dv] || c->device != dv) {
      if (cudaFuncSetAttribute(chol_blocked_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
          cudaSuccess)
        return ARMOR_ERR_CUDA;
      attr_bytes[dv] = smem;
    }
    chol_blocked_kernel<<<dim3(nb, slices), NT, smem, s>>>(mode, Gmat, rhs, out, dotw, A, c->cfg.ridge, db, w,
                                                          part, c->failflag, c->status);
    c->launches++;
    return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
  }
  const size_t smem = 2 * (size_t)db * (db + 1) * sizeof(float);
  static PerDeviceOnce attr_set;
  if (ensure_dynamic_smem(attr_set, c->device, chol_kernel, 2 * 128 * 129 * 4) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int nt = ((db + 31) / 32) * 32;
  chol_kernel<<<nb, nt < 64 ? 64 : nt, smem, s>>>(mode, Gmat, rhs, out, dotw, A, c->cfg.ridge, db, part,
                                                 c->failflag, c->status);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

namespace {

__global__ void identity_rhs_kernel(float* __restrict__ X, int db) {
  float* Xb = X + (int64_t)blockIdx.x * db * db;
  for (int e = threadIdx.x; e < db * db; e += blockDim.x) Xb[e] = (e / db == e % db) ? 1.f : 0.f;
}

__global__ void save_flags_kernel(const int32_t* __restrict__ failflag, int32_t* __restrict__ saved, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) saved[i] = failflag[i];
}

// one CTA per block: Delta_j = 0 and failflag[j] = 1 where the inverse does not exist; part[j] = <dotw_j, Delta_j>
__global__ void __launch_bounds__(NT) delta_finish_kernel(float* __restrict__ Delta, const float* __restrict__ dotw,
                                                          const int32_t* __restrict__ hinv_fail,
                                                          int32_t* __restrict__ failflag, double* __restrict__ part,
                                                          int db) {
  const int j = blockIdx.x;
  const int64_t off = (int64_t)j * db * db;
  const bool bad = hinv_fail[j] != 0;
  double acc = 0.0;
  for (int e = threadIdx.x; e < db * db; e += NT) {
    if (bad) Delta[off + e] = 0.f;
    else acc += (double)dotw[off + e] * (double)Delta[off + e];
  }
  __shared__ double red[NT / 32];
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < NT / 32; ++w) t += red[w];
    part[j] = t;
    if (bad) failflag[j] = 1;
  }
}

}  // namespace

armor_status launch_hjj_inverse(armor_ctx* c, cudaStream_t s) {
  const int nbi = c->nbi;
  if (cudaMemsetAsync(c->failflag, 0, (size_t)nbi * sizeof(int32_t), s) != cudaSuccess) return ARMOR_ERR_CUDA;
  {
    KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
    identity_rhs_kernel<<<nbi, NT, 0, s>>>(c->Ktmp, c->db);
    c->launches++;
  }
  armor_status st = launch_chol(c, 1, c->Hjj, c->Ktmp, c->Hinv, nullptr, nullptr, nbi, nullptr, s);
  if (st != ARMOR_OK) return st;
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  save_flags_kernel<<<(nbi + 255) / 256, 256, 0, s>>>(c->failflag, c->hinv_fail, nbi);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

void launch_delta_finish(armor_ctx* c, float* Delta, const float* dotw, double* part, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  delta_finish_kernel<<<c->nbi, NT, 0, s>>>(Delta, dotw, c->hinv_fail, c->failflag, part, c->db);
  c->launches++;
}

