// Per-block SPD solves for the wrapper updates.  The block systems are the zeros of the paper's
// gradients with respect to A and B (Appendix D.1 and D.2) made proximal by a relative ridge:
//   mode 0 (A update): X = Gamma (G + lam I)^-1;  A += X;  At = A^T;  dA = X;  part = <Gamma, X> + lam |X|^2
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

__global__ void __launch_bounds__(NT, 1)
chol_blocked_kernel(int mode, const float* __restrict__ Gmat, const float* __restrict__ rhs, float* __restrict__ out,
                    const float* __restrict__ dotw, float* __restrict__ A, float* __restrict__ At, float ridge, int db,
                    int w, double* __restrict__ part, int32_t* __restrict__ failflag, int32_t* __restrict__ status) {
  extern __shared__ float smem[];
  const PanelMap pm{db};
  const int np = db / NB;
  const int ldr = w + 1;
  float* Lp = smem;
  float* Rs = smem + panel_floats(db);                  // [db][w + 1]: row = unknown index, column = right-hand side
  double* invd = reinterpret_cast<double*>(smem + ((panel_floats(db) + (size_t)db * ldr + 1) & ~(size_t)1));  // [db]
  __shared__ double red[NT / 32];
  __shared__ float s_diag;
  __shared__ int s_fail;
  __shared__ double s_lam;
  const int b = blockIdx.x, q = blockIdx.y, tid = threadIdx.x;
  const int64_t off = (int64_t)b * db * db;
  const bool right = (mode != 1);
  const int v0 = q * w;  // first right-hand side of this CTA

  // ---- load: lower triangle of G, the slice of right-hand sides
  for (int e = tid; e < db * db; e += NT) {
    const int r = e / db, cidx = e % db;
    if (cidx <= r) Lp[pm.at(r, cidx)] = Gmat[off + e];
  }
  if (right) {
    // right-hand side v is row v0 + v of rhs; unknown index r runs along the row
    for (int e = tid; e < w * db; e += NT) {
      const int v = e / db, r = e % db;
      Rs[r * ldr + v] = rhs[off + (int64_t)(v0 + v) * db + r];
    }
  } else {
    for (int e = tid; e < db * w; e += NT) {
      const int r = e / w, v = e % w;
      Rs[r * ldr + v] = rhs[off + (int64_t)r * db + v0 + v];
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
#pragma unroll 4
          for (int p = 0; p < NB; ++p) {
            double li[4], lk[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) { li[a] = (double)Li[a * LDP + p]; lk[a] = (double)Lk[a * LDP + p]; }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
              for (int bb = 0; bb < 4; ++bb) acc[a][bb] = fma(li[a], lk[bb], acc[a][bb]);
          }
        }
        float* dst = Lp + pm.off(kb) + (4 * tr) * LDP + 4 * tc;
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int bb = 0; bb < 4; ++bb) dst[a * LDP + bb] = (float)((double)dst[a * LDP + bb] - acc[a][bb]);
      }
      __syncthreads();
    }
    // eliminate the 32 columns of the panel; thread i owns row c0 + i of the panel
    float* P = Lp + pm.off(kb);
    const int nrow = db - c0;
    for (int k = 0; k < NB; ++k) {
      double s = 0.0;
      if (tid >= k && tid < nrow) {
        s = (double)P[tid * LDP + k];
        double s1 = 0.0;
        int p = 0;
        for (; p + 1 < k; p += 2) {
          s = fma(-(double)P[tid * LDP + p], (double)P[k * LDP + p], s);
          s1 = fma(-(double)P[tid * LDP + p + 1], (double)P[k * LDP + p + 1], s1);
        }
        if (p < k) s = fma(-(double)P[tid * LDP + p], (double)P[k * LDP + p], s);
        s += s1;
        if (tid == k) {
          if (!(s > 0.0) || !isfinite(s)) s_fail = 1; else s_diag = (float)sqrt(s);
        }
      }
      __syncthreads();
      if (s_fail) break;
      if (tid >= k && tid < nrow) P[tid * LDP + k] = (tid == k) ? s_diag : (float)(s / (double)s_diag);
      __syncthreads();
    }
    if (s_fail) break;
  }
  __syncthreads();
  const bool fail = (s_fail != 0);

  if (!fail) {
    for (int i = tid; i < db; i += NT) invd[i] = 1.0 / (double)Lp[pm.at(i, i)];
    __syncthreads();
    const int wq = w / 4;          // column c of tile column tc: tc + wq * j  (conflict-free shared-memory rows)
    // ---- forward substitution  L y = r
    for (int kb = 0; kb < np; ++kb) {
      const int c0 = NB * kb;
      if (kb > 0) {
        const int ntiles = (NB / 4) * wq;
        for (int tix = tid; tix < ntiles; tix += NT) {
          const int ta = tix / wq, tc = tix % wq;
          double acc[4][4];
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[a][j] = 0.0;
          for (int pb = 0; pb < kb; ++pb) {
            const float* Li = Lp + pm.off(pb) + (c0 + 4 * ta - NB * pb) * LDP;
            const float* Xp = Rs + (NB * pb) * ldr + tc;
#pragma unroll 4
            for (int p = 0; p < NB; ++p) {
              double li[4], x[4];
#pragma unroll
              for (int a = 0; a < 4; ++a) { li[a] = (double)Li[a * LDP + p]; x[a] = (double)Xp[p * ldr + wq * a]; }
#pragma unroll
              for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[a][j] = fma(li[a], x[j], acc[a][j]);
            }
          }
          float* dst = Rs + (c0 + 4 * ta) * ldr + tc;
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[a * ldr + wq * j] = (float)((double)dst[a * ldr + wq * j] - acc[a][j]);
        }
        __syncthreads();
      }
      if (tid < w) {
        const float* D = Lp + pm.off(kb);   // diagonal block: rows 0..31 of the panel
        double sreg[NB];
#pragma unroll
        for (int r = 0; r < NB; ++r) sreg[r] = (double)Rs[(c0 + r) * ldr + tid];
#pragma unroll
        for (int r = 0; r < NB; ++r) {
          const double x = sreg[r] * invd[c0 + r];
          sreg[r] = x;
#pragma unroll
          for (int r2 = r + 1; r2 < NB; ++r2) sreg[r2] = fma(-(double)D[r2 * LDP + r], x, sreg[r2]);
        }
#pragma unroll
        for (int r = 0; r < NB; ++r) Rs[(c0 + r) * ldr + tid] = (float)sreg[r];
      }
      __syncthreads();
    }
    // ---- backward substitution  L^T x = y
    for (int kb = np - 1; kb >= 0; --kb) {
      const int c0 = NB * kb;
      if (kb < np - 1) {
        const int ntiles = (NB / 4) * wq;
        for (int tix = tid; tix < ntiles; tix += NT) {
          const int ta = tix / wq, tc = tix % wq;
          double acc[4][4];
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[a][j] = 0.0;
          // sum over p >= c0 + NB of L(p, c0 + 4 ta + a) x[p]: column c0 + 4 ta + a lives in panel kb
          const float* Lcol = Lp + pm.off(kb) + 4 * ta;
          const float* Xp = Rs + tc;
#pragma unroll 4
          for (int p = c0 + NB; p < db; ++p) {
            double lc[4], x[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) { lc[a] = (double)Lcol[(p - c0) * LDP + a]; x[a] = (double)Xp[p * ldr + wq * a]; }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
              for (int j = 0; j < 4; ++j) acc[a][j] = fma(lc[a], x[j], acc[a][j]);
          }
          float* dst = Rs + (c0 + 4 * ta) * ldr + tc;
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[a * ldr + wq * j] = (float)((double)dst[a * ldr + wq * j] - acc[a][j]);
        }
        __syncthreads();
      }
      if (tid < w) {
        const float* D = Lp + pm.off(kb);
        double sreg[NB];
#pragma unroll
        for (int r = 0; r < NB; ++r) sreg[r] = (double)Rs[(c0 + r) * ldr + tid];
#pragma unroll
        for (int r = NB - 1; r >= 0; --r) {
          const double x = sreg[r] * invd[c0 + r];
          sreg[r] = x;
#pragma unroll
          for (int r2 = 0; r2 < r; ++r2) sreg[r2] = fma(-(double)D[r * LDP + r2], x, sreg[r2]);
        }
#pragma unroll
        for (int r = 0; r < NB; ++r) Rs[(c0 + r) * ldr + tid] = (float)sreg[r];
      }
      __syncthreads();
    }
  }

  // ---- write back.  Right solves: solution v is row v0 + v of the result; left solves: column v0 + v.
  double acc = 0.0;
  const int n_el = db * w;
  for (int e = tid; e < n_el; e += NT) {
    int r, v;
    int64_t g;     // element of the [db][db] result
    if (right) { v = e / db; r = e % db; g = (int64_t)(v0 + v) * db + r; }
    else       { r = e / w;  v = e % w;  g = (int64_t)r * db + v0 + v; }
    const float x = fail ? 0.f : Rs[r * ldr + v];
    if (mode == 0) {
      const float a = A[off + g] + x;
      A[off + g] = a;
      At[off + (int64_t)r * db + (v0 + v)] = a;
      out[off + g] = x;
      acc += (double)rhs[off + g] * (double)x + lam * (double)x * (double)x;
    } else {
      out[off + g] = x;
      if (mode == 2) acc += (double)dotw[off + g] * (double)x;
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
                            float* __restrict__ At, float ridge, int db, double* __restrict__ part,
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
    if (!fail) x = right ? Rs[cidx * ld + r] : Rs[r * ld + cidx];
    if (mode == 0) {
      const float a = A[off + e] + x;
      A[off + e] = a;
      At[off + (int64_t)cidx * db + r] = a;
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

int chol_parts_per_block(int db) { return (db % NB == 0 && db > 128) ? db / 64 : 1; }

armor_status launch_chol(armor_ctx* c, int mode, const float* Gmat, const float* rhs, float* out, const float* dotw,
                         float* A, float* At, int nb, double* part, cudaStream_t s) {
  const int db = c->db;
  if (db % NB == 0) {
    const int slices = chol_parts_per_block(db);
    const int w = db / slices;
    const size_t smem = ((panel_floats(db) + (size_t)db * (w + 1) + 1) & ~(size_t)1) * sizeof(float) +
                        (size_t)db * sizeof(double);
    static size_t attr_bytes = 0;
    if (smem > attr_bytes) {
      if (cudaFuncSetAttribute(chol_blocked_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
          cudaSuccess)
        return ARMOR_ERR_CUDA;
      attr_bytes = smem;
    }
    chol_blocked_kernel<<<dim3(nb, slices), NT, smem, s>>>(mode, Gmat, rhs, out, dotw, A, At, c->cfg.ridge, db, w,
                                                          part, c->failflag, c->status);
    c->launches++;
    return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
  }
  const size_t smem = 2 * (size_t)db * (db + 1) * sizeof(float);
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(chol_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 128 * 129 * 4) != cudaSuccess)
      return ARMOR_ERR_CUDA;
    attr_set = true;
  }
  const int nt = ((db + 31) / 32) * 32;
  chol_kernel<<<nb, nt < 64 ? 64 : nt, smem, s>>>(mode, Gmat, rhs, out, dotw, A, At, c->cfg.ridge, db, part,
                                                 c->failflag, c->status);
  c->launches++;
  return ARMOR_OK;
}
