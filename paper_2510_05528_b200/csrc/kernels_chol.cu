// Per-block SPD solves for the wrapper updates: one CTA per d_block x d_block block, the matrix and
// the right-hand side resident in shared memory, Cholesky factorisation followed by two triangular
// solves.  The block systems are the zeros of the paper's gradients with respect to A and B
// (Appendix D.1 and D.2) made proximal by a relative ridge.
#include "armor_internal.cuh"

namespace {

// mode 0 (A update): X = Gamma (G + lam I)^-1;  A += X;  At = A^T;  dA = X;  part = <Gamma, X> + lam |X|^2
// mode 1 (left)    : out = (G + lam I)^-1 rhs
// mode 2 (right+gd): out = rhs (G + lam I)^-1;  part = <dotw, out>
// A failed factorisation leaves A unchanged / writes zeros and raises failflag[block].
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

  // left-looking Cholesky; thread i owns row i
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
    const int cidx = tid;  // thread c owns column c of Rs
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
  // write back (row-major [r][c] of the result); for right solves the result sits transposed in Rs
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

armor_status launch_chol(armor_ctx* c, int mode, const float* Gmat, const float* rhs, float* out, const float* dotw,
                         float* A, float* At, int nb, double* part, cudaStream_t s) {
  const int db = c->db;
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
