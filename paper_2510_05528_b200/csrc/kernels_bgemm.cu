// Strided batched fp32 GEMM on CUDA cores, and the block-diagonal products built on it.
//
// Products with the block-diagonal wrappers (Section 3.1 of the paper: A and B are stored as
// [nb, d_block, d_block] and applied as batched matrix products) have 2*d_block flops per element of
// the W-shaped operand; they are evaluated in plain fp32 so that only the dense .H contractions
// carry tensor-core rounding.
#include "armor_internal.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4, NT = 256;

__global__ void __launch_bounds__(NT) bgemm_kernel(BGemm g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int b = blockIdx.z;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const float* __restrict__ A = g.A + (int64_t)b * g.sAb;
  const float* __restrict__ B = g.B + (int64_t)b * g.sBb;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  // which index runs fastest over consecutive threads when a tile is fetched: the unit-stride one
  const bool a_k_fast = (g.sAk == 1);
  const bool b_n_fast = (g.sBn == 1);
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
    for (int e = 0; e < (BM * BK) / NT; ++e) {
      int idx = tid + e * NT;
      int m, k;
      if (a_k_fast) { k = idx % BK; m = idx / BK; } else { m = idx % BM; k = idx / BM; }
      float v = 0.f;
      if (m0 + m < g.M && k0 + k < g.K) v = A[(int64_t)(m0 + m) * g.sAm + (int64_t)(k0 + k) * g.sAk];
      As[k][m] = v;
    }
#pragma unroll
    for (int e = 0; e < (BN * BK) / NT; ++e) {
      int idx = tid + e * NT;
      int n, k;
      if (b_n_fast) { n = idx % BN; k = idx / BN; } else { k = idx % BK; n = idx / BK; }
      float v = 0.f;
      if (n0 + n < g.N && k0 + k < g.K) v = B[(int64_t)(k0 + k) * g.sBk + (int64_t)(n0 + n) * g.sBn];
      Bs[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * TM]);
      float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * TN]);
      float a[TM] = {a4.x, a4.y, a4.z, a4.w};
      float bb[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* C = g.C + (int64_t)b * g.sCb;
  const float* D = g.D ? g.D + (int64_t)b * g.sDb : nullptr;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    int m = m0 + ty * TM + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      int n = n0 + tx * TN + j;
      if (n >= g.N) continue;
      float v = g.alpha * acc[i][j];
      if (D) v += g.beta * D[(int64_t)m * g.sDm + (int64_t)n * g.sDn];
      C[(int64_t)m * g.sCm + (int64_t)n * g.sCn] = v;
    }
  }
}

}  // namespace

void launch_bgemm(armor_ctx* c, const BGemm& g, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  bgemm_kernel<<<grid, NT, 0, s>>>(g);
  c->launches++;
}

void bd_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
              int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  const int db = c->db;
  BGemm g{};
  g.A = in; g.sAb = db; g.sAm = cols; g.sAk = 1;
  g.B = Bblk; g.sBb = (int64_t)db * db;
  if (transB) { g.sBk = 1; g.sBn = db; } else { g.sBk = db; g.sBn = 1; }
  g.C = out; g.sCb = db; g.sCm = cols; g.sCn = 1;
  g.D = add; g.sDb = db; g.sDm = cols; g.sDn = 1;
  g.M = (int)rows; g.N = db; g.K = db; g.batch = (int)(cols / db);
  g.alpha = alpha; g.beta = beta;
  launch_bgemm(c, g, s);
}

void bd_left(armor_ctx* c, const float* Ablk, bool transA, const float* in, float* out, int64_t rows,
             int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  const int db = c->db;
  BGemm g{};
  g.A = Ablk; g.sAb = (int64_t)db * db;
  if (transA) { g.sAm = 1; g.sAk = db; } else { g.sAm = db; g.sAk = 1; }
  g.B = in; g.sBb = (int64_t)db * cols; g.sBk = cols; g.sBn = 1;
  g.C = out; g.sCb = (int64_t)db * cols; g.sCm = cols; g.sCn = 1;
  g.D = add; g.sDb = (int64_t)db * cols; g.sDm = cols; g.sDn = 1;
  g.M = db; g.N = (int)cols; g.K = db; g.batch = (int)(rows / db);
  g.alpha = alpha; g.beta = beta;
  launch_bgemm(c, g, s);
}
