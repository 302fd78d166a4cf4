// Strided batched fp32 GEMM on CUDA cores, and the block-diagonal products built on it.
//
// Products with the block-diagonal wrappers (Section 3.1 of the paper: A and B are stored as
// [nb, d_block, d_block] and applied as batched matrix products) have 2*d_block flops per element of
// the W-shaped operand; they are evaluated in plain fp32 so that only the dense .H contractions
// carry tensor-core rounding.
//
// Two kernels: bgemm_tile_kernel (128 x 128 x 16 tiles, 8 x 8 accumulators per thread, float4 global
// loads along whichever index of an operand is contiguous, register-prefetch double buffering) for
// aligned shapes, and bgemm_kernel (64 x 64, any strides, any sizes) for the rest.
#include "armor_internal.cuh"

namespace {

// ------------------------------------------------------------------------------ general fallback
constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4, NT = 256;

__device__ __forceinline__ void batch_offsets(const BGemm& g, int b, int64_t& oa, int64_t& ob, int64_t& oc, int64_t& od) {
  if (g.batch_inner > 0) {
    const int bo = b / g.batch_inner, bi = b % g.batch_inner;
    oa = (int64_t)bo * g.sAb2 + (int64_t)bi * g.sAb;
    ob = (int64_t)bo * g.sBb2 + (int64_t)bi * g.sBb;
    oc = (int64_t)bo * g.sCb2 + (int64_t)bi * g.sCb;
    od = (int64_t)bo * g.sDb2 + (int64_t)bi * g.sDb;
  } else {
    oa = (int64_t)b * g.sAb; ob = (int64_t)b * g.sBb; oc = (int64_t)b * g.sCb; od = (int64_t)b * g.sDb;
  }
}

__global__ void __launch_bounds__(NT) bgemm_kernel(BGemm g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int b = blockIdx.z;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  int64_t oa, ob, oc, od;
  batch_offsets(g, b, oa, ob, oc, od);
  const float* __restrict__ A = g.A + oa;
  const float* __restrict__ B = g.B + ob;
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
  float* C = g.C + oc;
  const float* D = g.D ? g.D + od : nullptr;
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

// ------------------------------------------------------------------------------ tiled kernel
constexpr int FM = 128, FN = 128, FK = 16, FLD = FM + 4;

// A_KFAST: element (m, k) of A is contiguous in k (sAk == 1), else contiguous in m (sAm == 1).
// B_NFAST: element (k, n) of B is contiguous in n (sBn == 1), else contiguous in k (sBk == 1).
// Requirements (checked by the launcher): K chunk a multiple of 16, M and N multiples of 4, the non-unit
// strides and all batch strides multiples of 4, 16-byte aligned bases, sCn == sDn == 1.
template <bool A_KFAST, bool B_NFAST>
__global__ void __launch_bounds__(NT, 2) bgemm_tile_kernel(BGemm g, float* __restrict__ part_out, int64_t part_stride) {
  __shared__ __align__(16) float As[2][FK][FLD];
  __shared__ __align__(16) float Bs[2][FK][FLD];
  const int ksplit = g.ksplit > 1 ? g.ksplit : 1;
  const int b = blockIdx.z / ksplit, ks = blockIdx.z % ksplit;
  const int m0 = blockIdx.y * FM, n0 = blockIdx.x * FN;
  int64_t oa, ob, oc, od;
  batch_offsets(g, b, oa, ob, oc, od);
  const int kc = g.K / ksplit;
  const float* __restrict__ A = g.A + oa + (int64_t)ks * kc * g.sAk;
  const float* __restrict__ B = g.B + ob + (int64_t)ks * kc * g.sBk;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;

  // global -> register fetch of one K step
  float4 ra[2], rb[2];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int f = tid + e * NT;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (A_KFAST) {
        const int m = f >> 2, kq = f & 3;
        if (m0 + m < g.M) v = *reinterpret_cast<const float4*>(A + (int64_t)(m0 + m) * g.sAm + k0 + 4 * kq);
      } else {
        const int k = f >> 5, mq = f & 31;
        if (m0 + 4 * mq < g.M) v = *reinterpret_cast<const float4*>(A + (int64_t)(k0 + k) * g.sAk + m0 + 4 * mq);
      }
      ra[e] = v;
      v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (B_NFAST) {
        const int k = f >> 5, nq = f & 31;
        if (n0 + 4 * nq < g.N) v = *reinterpret_cast<const float4*>(B + (int64_t)(k0 + k) * g.sBk + n0 + 4 * nq);
      } else {
        const int n = f >> 2, kq = f & 3;
        if (n0 + n < g.N) v = *reinterpret_cast<const float4*>(B + (int64_t)(n0 + n) * g.sBn + k0 + 4 * kq);
      }
      rb[e] = v;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int f = tid + e * NT;
      if (A_KFAST) {
        const int m = f >> 2, kq = f & 3;
        As[buf][4 * kq + 0][m] = ra[e].x; As[buf][4 * kq + 1][m] = ra[e].y;
        As[buf][4 * kq + 2][m] = ra[e].z; As[buf][4 * kq + 3][m] = ra[e].w;
      } else {
        const int k = f >> 5, mq = f & 31;
        *reinterpret_cast<float4*>(&As[buf][k][4 * mq]) = ra[e];
      }
      if (B_NFAST) {
        const int k = f >> 5, nq = f & 31;
        *reinterpret_cast<float4*>(&Bs[buf][k][4 * nq]) = rb[e];
      } else {
        const int n = f >> 2, kq = f & 3;
        Bs[buf][4 * kq + 0][n] = rb[e].x; Bs[buf][4 * kq + 1][n] = rb[e].y;
        Bs[buf][4 * kq + 2][n] = rb[e].z; Bs[buf][4 * kq + 3][n] = rb[e].w;
      }
    }
  };

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  const int nk = kc / FK;
  fetch(0);
  stash(0);
  __syncthreads();
  int cur = 0;
  for (int kt = 0; kt < nk; ++kt) {
    if (kt + 1 < nk) fetch((kt + 1) * FK);
#pragma unroll
    for (int k = 0; k < FK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[cur][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[cur][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[cur][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[cur][k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    if (kt + 1 < nk) stash(cur ^ 1);
    __syncthreads();
    cur ^= 1;
  }

  // epilogue: rows ty*4 + i (+64), columns tx*4 .. +3 (+64)
  float* C;
  int64_t ldc;
  if (ksplit > 1) {
    C = part_out + (int64_t)ks * part_stride + (int64_t)b * g.M * g.N;
    ldc = g.N;
  } else {
    C = g.C + oc;
    ldc = g.sCm;
  }
  const float* D = (g.D && ksplit == 1) ? g.D + od : nullptr;
  const float alpha = (ksplit > 1) ? 1.f : g.alpha;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + i - 4);
    if (m >= g.M) continue;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int n = n0 + h * 64 + tx * 4;
      if (n >= g.N) continue;
      float4 v = make_float4(alpha * acc[i][4 * h + 0], alpha * acc[i][4 * h + 1], alpha * acc[i][4 * h + 2],
                             alpha * acc[i][4 * h + 3]);
      if (D) {
        const float4 d = *reinterpret_cast<const float4*>(D + (int64_t)m * g.sDm + n);
        v.x = fmaf(g.beta, d.x, v.x); v.y = fmaf(g.beta, d.y, v.y);
        v.z = fmaf(g.beta, d.z, v.z); v.w = fmaf(g.beta, d.w, v.w);
      }
      *reinterpret_cast<float4*>(C + (int64_t)m * ldc + n) = v;
    }
  }
}

// out[b][m][n] = alpha * sum_ks part[ks][b][m][n]  (fixed order), scattered to the strided destination
__global__ void __launch_bounds__(NT) bgemm_splitsum_kernel(BGemm g, const float* __restrict__ part,
                                                            int64_t part_stride) {
  const int64_t per = (int64_t)g.M * g.N;
  const int64_t n4 = (int64_t)g.batch * per / 4;
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n4; i += (int64_t)gridDim.x * NT) {
    float4 acc = reinterpret_cast<const float4*>(part)[i];
    for (int ks = 1; ks < g.ksplit; ++ks) {
      const float4 v = reinterpret_cast<const float4*>(part + (int64_t)ks * part_stride)[i];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    const int64_t e = i * 4;
    const int b = (int)(e / per);
    const int64_t r = e % per;
    const int m = (int)(r / g.N), n = (int)(r % g.N);
    int64_t oa, ob, oc, od;
    batch_offsets(g, b, oa, ob, oc, od);
    *reinterpret_cast<float4*>(g.C + oc + (int64_t)m * g.sCm + n) =
        make_float4(g.alpha * acc.x, g.alpha * acc.y, g.alpha * acc.z, g.alpha * acc.w);
  }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

bool tile_kernel_ok(const BGemm& g, bool& a_kfast, bool& b_nfast) {
  if (g.M % 4 || g.N % 4) return false;
  const int ks = g.ksplit > 1 ? g.ksplit : 1;
  if (g.K % (16 * ks)) return false;
  if (g.sCn != 1 || (g.D && g.sDn != 1)) return false;
  if (g.sAk == 1) a_kfast = true; else if (g.sAm == 1) a_kfast = false; else return false;
  if (g.sBn == 1) b_nfast = true; else if (g.sBk == 1) b_nfast = false; else return false;
  const int64_t strides[] = {a_kfast ? g.sAm : g.sAk, b_nfast ? g.sBk : g.sBn, g.sCm, g.D ? g.sDm : 0,
                             g.sAb, g.sBb, g.sCb, g.D ? g.sDb : 0, g.sAb2, g.sBb2, g.sCb2, g.D ? g.sDb2 : 0};
  for (int64_t st : strides)
    if (st % 4) return false;
  if (!aligned16(g.A) || !aligned16(g.B) || !aligned16(g.C) || (g.D && !aligned16(g.D))) return false;
  return true;
}

}  // namespace

void launch_bgemm(armor_ctx* c, const BGemm& g_in, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);   // CUDA-core products: small block systems, or every product of a SIMT run
  BGemm g = g_in;
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return;
  if (g.ksplit > 1 && (g.D || !c->gpart || (int64_t)g.ksplit * g.batch * g.M * g.N > c->gpart_floats)) g.ksplit = 1;
  bool a_kfast = false, b_nfast = false;
  if (g.ksplit > 1 && !tile_kernel_ok(g, a_kfast, b_nfast)) g.ksplit = 1;
  if (tile_kernel_ok(g, a_kfast, b_nfast)) {
    const int ks = g.ksplit > 1 ? g.ksplit : 1;
    dim3 grid((g.N + FN - 1) / FN, (g.M + FM - 1) / FM, g.batch * ks);
    const int64_t pstride = (int64_t)g.batch * g.M * g.N;
    if (a_kfast && b_nfast) bgemm_tile_kernel<true, true><<<grid, NT, 0, s>>>(g, c->gpart, pstride);
    else if (a_kfast && !b_nfast) bgemm_tile_kernel<true, false><<<grid, NT, 0, s>>>(g, c->gpart, pstride);
    else if (!a_kfast && b_nfast) bgemm_tile_kernel<false, true><<<grid, NT, 0, s>>>(g, c->gpart, pstride);
    else bgemm_tile_kernel<false, false><<<grid, NT, 0, s>>>(g, c->gpart, pstride);
    c->launches++;
    if (ks > 1) {
      const int64_t n4 = pstride / 4;
      int64_t blocks = (n4 + NT - 1) / NT;
      if (blocks > 148 * 8) blocks = 148 * 8;
      bgemm_splitsum_kernel<<<(unsigned)blocks, NT, 0, s>>>(g, c->gpart, pstride);
      c->launches++;
    }
    return;
  }
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  bgemm_kernel<<<grid, NT, 0, s>>>(g);
  c->launches++;
}

void bd_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
              int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  if (c->tc_blocks && tc_block_ok(c, rows, cols) &&
      tc_done(c, tc_bd_right(c, in, Bblk, transB, out, rows, cols, alpha, add, beta, s)))
    return;
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
  if (c->tc_blocks && tc_block_ok(c, rows, cols) &&
      tc_done(c, tc_bd_left(c, Ablk, transA, in, out, rows, cols, alpha, add, beta, s)))
    return;
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

void bd_two_sided(armor_ctx* c, const float* Lblk, bool transL, const float* X, const float* Rblk, bool transR, float* tmp,
                  float* out, int64_t rows, int64_t cols, float alpha, cudaStream_t s) {
  if (c->tc_blocks == 3 && tc_block2_ok(c, rows, cols) &&
      tc_done(c, tc_two_sided(c, Lblk, transL, X, Rblk, transR, out, rows, cols, alpha, s)))
    return;
  bd_left(c, Lblk, transL, X, tmp, rows, cols, 1.f, nullptr, 0.f, s);
  bd_right(c, tmp, Rblk, transR, out, rows, cols, alpha, nullptr, 0.f, s);
}

void bd_left_dual(armor_ctx* c, const float* Ablk, const float* in1, const float* in2, float* tmp, float* out,
                  int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s) {
  if (c->tc_blocks && tc_block_ok(c, rows, cols) &&
      tc_done(c, tc_bd_left_dual(c, Ablk, false, in1, in2, out, rows, cols, part, n_part, s)))
    return;
  bd_left(c, Ablk, false, in1, tmp, rows, cols, 1.f, nullptr, 0.f, s);
  bd_left(c, Ablk, false, in2, out, rows, cols, 1.f, nullptr, 0.f, s);
  dot_partials(c, out, tmp, rows * cols, part, s);
  *n_part = ARMOR_DOT_BLOCKS;
}

extern "C" armor_status armor_block_product_two_sided(armor_ctx* c, const float* d_left, int32_t transpose_left,
                                                      const float* d_in, const float* d_right, int32_t transpose_right,
                                                      float* d_out, float alpha, int32_t path, armor_stream_t stream) {
  if (!c || !d_left || !d_in || !d_right || !d_out) return ARMOR_ERR_INVALID_ARG;
  if (path == 3 && !tc_block2_ok(c, c->d_out, c->d_in)) return ARMOR_ERR_UNSUPPORTED;
  if ((path == 1 || path == 2) && !tc_block_ok(c, c->d_out, c->d_in)) return ARMOR_ERR_UNSUPPORTED;
  if (path == 2 && !tc_blockres_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int saved = c->tc_blocks;
  c->tc_blocks = (path >= 0 && path <= 3) ? path : saved;
  bd_two_sided(c, d_left, transpose_left != 0, d_in, d_right, transpose_right != 0, c->Tmp, d_out, c->d_out, c->d_in, alpha, s);
  c->tc_blocks = saved;
  return finish_call(c);
}

extern "C" armor_status armor_block_product_dual(armor_ctx* c, const float* d_blocks, const float* d_in1,
                                                 const float* d_in2, float* d_out, double* d_dot, int32_t path,
                                                 armor_stream_t stream) {
  if (!c || !d_blocks || !d_in1 || !d_in2 || !d_out || !d_dot) return ARMOR_ERR_INVALID_ARG;
  if ((path == 1 || path == 2) && !tc_block_ok(c, c->d_out, c->d_in)) return ARMOR_ERR_UNSUPPORTED;
  if (path == 2 && !tc_blockres_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int saved = c->tc_blocks;
  c->tc_blocks = (path == 0 || path == 1 || path == 2) ? path : saved;
  int nq = 0;
  bd_left_dual(c, d_blocks, d_in1, d_in2, c->V, d_out, c->d_out, c->d_in, c->partials, &nq, s);
  reduce_partials_to(c, c->partials, nq, d_dot, s);
  c->tc_blocks = saved;
  return finish_call(c);
}

extern "C" armor_status armor_block_product(armor_ctx* c, int32_t side, int32_t transpose, const float* d_blocks,
                                            const float* d_in, float* d_out, int64_t rows, int64_t cols, float alpha,
                                            const float* d_add, float beta, int32_t path, armor_stream_t stream) {
  if (!c || !d_blocks || !d_in || !d_out || rows <= 0 || cols <= 0) return ARMOR_ERR_INVALID_ARG;
  if (side != 0 && side != 1) return ARMOR_ERR_INVALID_ARG;
  if (cols % 4 || (side == 0 ? cols : rows) % c->db) return ARMOR_ERR_SHAPE;
  if ((path == 1 || path == 2) && !tc_block_ok(c, rows, cols)) return ARMOR_ERR_UNSUPPORTED;
  if (path == 2 && !tc_blockres_ok(c)) return ARMOR_ERR_UNSUPPORTED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int saved = c->tc_blocks;
  c->tc_blocks = (path == 0 || path == 1 || path == 2) ? path : saved;
  if (side == 1) bd_left(c, d_blocks, transpose != 0, d_in, d_out, rows, cols, alpha, d_add, beta, s);
  else bd_right(c, d_in, d_blocks, transpose != 0, d_out, rows, cols, alpha, d_add, beta, s);
  c->tc_blocks = saved;
  return finish_call(c);
}
