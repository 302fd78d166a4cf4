// Operand preparation for the three-pass fp16 mode of the dense contractions (ARMOR_PREC_FP16X3).
//
// An fp32 value x is written as hi + lo with hi = fp16(x), lo = fp16(x - hi): 22 significant bits, as with two
// tf32 parts, but fp16 has 5 exponent bits only.  Every operand is therefore scaled by powers of two (exact)
// so that the entries that matter for a dot product land in the range where both parts are normal numbers:
//   * a left operand L of L.H is scaled per column by d_k = 2^floor(log2 sqrt(H_kk)) and then per row so that
//     the row's largest entry lies in [2^14, 2^15);
//   * H is replaced by H_kn / (d_k d_n) * 2^12: a positive semidefinite H has |H_kn| <= sqrt(H_kk H_nn), so these
//     entries are below 2^14 in magnitude whatever the spread of the channel scales;
//   * a chunk of activations X (Gram X^T X, Section 2 of the paper) is scaled per channel by its largest
//     magnitude inside the chunk.
// Entries far below their row's or column's maximum lose relative accuracy (absolute error 2^-25 after scaling,
// i.e. 2^-39 of the maximum) -- less than what the fp32 inputs themselves carry.  The GEMM's epilogue multiplies
// the accumulator by the inverse scales.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "armor_internal.cuh"

namespace {

constexpr int NT = 256;
constexpr int TARGET_EXP = 15;   // frexp exponent of the scaled maximum: values in [2^14, 2^15)
constexpr int H_SHIFT = 12;      // H / (d d^T) has entries below 4; times 2^12 they stay below 2^14

// Finite values beyond the fp16 range are clamped (after the scalings above this happens only to an H that is not
// positive semidefinite); NaN and Inf pass through, so that unusable inputs stay visible in the result.
__device__ __forceinline__ float clamp_f16(float v) { return isfinite(v) ? fminf(fmaxf(v, -65504.f), 65504.f) : v; }

__device__ __forceinline__ void split2(float v, __half& hi, __half& lo) {
  v = clamp_f16(v);
  hi = __float2half_rn(v);
  lo = __float2half_rn(v - __half2float(hi));
}

// power of two that brings a maximum magnitude `mx` into [2^14, 2^15); 0 for an all-zero or non-finite line
__device__ __forceinline__ int scale_exp(float mx) {
  if (!(mx > 0.f) || isinf(mx)) return 0;
  int ex;
  frexpf(mx, &ex);
  int e = TARGET_EXP - ex;
  return e < -100 ? -100 : (e > 100 ? 100 : e);
}

__device__ __forceinline__ float block_max(float v) {
  __shared__ float sm[32];
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) sm[w] = v;
  __syncthreads();
  const int nw = (blockDim.x + 31) >> 5;
  v = (lane < nw) ? sm[lane] : 0.f;
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  return v;   // valid in every thread
}

// hpow[k] = 2^floor(log2 sqrt(H_kk)) (1 for a dead channel)
__global__ void hpow_kernel(const float* __restrict__ hdiag, float* __restrict__ hpow, int64_t n) {
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n) return;
  const float h = hdiag[k];
  int e = 0;
  if (h > 0.f && !isinf(h)) {
    int q;
    frexpf(h, &q);                       // h = f 2^q, f in [0.5, 1)
    e = (q - 1) >> 1;                    // floor((q - 1) / 2)
  }
  hpow[k] = scalbnf(1.f, e);
}

// Hhi + Hlo = H_kn / (d_k d_n) * 2^H_SHIFT, four columns per thread
__global__ void __launch_bounds__(NT) split_H_kernel(const float4* __restrict__ H, const float* __restrict__ hpow,
                                                     __half2* __restrict__ hi, __half2* __restrict__ lo, int64_t n,
                                                     int32_t* __restrict__ status) {
  const int64_t n4 = n / 4;
  for (int64_t i = (int64_t)blockIdx.x * NT + threadIdx.x; i < n * n4; i += (int64_t)gridDim.x * NT) {
    const int64_t k = i / n4, c4 = (i % n4) * 4;
    const float rk = scalbnf(1.f / hpow[k], H_SHIFT);     // reciprocal of a power of two: exact
    const float4 v = H[i];
    const float4 d = *reinterpret_cast<const float4*>(hpow + c4);
    const float x0 = v.x * rk / d.x, x1 = v.y * rk / d.y, x2 = v.z * rk / d.z, x3 = v.w * rk / d.w;
    const int over = (fabsf(x0) > 65504.f && isfinite(x0)) + (fabsf(x1) > 65504.f && isfinite(x1)) +
                     (fabsf(x2) > 65504.f && isfinite(x2)) + (fabsf(x3) > 65504.f && isfinite(x3));
    if (over) atomicAdd(&status[ST_H_RANGE], over);
    __half h0, h1, h2, h3, l0, l1, l2, l3;
    split2(x0, h0, l0);
    split2(x1, h1, l1);
    split2(x2, h2, l2);
    split2(x3, h3, l3);
    hi[2 * i] = __halves2half2(h0, h1); hi[2 * i + 1] = __halves2half2(h2, h3);
    lo[2 * i] = __halves2half2(l0, l1); lo[2 * i + 1] = __halves2half2(l2, l3);
  }
}

// One CTA per row of `in` [rows, cols] (leading dimension ld): the row times the column scales, brought into
// range by a power of two of its own; out_scale[row] = post / that power.
__global__ void __launch_bounds__(NT) split_rows_kernel(const float* __restrict__ in, int64_t ld, int64_t cols,
                                                        const float* __restrict__ colscale, float post,
                                                        __half2* __restrict__ hi, __half2* __restrict__ lo,
                                                        float* __restrict__ out_scale) {
  const int64_t row = blockIdx.x;
  const float4* src = reinterpret_cast<const float4*>(in + row * ld);
  const float4* cs4 = reinterpret_cast<const float4*>(colscale);
  const int64_t c4n = cols / 4;
  float mx = 0.f;
  for (int64_t i = threadIdx.x; i < c4n; i += NT) {
    float4 v = src[i];
    if (colscale) { const float4 d = cs4[i]; v.x *= d.x; v.y *= d.y; v.z *= d.z; v.w *= d.w; }
    mx = fmaxf(mx, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
  }
  mx = block_max(mx);
  const int e = scale_exp(mx);
  if (threadIdx.x == 0) out_scale[row] = scalbnf(post, -e);
  __half2* dh = hi + row * (cols / 2);
  __half2* dl = lo + row * (cols / 2);
  for (int64_t i = threadIdx.x; i < c4n; i += NT) {
    float4 v = src[i];
    if (colscale) { const float4 d = cs4[i]; v.x *= d.x; v.y *= d.y; v.z *= d.z; v.w *= d.w; }
    __half h0, h1, h2, h3, l0, l1, l2, l3;
    split2(scalbnf(v.x, e), h0, l0);
    split2(scalbnf(v.y, e), h1, l1);
    split2(scalbnf(v.z, e), h2, l2);
    split2(scalbnf(v.w, e), h3, l3);
    dh[2 * i] = __halves2half2(h0, h1); dh[2 * i + 1] = __halves2half2(h2, h3);
    dl[2 * i] = __halves2half2(l0, l1); dl[2 * i + 1] = __halves2half2(l2, l3);
  }
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// Largest magnitude of every column of a chunk X [rows, cols]: the order of the atomic maxima does not matter,
// so the result is deterministic.  Magnitudes compare like their bit patterns.
template <typename TIn>
__global__ void __launch_bounds__(NT) colabsmax_kernel(const TIn* __restrict__ X, int64_t ldx, int64_t rows, int64_t cols,
                                                       unsigned* __restrict__ umax) {
  const int64_t col = (int64_t)blockIdx.x * NT + threadIdx.x;
  if (col >= cols) return;
  const int64_t r0 = (int64_t)blockIdx.y * 256;
  const int64_t r1 = r0 + 256 < rows ? r0 + 256 : rows;
  float mx = 0.f;
  for (int64_t r = r0; r < r1; ++r) {
    const float a = fabsf(to_f32(X[r * ldx + col]));
    mx = (a > mx || a != a) ? a : mx;           // a NaN sticks
  }
  atomicMax(umax + col, __float_as_uint(mx));
}

// gscale[c] = 2^-e_c, the factor the Gram's epilogue multiplies row c and column c by
__global__ void gram_scale_kernel(const unsigned* __restrict__ umax, float* __restrict__ gscale, int64_t n) {
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k < n) gscale[k] = scalbnf(1.f, -scale_exp(__uint_as_float(umax[k])));
}

// X [rows, cols] (ld ldx) -> Thi/Tlo [cols, ldt] fp16: transposed, column c scaled by 2^e_c, split.  bf16 input
// has 8 significant bits: it is exact in one fp16 part, Tlo is then not written.  Tiles of 64 tokens x 64
// channels: rows of 64 channels are read 128 bytes per warp instruction, and every channel's 64 tokens are written
// as 32 pairs (128 bytes per warp instruction).  ldt is a multiple of 64; tokens beyond `rows` are written as zeros.
template <typename TIn>
__global__ void __launch_bounds__(256) transpose_split_f16_kernel(const TIn* __restrict__ X, int64_t ldx, int64_t rows,
                                                                  int64_t cols, const unsigned* __restrict__ umax,
                                                                  __half* __restrict__ Thi, __half* __restrict__ Tlo,
                                                                  int64_t ldt) {
  __shared__ float tile[64][65];
  const int64_t c0 = (int64_t)blockIdx.x * 64, r0 = (int64_t)blockIdx.y * 64;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int rr = w + 8 * i;
    const int64_t r = r0 + rr;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int64_t cidx = c0 + lane + 32 * hf;
      tile[rr][lane + 32 * hf] = (r < rows && cidx < cols) ? to_f32(X[r * ldx + cidx]) : 0.f;
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int ch = w + 8 * j;
    const int64_t cidx = c0 + ch;
    if (cidx >= cols) continue;
    const int e = scale_exp(__uint_as_float(umax[cidx]));
    __half h0, l0, h1, l1;
    split2(scalbnf(tile[2 * lane][ch], e), h0, l0);
    split2(scalbnf(tile[2 * lane + 1][ch], e), h1, l1);
    const int64_t o = cidx * ldt + r0 + 2 * lane;             // even: ldt and r0 are multiples of 64
    *reinterpret_cast<__half2*>(Thi + o) = __halves2half2(h0, h1);
    if (Tlo) *reinterpret_cast<__half2*>(Tlo + o) = __halves2half2(l0, l1);
  }
}

inline unsigned grid_for(int64_t n) {
  int64_t b = (n + NT - 1) / NT;
  return (unsigned)(b < 148 * 8 ? (b < 1 ? 1 : b) : 148 * 8);
}

}  // namespace

void launch_f16_prepare_H(armor_ctx* c, const float* H, cudaStream_t s) {
  const int64_t n = c->d_in;
  KTimer kt(c, ARMOR_KC_OPERAND_SPLIT, 8.0 * (double)n * (double)n, s);
  hpow_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(c->hdiag, c->hpow, n);
  __half* hi = reinterpret_cast<__half*>(c->Hlo);
  split_H_kernel<<<grid_for(n * n / 4), NT, 0, s>>>(reinterpret_cast<const float4*>(H), c->hpow,
                                                    reinterpret_cast<__half2*>(hi), reinterpret_cast<__half2*>(hi + n * n), n, c->status);
  c->launches += 2;
}

void launch_f16_split_rows(armor_ctx* c, const float* in, int64_t ld, int64_t rows, int64_t cols, const float* colscale,
                           float post, void* hi, void* lo, float* out_scale, cudaStream_t s) {
  KTimer kt(c, ARMOR_KC_OPERAND_SPLIT, 8.0 * (double)rows * (double)cols, s);
  split_rows_kernel<<<(unsigned)rows, NT, 0, s>>>(in, ld, cols, colscale, post, static_cast<__half2*>(hi),
                                                  static_cast<__half2*>(lo), out_scale);
  c->launches++;
}

float f16_H_post_scale() { return 1.f / (float)(1 << H_SHIFT); }

armor_status launch_f16_gram_stage(armor_ctx* c, const void* X, int x_dtype, int64_t ldx, int64_t rows, int64_t cols,
                                   void* Thi, void* Tlo, int64_t ldt, float* gscale, cudaStream_t s) {
  if (cudaMemsetAsync(c->gmax, 0, (size_t)cols * sizeof(unsigned), s) != cudaSuccess) return ARMOR_ERR_CUDA;
  // one read for the maxima, one read and one 16-bit write per part for the staged chunk
  KTimer kt(c, ARMOR_KC_GRAM_STAGING, (double)rows * (double)cols * (x_dtype == ARMOR_DTYPE_BF16 ? 6.0 : 12.0), s);
  const dim3 g1((unsigned)((cols + NT - 1) / NT), (unsigned)((rows + 255) / 256));
  const dim3 g2((unsigned)((cols + 63) / 64), (unsigned)(ldt / 64));
  if (x_dtype == ARMOR_DTYPE_BF16) {
    const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
    colabsmax_kernel<<<g1, NT, 0, s>>>(Xb, ldx, rows, cols, c->gmax);
    transpose_split_f16_kernel<<<g2, 256, 0, s>>>(Xb, ldx, rows, cols, c->gmax, static_cast<__half*>(Thi),
                                                         (__half*)nullptr, ldt);
  } else {
    const float* Xf = static_cast<const float*>(X);
    colabsmax_kernel<<<g1, NT, 0, s>>>(Xf, ldx, rows, cols, c->gmax);
    transpose_split_f16_kernel<<<g2, 256, 0, s>>>(Xf, ldx, rows, cols, c->gmax, static_cast<__half*>(Thi),
                                                         static_cast<__half*>(Tlo), ldt);
  }
  gram_scale_kernel<<<(unsigned)((cols + 255) / 256), 256, 0, s>>>(c->gmax, gscale, cols);
  c->launches += 3;
  return ARMOR_OK;
}
