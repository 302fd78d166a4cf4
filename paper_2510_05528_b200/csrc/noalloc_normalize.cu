// armor_normalize_noalloc: the row/column normalisation as a stand-alone call for callers that cannot
// provide scratch memory.  Its only scratch, the per-chunk column sums of squares, lives in a fixed
// device array compiled into the library instead of in a caller-provided workspace.
#include <cuda_runtime.h>
#include <stdint.h>

#include "armor.h"

namespace {

constexpr int NT = 256;
constexpr int CHUNKS = ARMOR_NOALLOC_ROW_CHUNKS;
constexpr int64_t MAX_COLS = ARMOR_NOALLOC_MAX_COLS;
constexpr int MAX_DEVICES = 64;

// Built-in scratch: CHUNKS x MAX_COLS partial sums (4 MiB).  Every GPU that loads the library keeps this
// array until the process exits.  All calls on a device share it.
static __device__ __align__(256) double g_colpart[(size_t)CHUNKS * MAX_COLS];

// Device address of g_colpart per device ordinal, looked up once (0 = not looked up yet).  In host code
// the name g_colpart is only a handle for the runtime; kernels must be given the address obtained here.
double* g_colpart_addr[MAX_DEVICES] = {nullptr};

__global__ void __launch_bounds__(NT) na_colsumsq_kernel(const float* __restrict__ W, int64_t rows, int64_t cols,
                                                         double* __restrict__ part) {
  const int64_t col = (int64_t)blockIdx.x * NT + threadIdx.x;
  if (col >= cols) return;
  const int64_t per = (rows + CHUNKS - 1) / CHUNKS;
  const int64_t r0 = blockIdx.y * per, r1 = min(rows, r0 + per);
  double acc = 0.0;
  for (int64_t r = r0; r < r1; ++r) {
    const double w = W[r * cols + col];
    acc += w * w;
  }
  part[(int64_t)blockIdx.y * cols + col] = acc;   // every slot that is read later is written here first
}

__global__ void __launch_bounds__(NT) na_colnorm_kernel(const double* __restrict__ part, int64_t cols,
                                                        float* __restrict__ r1) {
  const int64_t col = (int64_t)blockIdx.x * NT + threadIdx.x;
  if (col >= cols) return;
  double acc = 0.0;
  for (int ch = 0; ch < CHUNKS; ++ch) acc += part[(int64_t)ch * cols + col];
  const float r = (float)sqrt(acc);
  r1[col] = (r == 0.f) ? 1.f : r;
}

__global__ void __launch_bounds__(NT) na_rownorm_scale_kernel(const float* __restrict__ W, const float* __restrict__ r1,
                                                              float* __restrict__ r2, float* __restrict__ Wbar,
                                                              int64_t cols) {
  __shared__ double warp_sum[NT / 32];
  __shared__ float r2s;
  const int64_t row = blockIdx.x;
  const float* w = W + row * cols;
  double acc = 0.0;
  for (int64_t c = threadIdx.x; c < cols; c += NT) {
    const double v = (double)w[c] / (double)r1[c];
    acc += v * v;
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    double v = (threadIdx.x < NT / 32) ? warp_sum[threadIdx.x] : 0.0;
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    if (threadIdx.x == 0) {
      float r = (float)sqrt(v);
      r = (r == 0.f) ? 1.f : r;
      r2[row] = r;
      r2s = r;
    }
  }
  __syncthreads();
  const float rr = r2s;
  for (int64_t c = threadIdx.x; c < cols; c += NT) Wbar[row * cols + c] = (w[c] / r1[c]) / rr;
}

}  // namespace

extern "C" armor_status armor_normalize_noalloc(const float* d_W, int64_t d_out, int64_t d_in, float* d_Wbar,
                                                float* d_r1, float* d_r2, armor_stream_t stream) {
  if (!d_W || !d_Wbar || !d_r1 || !d_r2) return ARMOR_ERR_INVALID_ARG;
  if (d_out <= 0 || d_in <= 0) return ARMOR_ERR_SHAPE;
  if (d_in > MAX_COLS || d_out > ARMOR_NOALLOC_MAX_ROWS) return ARMOR_ERR_TOO_LARGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return ARMOR_ERR_CUDA;
  if (dev < 0 || dev >= MAX_DEVICES) return ARMOR_ERR_UNSUPPORTED;
  if (!g_colpart_addr[dev]) {
    // one-time set-up for this device (it is the current one): ask the runtime where the array lives
    double* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_colpart) != cudaSuccess || !p) return ARMOR_ERR_CUDA;
    g_colpart_addr[dev] = p;
  }
  double* part = g_colpart_addr[dev];
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const unsigned gx = (unsigned)((d_in + NT - 1) / NT);
  na_colsumsq_kernel<<<dim3(gx, CHUNKS), NT, 0, s>>>(d_W, d_out, d_in, part);
  na_colnorm_kernel<<<gx, NT, 0, s>>>(part, d_in, d_r1);
  na_rownorm_scale_kernel<<<(unsigned)d_out, NT, 0, s>>>(d_W, d_r1, d_r2, d_Wbar, d_in);
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}
