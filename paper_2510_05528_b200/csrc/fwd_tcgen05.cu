// The two thin products of the deployment form (Section 3.1: y = A (S (B x)) with block-diagonal A and B applied
// as batched d_block x d_block products) in bf16:  out[t][n] = sum_k X[t][j*db + k] * Q[n][k]  for the block j that
// holds column n, with Q the wrapper's blocks stacked as [d][db] (row n of the stack = row n - j*db of block j).
// Both operands are K-major as they lie in memory, so the kernel is a batched GEMM over the blocks: 128 x 128
// output tiles, the contraction runs over the db columns of X that belong to the tile's block (two or four
// k-tiles of 64), bf16 operands by TMA (128-byte swizzle), tcgen05.mma kind::f16 with fp32 accumulation in tensor
// memory, bf16 output.  Per output element the product moves 2 bytes in and 2 bytes out and does 2*db flops: it
// is a streaming kernel, bound by HBM.
//
// Also here: the packing of the wrappers for this kernel (bf16, the normalisation's scales folded in, Section 3.2
// last paragraph) and the layer forward built from this kernel and the sparse core product.
//
// Kernel: persistent, 320 threads: warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 epilogue (accumulator ->
// bf16 -> shared-memory turn -> 128-byte row segments; warps 2-5 take the left 64 columns of the tile, warps 6-9
// the right 64: with four warps the epilogue, not HBM, set the pace).  Five stages of 32 KiB, two accumulator
// buffers.  Every wait is bounded.
#include <cuda_bf16.h>

#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128, BN = 128, BKE = 64;         // BKE bf16 = 128 bytes = one swizzle row
constexpr int NTHREADS = 320;
constexpr int STAGES = 5;
constexpr uint32_t TMEM_COLS = 256;                 // two accumulator buffers of BN columns
constexpr int A_BYTES = BM * BKE * 2;               // 16 KiB
constexpr int B_BYTES = BN * BKE * 2;               // 16 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;

struct FParams {
  __nv_bfloat16* out; int64_t ldo;   // [rows][ldo]
  int64_t rows, d;                   // tokens, output width (= number of rows of the stacked blocks)
  int db;
  int m_tiles, n_tiles, k_tiles;     // k_tiles = db / 64
  int32_t* status;
};

__device__ __forceinline__ uint64_t smem_desc_k(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__device__ __forceinline__ uint32_t instr_desc_bf16() {
  uint32_t d = 0;
  d |= 1u << 4;                   // D format: F32
  d |= 1u << 7;                   // A format: BF16
  d |= 1u << 10;                  // B format: BF16
  d |= (uint32_t)(BN >> 3) << 17;
  d |= (uint32_t)(BM >> 4) << 24;
  return d;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__global__ void __launch_bounds__(NTHREADS, 1)
fwd_block_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapQ, const FParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 4];
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[2 * STAGES]), tempty0 = smem_u32(&bars[2 * STAGES + 2]);
  const int n_tiles_total = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(tfull0 + 8 * s, 1); mbar_init(tempty0 + 8 * s, 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; long long issued = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x) {
        const int mt = tile / p.n_tiles, nt = tile - mt * p.n_tiles;   // the column tile runs fastest
        const int kx0 = (nt * BN / p.db) * p.db;                       // first column of X of the tile's block
        for (int kt = 0; kt < p.k_tiles; ++kt) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, STAGE_BYTES);
          const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          tma_load_2d(dst, &mapX, kx0 + kt * BKE, mt * BM, fb);
          tma_load_2d(dst + A_BYTES, &mapQ, kt * BKE, nt * BN, fb);
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        for (int back = 1; back <= STAGES && back <= issued; ++back) {
          int s = stage - back; uint32_t ph = phase;
          if (s < 0) { s += STAGES; ph ^= 1; }
          const long long t0 = clock64();
          while (!mbar_try(full0 + 8 * s, ph) && clock64() - t0 < 20000000ll) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16();
      int stage = 0; uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x, ++local) {
        const int as = local & 1;
        const uint32_t aphase = (uint32_t)(local >> 1) & 1u;
        if (!mbar_wait(tempty0 + 8 * as, aphase ^ 1, abortp, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(as * BN);
        for (int kt = 0; kt < p.k_tiles; ++kt) {
          if (!mbar_wait(full0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BKE / 16; ++k)
            umma_bf16(tacc, smem_desc_k(sa + k * 32), smem_desc_k(sb + k * 32), idesc, (uint32_t)((kt > 0) | (k != 0)));
          umma_commit(empty0 + 8 * stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit(tfull0 + 8 * as);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                 // tensor-memory lane quarter this warp may read
    const int half = (warp - 2) >> 2;       // which 64 columns of the tile
    uint32_t* tilebuf = reinterpret_cast<uint32_t*>(smem + (size_t)STAGES * STAGE_BYTES) + (warp - 2) * (32 * 33);
    int local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x, ++local) {
      const int mt = tile / p.n_tiles, nt = tile - mt * p.n_tiles;
      const int as = local & 1;
      const uint32_t aphase = (uint32_t)(local >> 1) & 1u;
      if (!mbar_wait(tfull0 + 8 * as, aphase, abortp, p.status)) { ok = false; break; }
      tc_fence_after();
      const int64_t row_base = (int64_t)mt * BM + q * 32;
      {
        const int ch = half;
        // 64 columns of the lane's row -> 32 words of two bf16; the 32 x 32 words are turned through shared
        // memory so that one store instruction writes 128 contiguous bytes of one row
        uint32_t r0[32], r1[32];
        tmem_ld32(tmem_base + (uint32_t)(as * BN + ch * 64) + ((uint32_t)(q * 32) << 16), r0);
        tmem_ld32(tmem_base + (uint32_t)(as * BN + ch * 64 + 32) + ((uint32_t)(q * 32) << 16), r1);
#pragma unroll
        for (int w = 0; w < 16; ++w) {
          tilebuf[lane * 33 + w] = pack_bf16(__uint_as_float(r0[2 * w]), __uint_as_float(r0[2 * w + 1]));
          tilebuf[lane * 33 + 16 + w] = pack_bf16(__uint_as_float(r1[2 * w]), __uint_as_float(r1[2 * w + 1]));
        }
        __syncwarp();
        const int64_t col = (int64_t)nt * BN + ch * 64 + 2 * lane;
        if (col < p.d) {
#pragma unroll 8
          for (int rr = 0; rr < 32; ++rr) {
            const int64_t grow = row_base + rr;
            if (grow < p.rows)
              *reinterpret_cast<uint32_t*>(p.out + grow * p.ldo + col) = tilebuf[rr * 33 + lane];
          }
        }
        __syncwarp();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * as);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Q[i][m][k] = rowscale[i*db + m] * colscale[i*db + k] * P[i][m][k], rounded to bf16 (either scale may be null)
__global__ void __launch_bounds__(256)
pack_blocks_kernel(const float* __restrict__ P, const float* __restrict__ rowscale, const float* __restrict__ colscale,
                   __nv_bfloat16* __restrict__ Q, int64_t n, int db) {
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < n; e += (int64_t)gridDim.x * 256) {
    const int64_t i = e / ((int64_t)db * db);
    const int m = (int)((e / db) % db), k = (int)(e % db);
    float v = P[e];
    if (rowscale) v *= rowscale[i * db + m];
    if (colscale) v *= colscale[i * db + k];
    Q[e] = __float2bfloat16(v);
  }
}

bool make_map_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BKE, 128};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

bool fwd_block_ok(const armor_ctx* c) { return c->db % 128 == 0 && c->d_in % 128 == 0 && c->d_out % 128 == 0; }

void launch_pack_blocks(armor_ctx* c, const float* P, const float* rowscale, const float* colscale, void* Q, int nb,
                        cudaStream_t s) {
  const int64_t n = (int64_t)nb * c->db * c->db;
  int64_t blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  KTimer kt(c, ARMOR_KC_FORWARD, 0.0, s);
  pack_blocks_kernel<<<(unsigned)blocks, 256, 0, s>>>(P, rowscale, colscale, static_cast<__nv_bfloat16*>(Q), n, c->db);
  c->launches++;
}

// out[rows][d] (bf16) = X[rows][d] (bf16) times the block-diagonal matrix whose stacked blocks are Q[d][db] (bf16):
// out[t][n] = sum_k X[t][j*db + k] Q[n][k], j = n / db
armor_status launch_fwd_block(armor_ctx* c, const void* X, const void* Q, void* out, int64_t rows, int64_t d,
                              cudaStream_t s) {
  if (!fwd_block_ok(c) || rows <= 0 || d % 128) return ARMOR_ERR_UNSUPPORTED;
  CUtensorMap mX, mQ;
  if (!make_map_bf16(&mX, X, rows, d, d)) return ARMOR_ERR_CUDA;
  if (!make_map_bf16(&mQ, Q, d, c->db, c->db)) return ARMOR_ERR_CUDA;
  FParams p{};
  p.out = static_cast<__nv_bfloat16*>(out); p.ldo = d; p.rows = rows; p.d = d; p.db = c->db;
  p.m_tiles = (int)((rows + BM - 1) / BM); p.n_tiles = (int)(d / BN); p.k_tiles = c->db / BKE;
  p.status = c->status;
  constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024 + 8 * 32 * 33 * sizeof(uint32_t);
  static PerDeviceOnce attr;
  if (ensure_dynamic_smem(attr, c->device, fwd_block_kernel, SMEM) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int n_sm = c->n_sm;
  const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
  const int grid = tiles < n_sm ? (int)tiles : n_sm;
  KTimer kt(c, ARMOR_KC_FORWARD, 4.0 * (double)rows * (double)d, s);
  fwd_block_kernel<<<grid, NTHREADS, SMEM, s>>>(mX, mQ, p);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}
