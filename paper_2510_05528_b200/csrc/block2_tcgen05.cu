// Two-sided products with the block-diagonal wrappers (Section 3.1 of the paper) for d_block = 128:
//
//   out[128 i + m][128 j + n] = alpha * sum_{k, l} Lop_i[m][k] * X[128 i + k][128 j + l] * Rop_j[l][n]
//
// (Lop_i = L_i or its transpose, Rop_j = R_j or its transpose).  Both wrappers are block diagonal with the block
// size of a tile, so a 128 x 128 tile of the result depends on the same tile of X only: the intermediate Lop_i X_ij
// never has to leave the SM.  It is formed in tensor memory (three tf32 passes, fp32 accumulator), split there
// into a high part (the accumulator's own words: the tensor core reads the top 19 bits) and a low part
// (tcgen05.ld, x - trunc_tf32(x), tcgen05.st), and used from tensor memory as the M-side operand of the second
// product.  One W-shaped read and one W-shaped write instead of two of each, and one launch instead of two.
// The MMAs are issued in the order of the two separate launches of block_tcgen05.cu and the intermediate is the
// same fp32 value, so the result has the same bits.
//
// Persistent kernel, 448 threads:
//   warp 0       : TMA producer.  Per tile four chunks (32 along k) of Lop_i and X_ij (product 1) and four chunks (32
//                  along l) of Rop_j (product 2)
//   warp 1       : MMA issuer: product 1 into D1[t % 2]; product 2 (A from tensor memory) into D2
//   warps 2-5    : low parts of the chunks in shared memory
//   warps 6-9    : epilogue of D2 (alpha, swizzled staging, TMA store)
//   warps 10-13  : split of D1 in tensor memory
// The products are software-pipelined: product 1 of tile t + 1 is issued BEFORE product 2 of tile t
// (P1(0), P1(1), P2(0), P1(2), P2(1), ...), so that the tensor pipe works on the next tile while four warps split this
// tile's intermediate, and the epilogue drains D2 while product 1 of the tile after next runs.  The producer and the
// splitter walk their chunks in the same order.
// Tensor memory: D1 0..127 and 128..255 (alternating), low part of D1 256..383, D2 384..511.
// Every wait is bounded; a wait that runs out raises a status word and the CTA leaves through the common exit that
// frees its tensor memory.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int TILE = 128, BK = 32;
constexpr int NTHREADS = 448;
constexpr int STAGES = 3;
constexpr int OP_BYTES = TILE * BK * 4;           // 16 KiB: one operand chunk
constexpr int STAGE_BYTES = 4 * OP_BYTES;         // M side raw, M side low part, N side raw, N side low part
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t T_D1 = 0, T_D1LO = 256, T_D2 = 384;
constexpr int EPI_BYTES = 32 * 64 * 4;            // per epilogue warp: two swizzled 32 x 32 boxes
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 4 * EPI_BYTES + 1024;

struct P2Params {
  int l_mn;                         // 1: Lop_i[m][k] = L_i[k][m] (M-major operand), 0: L_i[m][k] (K-major)
  int r_mn;                         // 1: the N-side operand [n][l] = R_j[l][n] (N-major), 0: R_j[n][l] (K-major: Rop = R_j^T)
  int nbi, nbj;                     // block rows and block columns of X
  int64_t c_rows, c_cols;
  float alpha;
  int32_t* status;
};



// chunk kc of a 128 x 128 block operand whose rows start at row0 of the [*, 128] array behind map: K-major as one
// box of 128 rows x 32 columns, MN-major as four boxes of 32 x 32 (rows 32 kc .., columns 32 q ..)
__device__ __forceinline__ void load_block_chunk(uint32_t dst, const CUtensorMap* map, int mn, int row0, int col0, int kc,
                                                 uint32_t bar) {
  if (mn) {
#pragma unroll
    for (int q = 0; q < 4; ++q) tma_load_2d(dst + q * 4096, map, col0 + 32 * q, row0 + BK * kc, bar);
  } else {
    tma_load_2d(dst, map, col0 + BK * kc, row0, bar);
  }
}

// Step o of a CTA's schedule over its n tiles: P1(0), then (P1(t + 1), P2(t)) for t = 0 .. n - 2, then P2(n - 1).
__device__ __forceinline__ void schedule_step(int o, int n, bool& second, int& t) {
  if (o == 0) { second = false; t = 0; return; }
  const int m = o - 1;
  if (m == 2 * n - 2) { second = true; t = n - 1; return; }
  second = (m & 1) != 0;
  t = second ? (m >> 1) : (m >> 1) + 1;
}

__device__ __forceinline__ uint64_t op_desc(uint32_t base, int mn) {
  return mn ? smem_desc_mn_sw128_32b(base, 4096, 512) : smem_desc_sw128(base, 16, 1024);
}

__global__ void __launch_bounds__(NTHREADS, 1)
tc_block2_kernel(const __grid_constant__ CUtensorMap mapL, const __grid_constant__ CUtensorMap mapX,
                 const __grid_constant__ CUtensorMap mapR, const __grid_constant__ CUtensorMap mapC, const P2Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[3 * STAGES + 5];
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), split0 = smem_u32(&bars[STAGES]), empty0 = smem_u32(&bars[2 * STAGES]);
  const uint32_t d1full0 = smem_u32(&bars[3 * STAGES]), convdone = d1full0 + 16;
  const uint32_t d2full = d1full0 + 24, d2empty = d1full0 + 32;
  const int n_items = p.nbi * p.nbj;
  const int n_local = (int)blockIdx.x < n_items ? (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;   // this CTA's tiles

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(split0 + 8 * s, 4);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(d1full0, 1);
    mbar_init(d1full0 + 8, 1);
    mbar_init(convdone, 4);
    mbar_init(d2full, 1);
    mbar_init(d2empty, 4);
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
      for (int o = 0; o < 2 * n_local && ok; ++o) {
        bool second; int t;
        schedule_step(o, n_local, second, t);
        const int item = (int)blockIdx.x + t * (int)gridDim.x;
        const int i = item / p.nbj, j = item - i * p.nbj;
        for (int kc = 0; kc < 4; ++kc) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          if (!second) {
            // product 1: Lop_i[:, 32 kc ..] and X_ij[32 kc .., :]
            mbar_expect_tx(fb, 2 * OP_BYTES);
            load_block_chunk(dst, &mapL, p.l_mn, TILE * i, 0, kc, fb);
            load_block_chunk(dst + 2 * OP_BYTES, &mapX, 1, TILE * i, TILE * j, kc, fb);
          } else {
            // product 2: Rop_j[32 kc .., :]
            mbar_expect_tx(fb, OP_BYTES);
            load_block_chunk(dst + 2 * OP_BYTES, &mapR, p.r_mn, TILE * j, 0, kc, fb);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        // leave no bulk copy in flight: wait (bounded) for the stages armed most recently
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
      const uint32_t idesc1 = instr_desc_tf32_mn(TILE, TILE, p.l_mn, 1);
      const uint32_t idesc2 = instr_desc_tf32_mn(TILE, TILE, 0, p.r_mn);
      // descriptors of stage 0; only their address field moves
      const uint64_t da0 = op_desc(smem_u32(smem), p.l_mn);
      const uint64_t dx0 = op_desc(smem_u32(smem) + 2 * OP_BYTES, 1);
      const uint64_t dr0 = op_desc(smem_u32(smem) + 2 * OP_BYTES, p.r_mn);
      const uint64_t kinc_a = p.l_mn ? (1024u >> 4) : (32u >> 4), kinc_x = 1024u >> 4;
      const uint64_t kinc_r = p.r_mn ? (1024u >> 4) : (32u >> 4);
      const uint32_t d1lo = tmem_base + T_D1LO, d2 = tmem_base + T_D2;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int o = 0; o < 2 * n_local && ok; ++o) {
        bool second; int t;
        schedule_step(o, n_local, second, t);
        const uint32_t d1 = tmem_base + T_D1 + (uint32_t)((t & 1) * TILE);
        if (!second) {
          // ---- product 1 of tile t: D1[t % 2] = Lop_i X_ij  (low part of Lop first, as in the one-sided kernel).  The
          // buffer was last read by product 2 of tile t - 2, which precedes this point in the pipe's order.
          for (int kc = 0; kc < 4; ++kc) {
            if (!mbar_wait(split0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
            tc_fence_after();
            const uint64_t so = (uint64_t)(uint32_t)(stage * (STAGE_BYTES >> 4));
            const uint64_t da = da0 + so, dal = da + (OP_BYTES >> 4), dx = dx0 + so, dxl = dx + (OP_BYTES >> 4);
            umma_tf32(d1, dal, dx, idesc1, (uint32_t)(kc > 0));
            umma_tf32_acc(d1, da, dxl, idesc1);
            umma_tf32_acc(d1, da, dx, idesc1);
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) {
              umma_tf32_acc(d1, dal + k * kinc_a, dx + k * kinc_x, idesc1);
              umma_tf32_acc(d1, da + k * kinc_a, dxl + k * kinc_x, idesc1);
              umma_tf32_acc(d1, da + k * kinc_a, dx + k * kinc_x, idesc1);
            }
            umma_commit(empty0 + 8 * stage);
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (!ok) break;
          umma_commit(d1full0 + 8 * (t & 1));
        } else {
          // ---- product 2 of tile t: D2 = D1[t % 2] Rop_j, D1 from tensor memory (its low part first: the M side of this
          // product).  Warps 10-13 have split D1; the epilogue has drained D2 of tile t - 1.
          if (!mbar_wait(convdone, (uint32_t)t & 1u, abortp, p.status)) { ok = false; break; }
          if (t > 0 && !mbar_wait(d2empty, (uint32_t)(t - 1) & 1u, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          for (int kc = 0; kc < 4; ++kc) {
            if (!mbar_wait(split0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
            tc_fence_after();
            const uint64_t dr = dr0 + (uint64_t)(uint32_t)(stage * (STAGE_BYTES >> 4)), drl = dr + (OP_BYTES >> 4);
            const uint32_t a_hi = d1 + (uint32_t)(kc * BK), a_lo = d1lo + (uint32_t)(kc * BK);
            umma_tf32_ta(d2, a_lo, dr, idesc2, (uint32_t)(kc > 0));
            umma_tf32_ta_acc(d2, a_hi, drl, idesc2);
            umma_tf32_ta_acc(d2, a_hi, dr, idesc2);
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) {
              umma_tf32_ta_acc(d2, a_lo + 8 * k, dr + k * kinc_r, idesc2);
              umma_tf32_ta_acc(d2, a_hi + 8 * k, drl + k * kinc_r, idesc2);
              umma_tf32_ta_acc(d2, a_hi + 8 * k, dr + k * kinc_r, idesc2);
            }
            umma_commit(empty0 + 8 * stage);
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (!ok) break;
          umma_commit(d2full);      // D2 is complete; the low part of D1 may be overwritten
        }
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ low parts of the chunks
    const int t = threadIdx.x - 64;   // 0..127
    int stage = 0; uint32_t phase = 0;
    bool ok = true;
    for (int o = 0; o < 2 * n_local && ok; ++o) {
      bool second; int tt;
      schedule_step(o, n_local, second, tt);
      for (int kc = 0; kc < 4; ++kc) {
        if (!mbar_wait(full0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
        float4* base = reinterpret_cast<float4*>(smem + (size_t)stage * STAGE_BYTES);
#pragma unroll
        for (int op = 0; op < 2; ++op) {
          if (op == 0 && second) continue;        // product 2 has no M-side chunk in shared memory
          float4* hi = base + op * (2 * OP_BYTES / 16);
          float4* lo = hi + OP_BYTES / 16;
#pragma unroll
          for (int e = 0; e < OP_BYTES / 16 / 128; ++e) {
            const int idx = t + e * 128;
            const float4 v = hi[idx];
            float4 h;
            h.x = __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
            h.y = __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
            h.z = __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
            h.w = __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
            lo[idx] = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
          }
        }
        // make the generic-proxy writes visible to the tensor-core (async proxy) reads
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(split0 + 8 * stage);
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------ epilogue warps
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    uint32_t local = 0;
    bool ok = true;
    uint8_t* buf = smem + (size_t)STAGES * STAGE_BYTES + (size_t)q * EPI_BYTES;   // two 4 KiB boxes of 32 x 32
    const uint32_t buf_u32 = smem_u32(buf);
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++local) {
      const int i = item / p.nbj, j = item - i * p.nbj;
      const int64_t row_base = (int64_t)TILE * i + q * 32;
      const int64_t col_tile = (int64_t)TILE * j;
      // The warp's 32 x 128 slab goes through shared memory in two halves of 64 columns (two 32 x 32 boxes).
#pragma unroll 1
      for (int hf = 0; hf < 2 && ok; ++hf) {
        if (lane == 0) tma_store_wait_read();        // the previous stores have read the staging boxes
        __syncwarp();
        if (hf == 0) {
          if (!__all_sync(0xffffffffu, mbar_wait(d2full, local & 1u, abortp, p.status))) { ok = false; break; }
          tc_fence_after();
        }
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t r[32];
          tmem_ld32(tmem_base + T_D2 + (uint32_t)(hf * 64 + ch * 32) + ((uint32_t)(q * 32) << 16), r);
          // lane = row of the box; 16-byte chunk c of the row sits at chunk c ^ (row % 8)  (128-byte swizzle)
          uint8_t* rowp = buf + ch * 4096 + lane * 128;
#pragma unroll
          for (int cq = 0; cq < 8; ++cq) {
            float4* cell = reinterpret_cast<float4*>(rowp + ((cq ^ (lane & 7)) << 4));
            *cell = make_float4(p.alpha * __uint_as_float(r[4 * cq]), p.alpha * __uint_as_float(r[4 * cq + 1]),
                                p.alpha * __uint_as_float(r[4 * cq + 2]), p.alpha * __uint_as_float(r[4 * cq + 3]));
          }
        }
        if (hf == 1) tc_fence_before();             // all reads of the accumulator are done
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          if (hf == 1) mbar_arrive(d2empty);
          for (int ch = 0; ch < 2; ++ch)
            tma_store_2d(&mapC, (int)(col_tile + 64 * hf + 32 * ch), (int)row_base, buf_u32 + ch * 4096);
          tma_store_commit();
        }
      }
    }
    if (lane == 0) tma_store_wait_read();           // shared memory stays valid until the stores have read it
  } else {
    // ------------------------------------------------------------ split of D1 in tensor memory
    const int q = warp & 3;
    const uint32_t lane_sel = (uint32_t)(q * 32) << 16;
    uint32_t local = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++local) {
      // product 1 of this tile has finished, and product 2 of the tile before has read the low part that is overwritten now
      if (!__all_sync(0xffffffffu, mbar_wait(d1full0 + 8 * (local & 1u), (local >> 1) & 1u, abortp, p.status))) { ok = false; break; }
      if (local > 0 && !__all_sync(0xffffffffu, mbar_wait(d2full, (local - 1) & 1u, abortp, p.status))) { ok = false; break; }
      tc_fence_after();
#pragma unroll 1
      for (int g = 0; g < 4; ++g) {
        uint32_t r[32];
        tmem_ld32(tmem_base + T_D1 + (uint32_t)((local & 1u) * TILE + 32 * g) + lane_sel, r);
#pragma unroll
        for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) - __uint_as_float(r[e] & 0xffffe000u));
        tmem_st32(tmem_base + T_D1LO + (uint32_t)(32 * g) + lane_sel, r);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(convdone);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

inline bool ptr_ok(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

}  // namespace

bool tc_block2_ok(const armor_ctx* c, int64_t rows, int64_t cols) {
  return c->cfg.precision != ARMOR_PREC_SIMT && c->db == TILE && rows > 0 && rows % TILE == 0 && cols > 0 && cols % TILE == 0 &&
         !c->block_one_pass;
}

// out[i-th block row, j-th block column] = alpha * Lop_i * X_ij * Rop_j,  Lop_i = Lblk[i] or its transpose, Rop_j = Rblk[j]
// or its transpose; X and out are [rows, cols] and must not overlap
armor_status tc_two_sided(armor_ctx* c, const float* Lblk, bool transL, const float* X, const float* Rblk, bool transR,
                          float* out, int64_t rows, int64_t cols, float alpha, cudaStream_t s) {
  if (!ptr_ok(Lblk) || !ptr_ok(X) || !ptr_ok(Rblk) || !ptr_ok(out)) return ARMOR_ERR_UNSUPPORTED;
  P2Params p{};
  p.l_mn = transL ? 1 : 0;
  p.r_mn = transR ? 0 : 1;
  p.nbi = (int)(rows / TILE); p.nbj = (int)(cols / TILE);
  p.c_rows = rows; p.c_cols = cols;
  p.alpha = alpha;
  p.status = c->status;
  CUtensorMap mL, mX, mR, mC;
  if (!make_map_2d(&mL, Lblk, TILE, rows, TILE, 32, p.l_mn ? 32 : TILE, p.l_mn != 0)) return ARMOR_ERR_CUDA;
  if (!make_map_2d(&mX, X, cols, rows, cols, 32, 32, true)) return ARMOR_ERR_CUDA;
  if (!make_map_2d(&mR, Rblk, TILE, cols, TILE, 32, p.r_mn ? 32 : TILE, p.r_mn != 0)) return ARMOR_ERR_CUDA;
  if (!make_map_2d(&mC, out, cols, rows, cols, 32, 32)) return ARMOR_ERR_CUDA;
  static PerDeviceOnce attr;
  if (ensure_dynamic_smem(attr, c->device, tc_block2_kernel, SMEM_BYTES) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int n_items = p.nbi * p.nbj;
  const int grid = n_items < c->n_sm ? n_items : c->n_sm;
  // one W-shaped read, one W-shaped write
  KTimer kt(c, ARMOR_KC_BLOCK_PRODUCT, 8.0 * (double)rows * (double)cols, s);
  tc_block2_kernel<<<grid, NTHREADS, SMEM_BYTES, s>>>(mL, mX, mR, mC, p);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}
