// Products with the block-diagonal wrappers (Section 3.1 of the paper) for d_block = 128, with the wrapper block
// held in TENSOR MEMORY as the M-side operand of tcgen05.mma and 128 x 256 accumulators.
//
// The streaming kernel of block_tcgen05.cu reads both operands of every MMA from shared memory: 8 KiB per
// 128 x 128 x 8 instruction, which at the instruction's 65 cycles is the whole shared-memory bandwidth of the SM.
// Here a CTA works through consecutive tiles of ONE wrapper block, two tiles (N = 256, 129 cycles) per instruction.
// The block (its fp32 words as the high part, x - trunc_tf32(x) as the low part) is written once into 2 x 128
// columns of tensor memory; the other 256 columns hold the accumulator; shared memory carries only the W-shaped
// operand (4 KiB per tile and instruction).  Measured on 4096 x 4096 the two kernels take the same time (both are
// within their head and tail of the HBM time of the pass), so the library uses the streaming one, which takes
// every d_block; this one is reachable through armor_block_product (path 2) and is the building block for
// products whose left operand is an accumulator (A from tensor memory).
//
//   side "left":   out[128 b + m][n]  = alpha * sum_k Qop_b[m][k] * X[128 b + k][n]  (+ beta * add)
//   side "right":  out[r][128 b + n]  = alpha * sum_k X[r][128 b + k] * Qop_b[k][n]  (+ beta * add)
//
// The right-hand product is issued transposed (M side = Qop_b^T from tensor memory, N side = the rows of X, a
// K-major operand), so its accumulator holds the tile transposed: lane = column of out.  The epilogue writes it
// into the swizzled staging boxes element by element (32 lanes write 32 consecutive words of a box row: no bank
// conflicts) and the TMA store is the same as on the left.
//
// Persistent kernel, 448 threads:
//   warp 0     : TMA producer (raw fp32 chunks of X, 32 along K, for one or two tiles; when the wrapper block changes,
//                the new block first, as two pieces through the same ring of stages)
//   warp 1     : MMA issuer   (tcgen05.mma kind::tf32 128 x 256 x 8 (128 x 128 x 8 for a single tile), A from
//                              tensor memory)
//   warps 2-5  : move the wrapper block from its two stages into tensor memory when the block changes (tcgen05.st),
//                then per chunk write the low part of X into a ring of its own
//   warps 6-13 : epilogue, four warps per tile of the pair (addend prefetched by TMA, tcgen05.ld, alpha / beta, TMA
//                store); the second half of a warp's share is taken into registers before the first half's store is
//                waited for, so the accumulator is released early
// The three MMAs per k-step are issued in the same order as in the streaming kernel (low part of the M-side
// operand of the UNtransposed product first), so both kernels give the same bits.
// Every wait is bounded; a wait that runs out raises a status word and the CTA leaves through the common exit that
// frees its tensor memory.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int TILE = 128, BK = 32;
constexpr int NTHREADS = 448;
constexpr int STAGES = 3;                         // raw chunks in flight
constexpr int LSTAGES = 2;                        // low-part chunks
constexpr int OP_BYTES = TILE * BK * 4;           // 16 KiB: one chunk of X for one tile
constexpr int STAGE_BYTES = 2 * OP_BYTES;         // a chunk for two tiles
constexpr uint32_t TMEM_COLS = 512;               // accumulator 0..255, wrapper high part 256..383, low part 384..511
constexpr uint32_t W_HI = 256, W_LO = 384;
constexpr int EPI_BYTES = 32 * 64 * 4;            // per epilogue warp: two swizzled 32 x 32 boxes
constexpr size_t LO_OFF = (size_t)STAGES * STAGE_BYTES, EPI_OFF = LO_OFF + (size_t)LSTAGES * STAGE_BYTES;
constexpr size_t SMEM_BYTES = EPI_OFF + 8 * EPI_BYTES + 1024;

struct XCoord {
  int mn_major;                     // 0: K-major (right), 1: N-major (left)
  int x_b, x_t, x_k;                // TMA x (inner) coordinate = x_b * block + x_t * tile + x_k * chunk
  int y_b, y_t, y_k;
};

struct RParams {
  XCoord x;
  int col_read;                     // 1: M-side operand element [m][k] = Q_b[k][m], 0: Q_b[m][k]
  int right;                        // 1: right-hand product (accumulator holds the tile transposed)
  const float* D;                   // addend or nullptr
  int64_t c_rows, c_cols;
  int tiles, batch;                 // tiles per wrapper block along the free dimension; work = batch * tiles tiles
  float alpha, beta;
  int32_t* status;
  int one_pass;
  int dual;                         // 1 (left only): the two halves of an instruction are the same tile of two inputs
                                    // (mapX, mapX2); out = alpha * Q.X2, dot_part = <Q.X1, Q.X2>
  double* dot_part;                 // dual: 8 partial sums per tile (one per epilogue warp), in tile order
};

// One or two neighbouring tiles of one wrapper block.
struct Unit { int b, t, nt; };
__device__ __forceinline__ bool next_unit(int& item, int i1, int tiles, int dual, Unit& u) {
  if (item >= i1) return false;
  u.b = item / tiles;
  u.t = item - u.b * tiles;
  u.nt = (dual || (u.t + 1 < tiles && item + 1 < i1)) ? 2 : 1;
  item += dual ? 1 : u.nt;
  return true;
}




__device__ __forceinline__ uint64_t x_desc(uint32_t base, int mn_major, int kstep) {
  return mn_major ? smem_desc_mn_sw128_32b(base + kstep * 1024, 4096, 512) : smem_desc_sw128(base + kstep * 32, 16, 1024);
}

__global__ void __launch_bounds__(NTHREADS, 1)
tc_blockres_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapX2,
                   const __grid_constant__ CUtensorMap mapQ,
                   const __grid_constant__ CUtensorMap mapC, const __grid_constant__ CUtensorMap mapD, const RParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[3 * STAGES + LSTAGES + 12];
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), split0 = smem_u32(&bars[STAGES]), empty0 = smem_u32(&bars[2 * STAGES]);
  const uint32_t lfree0 = smem_u32(&bars[3 * STAGES]);
  const uint32_t tfull = smem_u32(&bars[3 * STAGES + LSTAGES]), tempty = tfull + 8;
  const uint32_t wfull = tfull + 16, wfree = tfull + 24;
  const uint32_t dfull0 = tfull + 32;
  // the CTA's range of tiles (index = block * tiles + tile)
  // contiguous over all blocks, balanced to one tile
  const int64_t n_items = (int64_t)p.batch * p.tiles;
  const int i0 = (int)(n_items * blockIdx.x / gridDim.x), i1 = (int)(n_items * (blockIdx.x + 1) / gridDim.x);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(split0 + 8 * s, 4);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int s = 0; s < LSTAGES; ++s) mbar_init(lfree0 + 8 * s, 1);
    mbar_init(tfull, 1);
    mbar_init(tempty, 8);
    mbar_init(wfull, 4);
    mbar_init(wfree, 1);
    for (int s = 0; s < 8; ++s) mbar_init(dfull0 + 8 * s, 1);
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
      int cur_b = -1;
      Unit u;
      for (int item = i0; ok && next_unit(item, i1, p.tiles, p.dual, u);) {
        if (u.b != cur_b) {
          // the wrapper block: two pieces of 64 columns, each two boxes of 128 rows x 32 columns
          for (int piece = 0; piece < 2; ++piece) {
            if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
            const uint32_t fb = full0 + 8 * stage;
            mbar_expect_tx(fb, 2 * OP_BYTES);
            const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
            tma_load_2d(dst, &mapQ, 64 * piece, TILE * u.b, fb);
            tma_load_2d(dst + OP_BYTES, &mapQ, 64 * piece + 32, TILE * u.b, fb);
            ++issued;
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (!ok) break;
          cur_b = u.b;
        }
        for (int kc = 0; kc < TILE / BK; ++kc) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, (uint32_t)(u.nt * OP_BYTES));
          const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          for (int j = 0; j < u.nt; ++j) {
            const int tj = p.dual ? u.t : u.t + j;                      // dual: the same tile of the second input
            const CUtensorMap* mx = (p.dual && j) ? &mapX2 : &mapX;
            const int x = p.x.x_b * u.b + p.x.x_t * tj + p.x.x_k * kc;
            const int y = p.x.y_b * u.b + p.x.y_t * tj + p.x.y_k * kc;
            if (p.x.mn_major) {
#pragma unroll
              for (int q = 0; q < 4; ++q) tma_load_2d(dst + (j * 4 + q) * 4096, mx, x + 32 * q, y, fb);
            } else {
              tma_load_2d(dst + j * OP_BYTES, mx, x, y, fb);
            }
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
      const uint32_t idesc1 = instr_desc_tf32_mn(TILE, TILE, 0, p.x.mn_major);
      const uint32_t idesc2 = instr_desc_tf32_mn(TILE, 2 * TILE, 0, p.x.mn_major);
      const uint64_t dx0 = x_desc(smem_u32(smem), p.x.mn_major, 0), dl0 = x_desc(smem_u32(smem + LO_OFF), p.x.mn_major, 0);
      const uint64_t kinc = p.x.mn_major ? (1024u >> 4) : (32u >> 4);     // one k-step of 8 in the address field
      const uint32_t w_hi0 = tmem_base + W_HI, w_lo0 = tmem_base + W_LO;
      int stage = 0; uint32_t phase = 0;
      int lst = 0; uint32_t lphase = 0;
      int cur_b = -1;
      uint32_t local = 0, w_loads = 0;          // units issued, wrapper blocks waited for
      bool ok = true;
      Unit u;
      for (int item = i0; ok && next_unit(item, i1, p.tiles, p.dual, u); ++local) {
        if (u.b != cur_b) {
          if (!mbar_wait(wfull, w_loads & 1u, abortp, p.status)) { ok = false; break; }
          ++w_loads;
          cur_b = u.b;
          for (int piece = 0; piece < 2; ++piece)       // the block's two pieces went through the ring
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!mbar_wait(tempty, (local & 1u) ^ 1u, abortp, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t idesc = u.nt == 2 ? idesc2 : idesc1;
        for (int kc = 0; kc < TILE / BK; ++kc) {
          if (!mbar_wait(split0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          // One thread issues every MMA, so the instructions around each tcgen05.mma are what bounds the rate (a
          // descriptor built from scratch per MMA costs more than the MMA takes to execute): the descriptors of
          // stage 0 are formed once and only their address field moves.
          const uint64_t dx = dx0 + (uint64_t)(uint32_t)(stage * (STAGE_BYTES >> 4));
          const uint64_t dxl = dl0 + (uint64_t)(uint32_t)(lst * (STAGE_BYTES >> 4));
          const uint32_t w_hi = w_hi0 + (uint32_t)(kc * BK), w_lo = w_lo0 + (uint32_t)(kc * BK);
          if (p.one_pass) {
            umma_tf32_ta(tmem_base, w_hi, dx, idesc, (uint32_t)(kc > 0));
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) umma_tf32_ta_acc(tmem_base, w_hi + 8 * k, dx + k * kinc, idesc);
          } else if (p.right) {
            // low part of X (the M side of the untransposed product) first
            umma_tf32_ta(tmem_base, w_hi, dxl, idesc, (uint32_t)(kc > 0));
            umma_tf32_ta_acc(tmem_base, w_lo, dx, idesc);
            umma_tf32_ta_acc(tmem_base, w_hi, dx, idesc);
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) {
              umma_tf32_ta_acc(tmem_base, w_hi + 8 * k, dxl + k * kinc, idesc);
              umma_tf32_ta_acc(tmem_base, w_lo + 8 * k, dx + k * kinc, idesc);
              umma_tf32_ta_acc(tmem_base, w_hi + 8 * k, dx + k * kinc, idesc);
            }
          } else {
            umma_tf32_ta(tmem_base, w_lo, dx, idesc, (uint32_t)(kc > 0));
            umma_tf32_ta_acc(tmem_base, w_hi, dxl, idesc);
            umma_tf32_ta_acc(tmem_base, w_hi, dx, idesc);
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) {
              umma_tf32_ta_acc(tmem_base, w_lo + 8 * k, dx + k * kinc, idesc);
              umma_tf32_ta_acc(tmem_base, w_hi + 8 * k, dxl + k * kinc, idesc);
              umma_tf32_ta_acc(tmem_base, w_hi + 8 * k, dx + k * kinc, idesc);
            }
          }
          umma_commit(empty0 + 8 * stage);   // frees the raw chunk and the low-part chunk once these MMAs have read them
          umma_commit(lfree0 + 8 * lst);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
          if (++lst == LSTAGES) { lst = 0; lphase ^= 1; }
        }
        if (!ok) break;
        umma_commit(tfull);
        // the last tiles of this wrapper block: tensor memory may be rewritten once these MMAs have read it
        if (item < i1 && item / p.tiles != u.b) umma_commit(wfree);
      }
      (void)lphase;
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ wrapper block -> tensor memory, low parts of X
    const int q = warp & 3;                    // TMEM lane quarter this warp may write
    const int t = threadIdx.x - 64;            // 0..127
    const int m = q * 32 + lane;               // row of the M-side operand this thread holds
    const uint32_t lane_sel = (uint32_t)(q * 32) << 16;
    int stage = 0; uint32_t phase = 0;
    int lst = 0; uint32_t lphase = 0;
    int cur_b = -1;
    uint32_t w_loads = 0;
    bool ok = true;
    Unit u;
    for (int item = i0; ok && next_unit(item, i1, p.tiles, p.dual, u);) {
      if (u.b != cur_b) {
        // The block arrives as two pieces, each a stage holding two boxes of 128 rows x 32 columns (rows of 128
        // bytes, 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r % 8)); box g of the block covers
        // its columns 32 g ..
#pragma unroll 1
        for (int piece = 0; piece < 2 && ok; ++piece) {
          if (!__all_sync(0xffffffffu, mbar_wait(full0 + 8 * stage, phase, abortp, p.status))) { ok = false; break; }
          if (piece == 0 && w_loads > 0) {
            // the MMAs of the previous block have read the old contents of tensor memory
            if (!__all_sync(0xffffffffu, mbar_wait(wfree, (w_loads - 1) & 1u, abortp, p.status))) { ok = false; break; }
            tc_fence_after();
          }
          const uint8_t* pb = smem + (size_t)stage * STAGE_BYTES;
          if (p.col_read) {
            // element [m][k] = Q_b[k][m]: column m lives in box q, word `lane` of row k
            if ((q >> 1) == piece) {
              const uint8_t* colp = pb + (q & 1) * OP_BYTES + (lane & 3) * 4;
#pragma unroll 1
              for (int k0 = 0; k0 < TILE; k0 += 32) {
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  hi[i] = *reinterpret_cast<const uint32_t*>(colp + (k0 + i) * 128 + (((lane >> 2) ^ (i & 7)) << 4));
                tmem_st32(tmem_base + W_HI + (uint32_t)k0 + lane_sel, hi);
                if (!p.one_pass) {
#pragma unroll
                  for (int i = 0; i < 32; ++i)
                    lo[i] = __float_as_uint(__uint_as_float(hi[i]) - __uint_as_float(hi[i] & 0xffffe000u));
                  tmem_st32(tmem_base + W_LO + (uint32_t)k0 + lane_sel, lo);
                }
              }
            }
          } else {
            // element [m][k] = Q_b[m][k]: row m of the boxes for k = 64 piece + 32 g ..
#pragma unroll 1
            for (int g = 0; g < 2; ++g) {
              const uint8_t* rowp = pb + g * OP_BYTES + m * 128;
              const uint32_t k0 = (uint32_t)(64 * piece + 32 * g);
              uint32_t hi[32], lo[32];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + ((i ^ (m & 7)) << 4));
                hi[4 * i] = v.x; hi[4 * i + 1] = v.y; hi[4 * i + 2] = v.z; hi[4 * i + 3] = v.w;
              }
              tmem_st32(tmem_base + W_HI + k0 + lane_sel, hi);
              if (!p.one_pass) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  lo[i] = __float_as_uint(__uint_as_float(hi[i]) - __uint_as_float(hi[i] & 0xffffe000u));
                tmem_st32(tmem_base + W_LO + k0 + lane_sel, lo);
              }
            }
          }
          // the stage goes back to the producer once all four warps have read it (every barrier of a stage
          // completes once per pass of the ring, whatever the stage carried)
          __syncwarp();
          if (lane == 0) mbar_arrive(split0 + 8 * stage);
          if (t == 0) {
            if (mbar_wait(split0 + 8 * stage, phase, abortp, p.status)) mbar_arrive(empty0 + 8 * stage);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(wfull);
        ++w_loads;
        cur_b = u.b;
      }
      for (int kc = 0; kc < TILE / BK; ++kc) {
        if (!mbar_wait(full0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
        if (!mbar_wait(lfree0 + 8 * lst, lphase ^ 1, abortp, p.status)) { ok = false; break; }
        if (!p.one_pass) {
          const float4* hi = reinterpret_cast<const float4*>(smem + (size_t)stage * STAGE_BYTES);
          float4* lo = reinterpret_cast<float4*>(smem + LO_OFF + (size_t)lst * STAGE_BYTES);
          const int n4 = u.nt * (OP_BYTES / 16 / 128);
#pragma unroll 4
          for (int e = 0; e < n4; ++e) {
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
        if (++lst == LSTAGES) { lst = 0; lphase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int e = warp - 6;                 // 0..7
    const int h = e >> 2;                   // which tile of the pair this warp stores
    uint32_t local = 0;
    uint32_t d_loads = 0;   // addend slabs requested so far: parity of their barrier
    bool ok = true;
    uint8_t* buf = smem + EPI_OFF + (size_t)e * EPI_BYTES;   // two 4 KiB boxes of 32 x 32
    const uint32_t buf_u32 = smem_u32(buf);
    const uint32_t dbar = dfull0 + 8 * e;
    Unit u;
    for (int item = i0; ok && next_unit(item, i1, p.tiles, p.dual, u); ++local) {
      if (p.dual) {
        // Accumulator columns 0..127 hold Q.X1 and 128..255 hold Q.X2 of the same tile.  Warp (q, h) takes rows
        // 32 q .. and columns 64 h .. of the tile: both products of its two boxes, their dot product, and the store
        // of alpha * Q.X2.
        const int64_t row0 = (int64_t)TILE * u.b + 32 * q, col0 = (int64_t)TILE * u.t + 64 * h;
        int n_box = 0;
        for (int ch = 0; ch < 2; ++ch) n_box += (col0 + 32 * ch < p.c_cols && row0 < p.c_rows) ? 1 : 0;
        if (lane == 0) tma_store_wait_read();        // the previous stores have read the staging boxes
        __syncwarp();
        if (!__all_sync(0xffffffffu, mbar_wait(tfull, local & 1u, abortp, p.status))) { ok = false; break; }
        tc_fence_after();
        double dot = 0.0;
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t r1[32], r2[32];
          const uint32_t col = (uint32_t)(64 * h + 32 * ch) + ((uint32_t)(q * 32) << 16);
          tmem_ld32(tmem_base + col, r1);
          tmem_ld32(tmem_base + (uint32_t)TILE + col, r2);
          float part = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) part = fmaf(__uint_as_float(r1[i]), __uint_as_float(r2[i]), part);
          dot += (double)part;
          if (ch >= n_box) continue;                 // warp-uniform
          uint8_t* rowp = buf + ch * 4096 + lane * 128;
#pragma unroll
          for (int cq = 0; cq < 8; ++cq) {
            float4* cell = reinterpret_cast<float4*>(rowp + ((cq ^ (lane & 7)) << 4));
            *cell = make_float4(p.alpha * __uint_as_float(r2[4 * cq]), p.alpha * __uint_as_float(r2[4 * cq + 1]),
                                p.alpha * __uint_as_float(r2[4 * cq + 2]), p.alpha * __uint_as_float(r2[4 * cq + 3]));
          }
        }
        tc_fence_before();                           // all reads of the accumulator are done
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(tempty);
          for (int ch = 0; ch < n_box; ++ch)
            tma_store_2d(&mapC, (int)(col0 + 32 * ch), (int)row0, buf_u32 + ch * 4096);
          tma_store_commit();
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        if (lane == 0) p.dot_part[((size_t)u.b * p.tiles + u.t) * 8 + e] = dot;
        continue;
      }
      if (h >= u.nt) {
        // a single tile: nothing to store, but the accumulator's hand-over is counted per warp
        if (!__all_sync(0xffffffffu, mbar_wait(tfull, local & 1u, abortp, p.status))) { ok = false; break; }
        if (lane == 0) mbar_arrive(tempty);
        continue;
      }
      const int tt = u.t + h;
      // origin of the 128 x 128 tile in out
      const int64_t row_tile = (int64_t)TILE * (p.right ? tt : u.b);
      const int64_t col_tile = (int64_t)TILE * (p.right ? u.b : tt);
      // The warp's share of the tile goes through shared memory in two halves of two 32 x 32 boxes.  Left: the
      // warp holds rows 32 q .. of the tile and box (hf, ch) covers columns 64 hf + 32 ch ..; right: the warp holds
      // columns 32 q .. and box (hf, ch) covers rows 64 hf + 32 ch ..  Either way the accumulator columns
      // 128 h + 64 hf + 32 ch .. of the warp's lanes hold the box.
      const int bxs = p.right ? 0 : 32, bys = p.right ? 32 : 0;      // step from box 0 to box 1 of a half
      int64_t bx0[2], by0[2];
      int n_box[2];                  // boxes of each half that start inside out (warp-uniform); the TMA clips a box
      for (int hf = 0; hf < 2; ++hf) {
        bx0[hf] = p.right ? col_tile + 32 * q : col_tile + 64 * hf;
        by0[hf] = p.right ? row_tile + 64 * hf : row_tile + 32 * q;
        n_box[hf] = 0;
        for (int ch = 0; ch < 2; ++ch)
          n_box[hf] += (bx0[hf] + bxs * ch < p.c_cols && by0[hf] + bys * ch < p.c_rows) ? 1 : 0;
      }
      // alpha * accumulator (+ beta * addend, which sits in the box already) into staging box ch
      auto stage_box = [&](int ch, const uint32_t (&r)[32]) {
        if (p.right) {
          // r[i] = out[by + i][bx + lane]: word `lane` of box row i; 16-byte chunk c of a row sits at chunk
          // c ^ (row % 8)  (128-byte swizzle)
          uint8_t* colp = buf + ch * 4096 + (lane & 3) * 4;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float* cell = reinterpret_cast<float*>(colp + i * 128 + (((lane >> 2) ^ (i & 7)) << 4));
            float v = p.alpha * __uint_as_float(r[i]);
            if (p.D) v = fmaf(p.beta, *cell, v);
            *cell = v;
          }
        } else {
          // lane = row of the box
          uint8_t* rowp = buf + ch * 4096 + lane * 128;
#pragma unroll
          for (int cq = 0; cq < 8; ++cq) {
            float4* cell = reinterpret_cast<float4*>(rowp + ((cq ^ (lane & 7)) << 4));
            float4 v = make_float4(p.alpha * __uint_as_float(r[4 * cq]), p.alpha * __uint_as_float(r[4 * cq + 1]),
                                   p.alpha * __uint_as_float(r[4 * cq + 2]), p.alpha * __uint_as_float(r[4 * cq + 3]));
            if (p.D) {
              const float4 d = *cell;
              v.x = fmaf(p.beta, d.x, v.x); v.y = fmaf(p.beta, d.y, v.y);
              v.z = fmaf(p.beta, d.z, v.z); v.w = fmaf(p.beta, d.w, v.w);
            }
            *cell = v;
          }
        }
      };
      // staging boxes free (the previous stores have read them); the addend of half hf requested
      auto open_half = [&](int hf) {
        if (lane == 0) {
          tma_store_wait_read();
          if (p.D && n_box[hf] > 0) {
            mbar_expect_tx(dbar, (uint32_t)n_box[hf] * 4096u);
            for (int ch = 0; ch < n_box[hf]; ++ch)
              tma_load_2d(buf_u32 + ch * 4096, &mapD, (int)(bx0[hf] + bxs * ch), (int)(by0[hf] + bys * ch), dbar);
          }
        }
        __syncwarp();
      };
      auto store_half = [&](int hf) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          for (int ch = 0; ch < n_box[hf]; ++ch)
            tma_store_2d(&mapC, (int)(bx0[hf] + bxs * ch), (int)(by0[hf] + bys * ch), buf_u32 + ch * 4096);
          tma_store_commit();
        }
      };
      const uint32_t tacc = tmem_base + (uint32_t)(h * TILE) + ((uint32_t)(q * 32) << 16);

      open_half(0);                                  // the addend's first half travels while the MMAs run
      if (!__all_sync(0xffffffffu, mbar_wait(tfull, local & 1u, abortp, p.status))) { ok = false; break; }
      tc_fence_after();
      if (p.D && n_box[0] > 0) {
        if (!__all_sync(0xffffffffu, mbar_wait(dbar, d_loads & 1u, abortp, p.status))) { ok = false; break; }
        ++d_loads;
      }
#pragma unroll 1
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t r[32];
        tmem_ld32(tacc + (uint32_t)(ch * 32), r);
        if (ch < n_box[0]) stage_box(ch, r);         // warp-uniform
      }
      store_half(0);
      // the second half is taken into registers at once, so that the accumulator goes back to the MMA issuer
      // before this warp waits for its first store
      uint32_t r2[32], r3[32];
      tmem_ld32(tacc + 64u, r2);
      tmem_ld32(tacc + 96u, r3);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty);
      open_half(1);
      if (p.D && n_box[1] > 0) {
        if (!__all_sync(0xffffffffu, mbar_wait(dbar, d_loads & 1u, abortp, p.status))) { ok = false; break; }
        ++d_loads;
      }
      if (0 < n_box[1]) stage_box(0, r2);
      if (1 < n_box[1]) stage_box(1, r3);
      store_half(1);
    }
    if (lane == 0) tma_store_wait_read();           // shared memory stays valid until the stores have read it
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

armor_status launch(armor_ctx* c, const float* X, const float* Q, int64_t rows, int64_t cols, RParams p, float* out,
                    cudaStream_t s, const float* X2 = nullptr) {
  CUtensorMap mX, mX2, mQ, mC, mD;
  if (!make_map_2d(&mQ, Q, TILE, (int64_t)p.batch * TILE, TILE, 32, TILE)) return ARMOR_ERR_CUDA;
  if (!make_map_2d(&mC, out, cols, rows, cols, 32, 32)) return ARMOR_ERR_CUDA;
  if (p.D) {
    if (!make_map_2d(&mD, p.D, cols, rows, cols, 32, 32)) return ARMOR_ERR_CUDA;
  } else {
    mD = mC;
  }
  if (!make_map_2d(&mX, X, cols, rows, cols, 32, p.x.mn_major ? 32 : TILE, p.x.mn_major != 0)) return ARMOR_ERR_CUDA;
  if (X2) {
    if (!make_map_2d(&mX2, X2, cols, rows, cols, 32, p.x.mn_major ? 32 : TILE, p.x.mn_major != 0)) return ARMOR_ERR_CUDA;
  } else {
    mX2 = mX;
  }
  p.c_rows = rows; p.c_cols = cols;
  p.status = c->status;
  p.one_pass = c->block_one_pass;
  static PerDeviceOnce attr;
  if (ensure_dynamic_smem(attr, c->device, tc_blockres_kernel, SMEM_BYTES) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int64_t n_items = (int64_t)p.batch * p.tiles;
  const int grid = (int)(n_items < c->n_sm ? n_items : c->n_sm);
  KTimer kt(c, ARMOR_KC_BLOCK_PRODUCT, ((p.D || p.dual) ? 12.0 : 8.0) * (double)rows * (double)cols, s);
  tc_blockres_kernel<<<grid, NTHREADS, SMEM_BYTES, s>>>(mX, mX2, mQ, mC, mD, p);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

inline bool ptr_ok(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

}  // namespace

bool tc_blockres_ok(const armor_ctx* c) { return c->db == TILE; }

// out[:, j-th block] = alpha * in[:, j-th block] * Q_j (+ beta * add[:, j-th block]),  Q_j = Bblk[j] or its transpose
armor_status tc_blockres_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
                               int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  if (!ptr_ok(in) || !ptr_ok(Bblk) || !ptr_ok(out) || (add && !ptr_ok(add))) return ARMOR_ERR_UNSUPPORTED;
  RParams p{};
  p.x = {0, TILE, 0, BK, 0, TILE, 0};     // N side [n = row of in][k]: x = 128 j + 32 kc, y = 128 t  (K-major)
  p.col_read = transB ? 0 : 1; p.right = 1;
  p.D = add; p.alpha = alpha; p.beta = add ? beta : 0.f;
  p.batch = (int)(cols / TILE); p.tiles = (int)((rows + TILE - 1) / TILE);
  return launch(c, in, Bblk, rows, cols, p, out, s);
}

// out[i-th block, :] = alpha * P_i * in[i-th block, :] (+ beta * add[i-th block, :]),  P_i = Ablk[i] or its transpose
armor_status tc_blockres_left(armor_ctx* c, const float* Ablk, bool transA, const float* in, float* out, int64_t rows,
                              int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  if (!ptr_ok(in) || !ptr_ok(Ablk) || !ptr_ok(out) || (add && !ptr_ok(add))) return ARMOR_ERR_UNSUPPORTED;
  RParams p{};
  p.x = {1, 0, TILE, 0, TILE, 0, BK};     // N side [n = column of in][k]: x = 128 t, y = 128 i + 32 kc  (N-major)
  p.col_read = transA ? 1 : 0; p.right = 0;
  p.D = add; p.alpha = alpha; p.beta = add ? beta : 0.f;
  p.batch = (int)(rows / TILE); p.tiles = (int)((cols + TILE - 1) / TILE);
  return launch(c, in, Ablk, rows, cols, p, out, s);
}

// out[i-th block, :] = P_i * in2[i-th block, :] and 8 partial sums per 128 x 128 tile of <P_i * in1, P_i * in2> at part
// (tile order, then the eight 32 x 64 pieces of the tile); the number of partial sums comes back through n_part
armor_status tc_blockres_left_dual(armor_ctx* c, const float* Ablk, const float* in1, const float* in2, float* out,
                                   int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s) {
  if (!ptr_ok(in1) || !ptr_ok(in2) || !ptr_ok(Ablk) || !ptr_ok(out)) return ARMOR_ERR_UNSUPPORTED;
  RParams p{};
  p.x = {1, 0, TILE, 0, TILE, 0, BK};
  p.col_read = 0; p.right = 0;
  p.D = nullptr; p.alpha = 1.f; p.beta = 0.f;
  p.batch = (int)(rows / TILE); p.tiles = (int)((cols + TILE - 1) / TILE);
  p.dual = 1; p.dot_part = part;
  *n_part = 8 * p.batch * p.tiles;
  return launch(c, in1, Ablk, rows, cols, p, out, s, in2);
}
