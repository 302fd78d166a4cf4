// Batched 128 x 128 x K products on the tensor cores for the block-diagonal wrappers (Section 3.1 of the
// paper: A and B are block diagonal, so A.Y and Y.B are one small dense product per d_block x d_block tile
// of the W-shaped operand).  Per tile the product has only 2*d_block flops per element moved, so these passes
// are bound by HBM once the arithmetic runs on the tensor cores.
//
//   C_tile = alpha * sum_k Aop[m][k] * Bop[n][k] (+ beta * D_tile)
//
// Both operands are plain fp32 in global memory.  Either may be K-major (k contiguous) or MN-major (m or n
// contiguous); tcgen05 reads both from swizzled shared memory (MN-major 32-bit operands in the 128-byte swizzle
// with 32-byte atoms, which TMA writes directly), so no transposed copies are made.
// fp32-grade accuracy comes from splitting every operand chunk, in shared memory, into a high part and an fp32
// low part and issuing three MMAs (lo*hi + hi*lo + hi*hi) into one fp32 accumulator.  The tensor core reads the
// top 19 bits of a 32-bit tf32 operand and ignores the rest, so the raw fp32 word serves as the high part and
// only the low part x - trunc_tf32(x) has to be written (checked against a masked copy: same bits).
//
// Persistent kernel, 320 threads:
//   warp 0    : TMA producer (raw fp32 chunks of 32 along K; MN-major chunks as four 32 x 32 boxes)
//   warp 1    : MMA issuer   (tcgen05.mma kind::tf32, 128 x 128 x 8, two accumulators of 128 TMEM columns)
//   warps 2-5 : splitter     (raw chunk -> low part next to it, proxy fence)
//   warps 6-9 : epilogue     (D tile prefetched by TMA into swizzled shared memory, tcgen05.ld, alpha / beta
//                             in place, TMA store: no strided global access)
// Dual mode: two inputs share the wrapper, A.X1 and A.X2 of a tile go through the pipeline back to back into
// two accumulators, and the epilogue stores alpha * A.X2 only and writes partial sums of <A.X1, A.X2> (the
// quadratic form of a line search needs the first product only inside that dot product, so it never
// reaches HBM).
// Every wait is bounded; a wait that runs out raises a status word and the CTA leaves through the common
// exit that frees its tensor memory.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int TILE = 128, BK = 32;
constexpr int NTHREADS = 320;
constexpr int OP_BYTES = TILE * BK * 4;           // 16 KiB: one operand chunk
// A stage holds SLOTS operand chunks, each as its raw words (= high part) followed by its low part: the M-side and the
// N-side chunk, and in the pair mode with a shared N side a second M-side chunk.
template <int SLOTS> struct Geo {
  static constexpr int STAGES = SLOTS == 3 ? 2 : 3;
  static constexpr int STAGE_BYTES = 2 * SLOTS * OP_BYTES;
};
constexpr uint32_t TMEM_COLS = 512;               // four accumulators of 128 columns (two in use outside the dual mode)
constexpr int EPI_BYTES = 32 * 64 * 4;            // per epilogue warp: 32 rows x 64 columns (half a tile row) as two swizzled boxes
template <int SLOTS> constexpr size_t smem_bytes() {
  return (size_t)Geo<SLOTS>::STAGES * Geo<SLOTS>::STAGE_BYTES + 4 * EPI_BYTES + 1024;
}

struct OpCoord {
  int mn_major;                     // 0: K-major, 1: MN-major
  int x_b, x_t, x_k;                // TMA x (inner) coordinate = x_b * batch + x_t * tile + x_k * chunk
  int y_b, y_t, y_k;                // TMA y (outer) coordinate likewise
};

struct BParams {
  OpCoord a, b;
  float* C; const float* D;
  int64_t ldc, ldd;
  int64_t c_rows, c_cols;           // extent of C (stores are guarded)
  int64_t r_b, c_b;                 // tile origin: row = r_b * batch + 128 * tm (+ r_s * split), column = c_b * batch + 128 * tn
  int64_t r_s;
  int m_valid;                      // rows of a batch's tile range that exist (boxes of 32 rows beyond it are not stored)
  int m_tiles, n_tiles, batch, k_chunks;   // k_chunks: chunks of 32 along K per work item
  int n_split;                      // the contraction is cut into n_split items of k_chunks chunks each
  float alpha, beta;
  int32_t* status;
  int batch_fastest;                // 1: consecutive work items are consecutive batches (neighbouring column blocks)
  int one_pass;                     // 1: operands as they are, rounded to tf32 by the tensor core; no low parts
  int pair;                         // two products per tile into two accumulators from the SAME stages, both stored (C
                                    // and, through mapD, C2).  1: a second M-side operand (mapB2, addressed like A):
                                    // C = A.B, C2 = A2.B;  2: the M-side chunk also serves as N side: C = A.A^T-like
                                    // (the operand with itself), C2 = A.B
  int dual;                         // 1: two B operands per tile (mapB, mapB2); C = alpha * A.B2, dot_part = <A.B1, A.B2>
  double* dot_part;                 // dual, colw: 4 partial sums per tile (one per epilogue warp), in tile order
  const float* colw;                // not null: a second output C2 (through mapB2) = C scaled per column by colw, and
                                    // dot_part = sum of C * C2 (the residual, its weighted form and the loss of the
                                    // diagonal weighting, Eq. 2 with H_w = diag(h), in one pass)
};

__device__ __forceinline__ void load_operand(uint32_t dst, const CUtensorMap* map, const OpCoord& o, int b, int t, int kc,
                                             uint32_t bar) {
  const int x = o.x_b * b + o.x_t * t + o.x_k * kc;
  const int y = o.y_b * b + o.y_t * t + o.y_k * kc;
  if (o.mn_major) {
#pragma unroll
    for (int q = 0; q < 4; ++q) tma_load_2d(dst + q * 4096, map, x + 32 * q, y, bar);
  } else {
    tma_load_2d(dst, map, x, y, bar);
  }
}

__device__ __forceinline__ void item_decode(const BParams& p, int item, int& tn, int& tm, int& b, int& ks) {
  if (p.batch_fastest) {
    b = item % p.batch;
    const int rest = item / p.batch;
    tn = rest % p.n_tiles;
    tm = (rest / p.n_tiles) % p.m_tiles;
    ks = rest / (p.n_tiles * p.m_tiles);
  } else {
    tn = item % p.n_tiles;
    tm = (item / p.n_tiles) % p.m_tiles;
    b = (item / (p.n_tiles * p.m_tiles)) % p.batch;
    ks = item / (p.n_tiles * p.m_tiles * p.batch);
  }
}

__device__ __forceinline__ uint64_t operand_desc(uint32_t base, int mn_major, int kstep) {
  // K-major: 8 columns of K are 32 bytes further along the 128-byte row.
  // MN-major: 8 k-rows are two groups of 4 k-rows (512 bytes each); 32 more elements along M / N are the next
  // 4 KiB box.
  return mn_major ? smem_desc_mn_sw128_32b(base + kstep * 1024, 4096, 512) : smem_desc_sw128(base + kstep * 32, 16, 1024);
}


template <int SLOTS>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_block_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                const __grid_constant__ CUtensorMap mapB2, const __grid_constant__ CUtensorMap mapC,
                const __grid_constant__ CUtensorMap mapD, const BParams p) {
  constexpr int STAGES = Geo<SLOTS>::STAGES, STAGE_BYTES = Geo<SLOTS>::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[3 * STAGES + 12];
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), split0 = smem_u32(&bars[STAGES]), empty0 = smem_u32(&bars[2 * STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[3 * STAGES]), tempty0 = smem_u32(&bars[3 * STAGES + 4]);
  const uint32_t dfull0 = smem_u32(&bars[3 * STAGES + 8]);
  const int n_items = p.batch * p.m_tiles * p.n_tiles * p.n_split;   // tiles (x slabs of the contraction)
  const int n_sub = p.dual ? 2 : 1;                                  // passes through the pipeline per tile
  const int n_acc = (p.dual || p.pair) ? 2 : 1;                      // accumulators per tile

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(split0 + 8 * s, 4);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int s = 0; s < 4; ++s) { mbar_init(tfull0 + 8 * s, 1); mbar_init(tempty0 + 8 * s, 4); }
    for (int s = 0; s < 4; ++s) mbar_init(dfull0 + 8 * s, 1);
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
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        int tn, tm, b, ks;
        item_decode(p, item, tn, tm, b, ks);
        for (int sub = 0; sub < n_sub && ok; ++sub)
        for (int kc = 0; kc < p.k_chunks; ++kc) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, SLOTS * OP_BYTES);
          const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          load_operand(dst, &mapA, p.a, b, tm, ks * p.k_chunks + kc, fb);
          load_operand(dst + 2 * OP_BYTES, sub ? &mapB2 : &mapB, p.b, b, tn, ks * p.k_chunks + kc, fb);
          if (SLOTS == 3) load_operand(dst + 4 * OP_BYTES, &mapB2, p.a, b, tm, ks * p.k_chunks + kc, fb);
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
      const uint32_t idesc = instr_desc_tf32_mn(TILE, TILE, p.a.mn_major, p.b.mn_major);
      const uint64_t da0 = operand_desc(smem_u32(smem), p.a.mn_major, 0);
      const uint64_t db0 = operand_desc(smem_u32(smem) + 2 * OP_BYTES, p.b.mn_major, 0);
      const uint64_t kinc_a = p.a.mn_major ? (1024u >> 4) : (32u >> 4);   // one k-step of 8 in the address field
      const uint64_t kinc_b = p.b.mn_major ? (1024u >> 4) : (32u >> 4);
      const uint32_t idesc_self = instr_desc_tf32_mn(TILE, TILE, p.a.mn_major, p.a.mn_major);   // pair 2: A chunk on both sides
      int stage = 0; uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x)
      for (int sub = 0; sub < n_sub && ok; ++sub, ++local) {
        // accumulators rotate: two of them, or (dual, pair) four, of which a tile takes two
        const int as = p.pair ? ((2 * local) & 3) : (local & (2 * n_acc - 1));
        const uint32_t aphase = (uint32_t)(local >> (p.pair ? 1 : n_acc)) & 1u;
        if (!mbar_wait(tempty0 + 8 * as, aphase ^ 1, abortp, p.status)) { ok = false; break; }
        if (p.pair && !mbar_wait(tempty0 + 8 * (as + 1), aphase ^ 1, abortp, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(as * TILE);
        for (int kc = 0; kc < p.k_chunks; ++kc) {
          if (!mbar_wait(split0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          // One thread issues every MMA, so the instructions around each tcgen05.mma bound the rate (a descriptor
          // built from scratch per MMA costs more than the MMA takes to execute): the descriptors of stage 0 are
          // formed once and only their address field moves.
          const uint64_t so = (uint64_t)(uint32_t)(stage * (STAGE_BYTES >> 4));
          const uint64_t da = da0 + so, dal = da + (OP_BYTES >> 4);
          const uint64_t dbm = db0 + so, dbl = dbm + (OP_BYTES >> 4);
          const uint32_t first = (uint32_t)(kc > 0);
          if (p.pair) {
            // two products from the same stage.  Accumulator 0: pair 1 A.B, pair 2 the M-side chunk with itself as N
            // side; accumulator 1: pair 1 A2.B (third slot), pair 2 A.B.  Per accumulator the order of the one-product
            // kernel (low part of the M side first).
            const uint32_t tacc1 = tacc + (uint32_t)TILE;
            const uint64_t m1 = (p.pair == 1) ? da + (4 * OP_BYTES >> 4) : da, m1l = m1 + (OP_BYTES >> 4);   // M side of accumulator 1
            const uint64_t n0 = (p.pair == 1) ? dbm : da, n0l = n0 + (OP_BYTES >> 4);                       // N side of accumulator 0
            const uint64_t kinc_n0 = (p.pair == 1) ? kinc_b : kinc_a;
            const uint32_t id0 = (p.pair == 1) ? idesc : idesc_self;
#pragma unroll
            for (int k = 0; k < BK / 8; ++k) {
              if (k == 0) umma_tf32(tacc, dal, n0, id0, first); else umma_tf32_acc(tacc, dal + k * kinc_a, n0 + k * kinc_n0, id0);
              umma_tf32_acc(tacc, da + k * kinc_a, n0l + k * kinc_n0, id0);
              umma_tf32_acc(tacc, da + k * kinc_a, n0 + k * kinc_n0, id0);
            }
#pragma unroll
            for (int k = 0; k < BK / 8; ++k) {
              if (k == 0) umma_tf32(tacc1, m1l, dbm, idesc, first); else umma_tf32_acc(tacc1, m1l + k * kinc_a, dbm + k * kinc_b, idesc);
              umma_tf32_acc(tacc1, m1 + k * kinc_a, dbl + k * kinc_b, idesc);
              umma_tf32_acc(tacc1, m1 + k * kinc_a, dbm + k * kinc_b, idesc);
            }
          } else if (p.one_pass) {
            umma_tf32(tacc, da, dbm, idesc, first);
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) umma_tf32_acc(tacc, da + k * kinc_a, dbm + k * kinc_b, idesc);
          } else {
            umma_tf32(tacc, dal, dbm, idesc, first);
            umma_tf32_acc(tacc, da, dbl, idesc);
            umma_tf32_acc(tacc, da, dbm, idesc);
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) {
              umma_tf32_acc(tacc, dal + k * kinc_a, dbm + k * kinc_b, idesc);
              umma_tf32_acc(tacc, da + k * kinc_a, dbl + k * kinc_b, idesc);
              umma_tf32_acc(tacc, da + k * kinc_a, dbm + k * kinc_b, idesc);
            }
          }
          umma_commit(empty0 + 8 * stage);   // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) {
          umma_commit(tfull0 + 8 * as);
          if (p.pair) umma_commit(tfull0 + 8 * (as + 1));
        }
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ splitter warps
    const int t = threadIdx.x - 64;   // 0..127
    int stage = 0; uint32_t phase = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      for (int kc = 0; kc < n_sub * p.k_chunks; ++kc) {
        if (!mbar_wait(full0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
        float4* base = reinterpret_cast<float4*>(smem + (size_t)stage * STAGE_BYTES);
#pragma unroll
        for (int op = 0; op < (p.one_pass ? 0 : SLOTS); ++op) {
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
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    int local = 0;
    uint32_t d_loads = 0;   // D slabs requested so far: parity of their barrier
    bool ok = true;
    uint8_t* buf = smem + (size_t)STAGES * STAGE_BYTES + (size_t)q * EPI_BYTES;   // two 4 KiB boxes of 32 x 32
    const uint32_t buf_u32 = smem_u32(buf);
    const uint32_t dbar = dfull0 + 8 * q;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++local) {
      int tn, tm, b, ks;
      item_decode(p, item, tn, tm, b, ks);
      const int as = (p.dual || p.pair) ? ((2 * local) & 3) : (local & 1);   // dual, pair: accumulators as and as + 1
      const uint32_t aphase = (uint32_t)(local >> 1) & 1u;
      const int64_t row_base = p.r_b * b + p.r_s * ks + (int64_t)tm * TILE + q * 32;
      const int64_t col_tile = p.c_b * b + (int64_t)tn * TILE;
      if (p.pair) {
        // both accumulators are stored: as through mapC, as + 1 through mapD (the second output)
        bool got = false;
#pragma unroll 1
        for (int part = 0; part < 4 && ok; ++part) {
          const int which = part >> 1, hf = part & 1;
          int n_box = 0;
          if (row_base < p.c_rows && tm * TILE + q * 32 < p.m_valid)
            for (int ch = 0; ch < 2; ++ch) n_box += (col_tile + 64 * hf + 32 * ch < p.c_cols) ? 1 : 0;
          if (lane == 0) tma_store_wait_read();       // the previous stores have read the staging boxes
          __syncwarp();
          if (!got) {
            if (!mbar_wait(tfull0 + 8 * as, aphase, abortp, p.status)) { ok = false; break; }
            if (!mbar_wait(tfull0 + 8 * (as + 1), aphase, abortp, p.status)) { ok = false; break; }
            tc_fence_after();
            got = true;
          }
#pragma unroll 1
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t r[32];
            tmem_ld32(tmem_base + (uint32_t)((as + which) * TILE + hf * 64 + ch * 32) + ((uint32_t)(q * 32) << 16), r);
            if (ch >= n_box) continue;                // warp-uniform
            uint8_t* rowp = buf + ch * 4096 + lane * 128;
#pragma unroll
            for (int cq = 0; cq < 8; ++cq) {
              float4* cell = reinterpret_cast<float4*>(rowp + ((cq ^ (lane & 7)) << 4));
              *cell = make_float4(p.alpha * __uint_as_float(r[4 * cq]), p.alpha * __uint_as_float(r[4 * cq + 1]),
                                  p.alpha * __uint_as_float(r[4 * cq + 2]), p.alpha * __uint_as_float(r[4 * cq + 3]));
            }
          }
          if (part == 3) tc_fence_before();           // all reads of the accumulators are done
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (part == 3) { mbar_arrive(tempty0 + 8 * as); mbar_arrive(tempty0 + 8 * (as + 1)); }
            for (int ch = 0; ch < n_box; ++ch)
              tma_store_2d(which ? &mapD : &mapC, (int)(col_tile + 64 * hf + 32 * ch), (int)row_base, buf_u32 + ch * 4096);
            tma_store_commit();
          }
        }
        continue;
      }
      if (p.dual) {
        // C = alpha * (A.B2); partial sum of <A.B1, A.B2> over this warp's 32 x 128 slab (rows or columns past the
        // end of the operands were read as zeros and add nothing)
        double dot = 0.0;
#pragma unroll 1
        for (int hf = 0; hf < 2 && ok; ++hf) {
          int n_box = 0;
          if (row_base < p.c_rows && tm * TILE + q * 32 < p.m_valid)
            for (int ch = 0; ch < 2; ++ch) n_box += (col_tile + 64 * hf + 32 * ch < p.c_cols) ? 1 : 0;
          if (lane == 0) tma_store_wait_read();       // the previous stores have read the staging boxes
          __syncwarp();
          if (hf == 0) {
            if (!mbar_wait(tfull0 + 8 * as, aphase, abortp, p.status)) { ok = false; break; }
            if (!mbar_wait(tfull0 + 8 * (as + 1), aphase, abortp, p.status)) { ok = false; break; }
            tc_fence_after();
          }
#pragma unroll 1
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t r1[32], r2[32];
            const uint32_t col = (uint32_t)(hf * 64 + ch * 32) + ((uint32_t)(q * 32) << 16);
            tmem_ld32(tmem_base + (uint32_t)(as * TILE) + col, r1);
            tmem_ld32(tmem_base + (uint32_t)((as + 1) * TILE) + col, r2);
            float part = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) part = fmaf(__uint_as_float(r1[i]), __uint_as_float(r2[i]), part);
            dot += (double)part;
            if (ch >= n_box) continue;                // warp-uniform
            uint8_t* rowp = buf + ch * 4096 + lane * 128;
#pragma unroll
            for (int cq = 0; cq < 8; ++cq) {
              float4* cell = reinterpret_cast<float4*>(rowp + ((cq ^ (lane & 7)) << 4));
              *cell = make_float4(p.alpha * __uint_as_float(r2[4 * cq]), p.alpha * __uint_as_float(r2[4 * cq + 1]),
                                  p.alpha * __uint_as_float(r2[4 * cq + 2]), p.alpha * __uint_as_float(r2[4 * cq + 3]));
            }
          }
          if (hf == 1) tc_fence_before();             // all reads of the accumulators are done
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (hf == 1) { mbar_arrive(tempty0 + 8 * as); mbar_arrive(tempty0 + 8 * (as + 1)); }
            for (int ch = 0; ch < n_box; ++ch)
              tma_store_2d(&mapC, (int)(col_tile + 64 * hf + 32 * ch), (int)row_base, buf_u32 + ch * 4096);
            tma_store_commit();
          }
        }
        // lanes in a fixed order
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        if (ok && lane == 0) p.dot_part[(size_t)item * 4 + q] = dot;
        continue;
      }
      // The warp's 32 x 128 slab goes through shared memory in two halves of 64 columns (two 32 x 32 boxes).
      bool waited = false;
      double wdot = 0.0;
#pragma unroll 1
      for (int hf = 0; hf < 2 && ok; ++hf) {
        // boxes of this half that lie inside C (warp-uniform)
        int n_box = 0;
        if (row_base < p.c_rows && tm * TILE + q * 32 < p.m_valid)
          for (int ch = 0; ch < 2; ++ch) n_box += (col_tile + 64 * hf + 32 * ch < p.c_cols) ? 1 : 0;
        if (lane == 0) {
          tma_store_wait_read();                    // the previous stores have read the staging boxes
          if (p.D && n_box > 0) {
            mbar_expect_tx(dbar, (uint32_t)n_box * 4096u);
            for (int ch = 0; ch < n_box; ++ch)
              tma_load_2d(buf_u32 + ch * 4096, &mapD, (int)(col_tile + 64 * hf + 32 * ch), (int)row_base, dbar);
          }
        }
        __syncwarp();
        if (!waited) {
          if (!mbar_wait(tfull0 + 8 * as, aphase, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          waited = true;
        }
        if (p.D && n_box > 0) {
          if (!mbar_wait(dbar, d_loads & 1u, abortp, p.status)) { ok = false; break; }
          ++d_loads;
        }
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t r[32];
          tmem_ld32(tmem_base + (uint32_t)(as * TILE + hf * 64 + ch * 32) + ((uint32_t)(q * 32) << 16), r);
          if (ch >= n_box) continue;                // warp-uniform
          // lane = row of the box; 16-byte chunk c of the row sits at chunk c ^ (row % 8)  (128-byte swizzle)
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
        if (hf == 1) tc_fence_before();             // all reads of the accumulator are done
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          if (hf == 1) mbar_arrive(tempty0 + 8 * as);   // accumulator buffer is free again
          for (int ch = 0; ch < n_box; ++ch)
            tma_store_2d(&mapC, (int)(col_tile + 64 * hf + 32 * ch), (int)row_base, buf_u32 + ch * 4096);
          tma_store_commit();
        }
        if (p.colw) {
          // the boxes still hold C: once the store has read them they become C2 = C * colw[column]
          if (lane == 0) tma_store_wait_read();
          __syncwarp();
          float part = 0.f;
          for (int ch = 0; ch < n_box; ++ch) {
            const float4* w4 = reinterpret_cast<const float4*>(p.colw + col_tile + 64 * hf + 32 * ch);
            uint8_t* rowp = buf + ch * 4096 + lane * 128;
#pragma unroll
            for (int cq = 0; cq < 8; ++cq) {
              float4* cell = reinterpret_cast<float4*>(rowp + ((cq ^ (lane & 7)) << 4));
              const float4 v = *cell, w = __ldg(w4 + cq);
              const float4 e = make_float4(v.x * w.x, v.y * w.y, v.z * w.z, v.w * w.w);
              part = fmaf(v.x, e.x, part); part = fmaf(v.y, e.y, part); part = fmaf(v.z, e.z, part); part = fmaf(v.w, e.w, part);
              *cell = e;
            }
          }
          wdot += (double)part;
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            for (int ch = 0; ch < n_box; ++ch)
              tma_store_2d(&mapB2, (int)(col_tile + 64 * hf + 32 * ch), (int)row_base, buf_u32 + ch * 4096);
            tma_store_commit();
          }
        }
      }
      if (p.colw) {
        // lanes in a fixed order
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) wdot += __shfl_xor_sync(0xffffffffu, wdot, o);
        if (ok && lane == 0) p.dot_part[(size_t)item * 4 + q] = wdot;
      }
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

struct HostOp {
  const float* base; int64_t inner, outer, ld;   // global 2-D view [outer][inner]
  OpCoord c;
};

// B2: the second N-side operand (dual) or the second M-side operand (pair 1); C2: the second output (pair)
armor_status launch(armor_ctx* c, const HostOp& A, const HostOp& B, BParams p, int kclass, double kbytes, cudaStream_t s,
                    const float* B2 = nullptr, float* C2 = nullptr) {
  CUtensorMap mA, mB, mB2, mC, mD;
  if (!make_map_2d(&mC, p.C, p.c_cols, p.c_rows, p.ldc, 32, 32)) return ARMOR_ERR_CUDA;
  if (p.pair) {
    if (!C2 || p.D) return ARMOR_ERR_INVALID_ARG;
    if (!make_map_2d(&mD, C2, p.c_cols, p.c_rows, p.ldc, 32, 32)) return ARMOR_ERR_CUDA;
  } else if (p.D) {
    if (!make_map_2d(&mD, p.D, p.c_cols, p.c_rows, p.ldd, 32, 32)) return ARMOR_ERR_CUDA;
  } else {
    mD = mC;
  }
  if (!make_map_2d(&mA, A.base, A.inner, A.outer, A.ld, 32, A.c.mn_major ? 32 : TILE, A.c.mn_major != 0)) return ARMOR_ERR_CUDA;
  if (!make_map_2d(&mB, B.base, B.inner, B.outer, B.ld, 32, B.c.mn_major ? 32 : TILE, B.c.mn_major != 0)) return ARMOR_ERR_CUDA;
  if (p.colw) {
    // the second output has the geometry of C
    if (!C2 || p.pair || p.dual) return ARMOR_ERR_INVALID_ARG;
    if (!make_map_2d(&mB2, C2, p.c_cols, p.c_rows, p.ldc, 32, 32)) return ARMOR_ERR_CUDA;
  } else if (B2 && p.pair == 1) {
    if (!make_map_2d(&mB2, B2, A.inner, A.outer, A.ld, 32, A.c.mn_major ? 32 : TILE, A.c.mn_major != 0)) return ARMOR_ERR_CUDA;
  } else if (B2) {
    if (!make_map_2d(&mB2, B2, B.inner, B.outer, B.ld, 32, B.c.mn_major ? 32 : TILE, B.c.mn_major != 0)) return ARMOR_ERR_CUDA;
  } else {
    mB2 = mB;
  }
  p.a = A.c; p.b = B.c;
  p.status = c->status;
  static PerDeviceOnce attr2, attr3;
  if (ensure_dynamic_smem(attr2, c->device, tc_block_kernel<2>, smem_bytes<2>()) != ARMOR_OK) return ARMOR_ERR_CUDA;
  if (ensure_dynamic_smem(attr3, c->device, tc_block_kernel<3>, smem_bytes<3>()) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int n_sm = c->n_sm;
  const int n_items = p.batch * p.m_tiles * p.n_tiles * p.n_split;
  const int grid = n_items < n_sm ? n_items : n_sm;
  KTimer kt(c, kclass, kbytes, s);
  if (p.pair == 1) tc_block_kernel<3><<<grid, NTHREADS, smem_bytes<3>(), s>>>(mA, mB, mB2, mC, mD, p);
  else tc_block_kernel<2><<<grid, NTHREADS, smem_bytes<2>(), s>>>(mA, mB, mB2, mC, mD, p);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

inline bool ptr_ok(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

}  // namespace

bool tc_block_ok(const armor_ctx* c, int64_t rows, int64_t cols) {
  return c->cfg.precision != ARMOR_PREC_SIMT && c->db % TILE == 0 && rows > 0 && cols % 4 == 0;
}

// out[:, j-th block] = alpha * in[:, j-th block] * Q_j (+ beta * add[:, j-th block]),  Q_j = Bblk[j] or its transpose
armor_status tc_bd_right(armor_ctx* c, const float* in, const float* Bblk, bool transB, float* out, int64_t rows,
                         int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  if (c->tc_blocks == 2 && tc_blockres_ok(c)) return tc_blockres_right(c, in, Bblk, transB, out, rows, cols, alpha, add, beta, s);
  const int db = c->db;
  const int nb = (int)(cols / db);
  if (!ptr_ok(in) || !ptr_ok(Bblk) || !ptr_ok(out)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{in, cols, rows, cols, {0, db, 0, BK, 0, TILE, 0}};
  HostOp B{Bblk, db, (int64_t)nb * db, db, {}};
  if (transB) B.c = {0, 0, 0, BK, db, TILE, 0};         // Bop[n][k] = B_j[n][k]: K-major
  else        B.c = {1, 0, TILE, 0, db, 0, BK};         // Bop[n][k] = B_j[k][n]: N-major
  BParams p{};
  p.C = out; p.D = add; p.ldc = cols; p.ldd = cols; p.c_rows = rows; p.c_cols = cols;
  p.r_b = 0; p.c_b = db;
  p.m_tiles = (int)((rows + TILE - 1) / TILE); p.n_tiles = db / TILE; p.batch = nb; p.k_chunks = db / BK;
  p.alpha = alpha; p.beta = add ? beta : 0.f;
  p.n_split = 1; p.r_s = 0; p.m_valid = 1 << 30;
  p.batch_fastest = 1;   // neighbouring CTAs read neighbouring column blocks of the same rows
  p.one_pass = c->block_one_pass;
  return launch(c, A, B, p, ARMOR_KC_BLOCK_PRODUCT, (add ? 12.0 : 8.0) * (double)rows * (double)cols, s);
}

// out[i-th block, :] = alpha * P_i * in[i-th block, :] (+ beta * add[i-th block, :]),  P_i = Ablk[i] or its transpose
armor_status tc_bd_left(armor_ctx* c, const float* Ablk, bool transA, const float* in, float* out, int64_t rows,
                        int64_t cols, float alpha, const float* add, float beta, cudaStream_t s) {
  if (c->tc_blocks == 2 && tc_blockres_ok(c)) return tc_blockres_left(c, Ablk, transA, in, out, rows, cols, alpha, add, beta, s);
  const int db = c->db;
  const int nb = (int)(rows / db);
  if (!ptr_ok(in) || !ptr_ok(Ablk) || !ptr_ok(out)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{Ablk, db, (int64_t)nb * db, db, {}};
  if (transA) A.c = {1, 0, TILE, 0, db, 0, BK};         // Aop[m][k] = A_i[k][m]: M-major
  else        A.c = {0, 0, 0, BK, db, TILE, 0};         // Aop[m][k] = A_i[m][k]: K-major
  HostOp B{in, cols, rows, cols, {1, 0, TILE, 0, db, 0, BK}};   // Bop[n][k] = in[i*db + k][n]: N-major
  BParams p{};
  p.C = out; p.D = add; p.ldc = cols; p.ldd = cols; p.c_rows = rows; p.c_cols = cols;
  p.r_b = db; p.c_b = 0;
  p.m_tiles = db / TILE; p.n_tiles = (int)((cols + TILE - 1) / TILE); p.batch = nb; p.k_chunks = db / BK;
  p.alpha = alpha; p.beta = add ? beta : 0.f;
  p.n_split = 1; p.r_s = 0; p.m_valid = 1 << 30;
  p.one_pass = c->block_one_pass;
  return launch(c, A, B, p, ARMOR_KC_BLOCK_PRODUCT, (add ? 12.0 : 8.0) * (double)rows * (double)cols, s);
}

// out[i-th block, :] = P_i * in2[i-th block, :] and 4 partial sums per 128 x 128 tile of <P_i * in1, P_i * in2> at part
// (tile order, then the four 32-row slabs of the tile); returns the number of partial sums through n_part
armor_status tc_bd_left_dual(armor_ctx* c, const float* Ablk, bool transA, const float* in1, const float* in2, float* out,
                             int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s) {
  // with d_block = 128 the kernel that keeps the wrapper block in tensor memory takes both inputs of a tile in one
  // instruction (half the shared-memory traffic of two passes through the streaming kernel)
  if (c->tc_blocks != 1 && !transA && tc_blockres_ok(c))
    return tc_blockres_left_dual(c, Ablk, in1, in2, out, rows, cols, part, n_part, s);
  const int db = c->db;
  const int nb = (int)(rows / db);
  if (!ptr_ok(in1) || !ptr_ok(in2) || !ptr_ok(Ablk) || !ptr_ok(out)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{Ablk, db, (int64_t)nb * db, db, {}};
  if (transA) A.c = {1, 0, TILE, 0, db, 0, BK};
  else        A.c = {0, 0, 0, BK, db, TILE, 0};
  HostOp B{in1, cols, rows, cols, {1, 0, TILE, 0, db, 0, BK}};
  BParams p{};
  p.C = out; p.D = nullptr; p.ldc = cols; p.ldd = cols; p.c_rows = rows; p.c_cols = cols;
  p.r_b = db; p.c_b = 0;
  p.m_tiles = db / TILE; p.n_tiles = (int)((cols + TILE - 1) / TILE); p.batch = nb; p.k_chunks = db / BK;
  p.alpha = 1.f; p.beta = 0.f;
  p.n_split = 1; p.r_s = 0; p.m_valid = 1 << 30;
  p.one_pass = c->block_one_pass;
  p.dual = 1; p.dot_part = part;
  *n_part = 4 * p.batch * p.m_tiles * p.n_tiles;
  // two W-shaped reads, one W-shaped write
  return launch(c, A, B, p, ARMOR_KC_BLOCK_PRODUCT, 12.0 * (double)rows * (double)cols, s, in2);
}

// E = add - P_i * in per block row, EH = E scaled per column by colw, and 4 partial sums per 128 x 128 tile of <E, EH> at
// part (the residual E = W - A T, E diag(h) and the proxy loss of the diagonal weighting in one pass)
armor_status tc_bd_left_residual(armor_ctx* c, const float* Ablk, const float* in, const float* add, const float* colw,
                                 float* E, float* EH, int64_t rows, int64_t cols, double* part, int* n_part, cudaStream_t s) {
  const int db = c->db;
  const int nb = (int)(rows / db);
  if (!ptr_ok(in) || !ptr_ok(Ablk) || !ptr_ok(add) || !ptr_ok(colw) || !ptr_ok(E) || !ptr_ok(EH) || cols % TILE) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{Ablk, db, (int64_t)nb * db, db, {0, 0, 0, BK, db, TILE, 0}};
  HostOp B{in, cols, rows, cols, {1, 0, TILE, 0, db, 0, BK}};
  BParams p{};
  p.C = E; p.D = add; p.ldc = cols; p.ldd = cols; p.c_rows = rows; p.c_cols = cols;
  p.r_b = db; p.c_b = 0;
  p.m_tiles = db / TILE; p.n_tiles = (int)(cols / TILE); p.batch = nb; p.k_chunks = db / BK;
  p.alpha = -1.f; p.beta = 1.f;
  p.n_split = 1; p.r_s = 0; p.m_valid = 1 << 30;
  p.one_pass = c->block_one_pass;
  p.colw = colw; p.dot_part = part;
  *n_part = 4 * p.batch * p.m_tiles * p.n_tiles;
  // two W-shaped reads (in, add), two writes
  return launch(c, A, B, p, ARMOR_KC_BLOCK_PRODUCT, 16.0 * (double)rows * (double)cols, s, nullptr, EH);
}

namespace {

// out[e] = sum over the slabs, in slab order
__global__ void __launch_bounds__(256) sum_slabs_kernel(const float4* __restrict__ part, int64_t n4, int n_slab,
                                                        float4* __restrict__ out) {
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n4; i += (int64_t)gridDim.x * 256) {
    float4 acc = part[i];
    for (int k = 1; k < n_slab; ++k) {
      const float4 v = part[(int64_t)k * n4 + i];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    out[i] = acc;
  }
}

// chunks of the contraction per work item so that about one CTA per SM has work
int pick_split(int64_t items, int64_t chunks) {
  int64_t ks = (148 + items - 1) / items;
  if (ks > chunks / 8) ks = chunks / 8;
  while (ks > 1 && chunks % ks) --ks;
  return ks < 1 ? 1 : (int)ks;
}

armor_status gram_launch(armor_ctx* c, const HostOp& A, const HostOp& B, float* G, int nb, int64_t K, cudaStream_t s) {
  const int db = c->db;
  const int64_t chunks = K / BK;
  const int tiles = (db / TILE) * (db / TILE);
  int ks = pick_split((int64_t)nb * tiles, chunks);
  const int64_t slab = (int64_t)nb * db * db;
  if (ks > 1 && (!c->gpart || ks * slab > c->gpart_floats)) ks = 1;
  BParams p{};
  p.C = ks > 1 ? c->gpart : G; p.D = nullptr; p.ldc = db; p.ldd = db;
  p.c_rows = (int64_t)ks * nb * db; p.c_cols = db;
  p.r_b = db; p.c_b = 0; p.r_s = (int64_t)nb * db;
  p.m_tiles = db / TILE; p.n_tiles = db / TILE; p.batch = nb; p.k_chunks = (int)(chunks / ks); p.n_split = ks;
  p.alpha = 1.f; p.beta = 0.f; p.m_valid = 1 << 30;
  // two W-shaped operands are read once each
  armor_status st = launch(c, A, B, p, ARMOR_KC_BLOCK_GRAM, 8.0 * (double)c->wn, s);
  if (st != ARMOR_OK || ks == 1) return st;
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  int64_t blocks = (slab / 4 + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  sum_slabs_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(c->gpart), slab / 4, ks,
                                                   reinterpret_cast<float4*>(G));
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

// Two Grams in one launch from the same stages.  pair 1: G = A.B, G2 = A2.B (A2 addressed like A); pair 2: G = A with
// itself, G2 = A.B.  Every shared chunk is read once.
armor_status gram_pair_launch(armor_ctx* c, const HostOp& A, const HostOp& B, const float* A2, int pair, float* G, float* G2,
                              int nb, int64_t K, cudaStream_t s) {
  const int db = c->db;
  const int64_t chunks = K / BK;
  const int tiles = (db / TILE) * (db / TILE);
  int ks = pick_split((int64_t)nb * tiles, chunks);
  const int64_t slab = (int64_t)nb * db * db;
  if (ks > 1 && (!c->gpart || 2 * ks * slab > c->gpart_floats)) ks = 1;
  BParams p{};
  p.C = ks > 1 ? c->gpart : G; p.D = nullptr; p.ldc = db; p.ldd = db;
  float* C2 = ks > 1 ? c->gpart + ks * slab : G2;
  p.c_rows = (int64_t)ks * nb * db; p.c_cols = db;
  p.r_b = db; p.c_b = 0; p.r_s = (int64_t)nb * db;
  p.m_tiles = db / TILE; p.n_tiles = db / TILE; p.batch = nb; p.k_chunks = (int)(chunks / ks); p.n_split = ks;
  p.alpha = 1.f; p.beta = 0.f; p.m_valid = 1 << 30;
  p.pair = pair;
  // three (pair 1) or two (pair 2) W-shaped operands are read once each
  armor_status st = launch(c, A, B, p, ARMOR_KC_BLOCK_GRAM, (pair == 1 ? 12.0 : 8.0) * (double)c->wn, s, A2, C2);
  if (st != ARMOR_OK || ks == 1) return st;
  KTimer kt(c, ARMOR_KC_SMALL, 0.0, s);
  int64_t blocks = (slab / 4 + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  sum_slabs_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(c->gpart), slab / 4, ks,
                                                   reinterpret_cast<float4*>(G));
  sum_slabs_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(c->gpart + ks * slab), slab / 4, ks,
                                                   reinterpret_cast<float4*>(G2));
  c->launches += 2;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

}  // namespace

bool tc_gram_ok(const armor_ctx* c) {
  return c->cfg.precision != ARMOR_PREC_SIMT && c->db % TILE == 0 && c->d_in % BK == 0 && c->d_out % BK == 0;
}

// G_i = P_i T_i^T over the row-blocks i (contraction over d_in)
armor_status tc_rowblock_gram(armor_ctx* c, const float* P, const float* T, float* G, cudaStream_t s) {
  const int db = c->db;
  if (!ptr_ok(P) || !ptr_ok(T) || !ptr_ok(G)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{P, c->d_in, c->d_out, c->d_in, {0, 0, 0, BK, db, TILE, 0}};   // Aop[m][k] = P[i*db + m][k]: K-major
  HostOp B{T, c->d_in, c->d_out, c->d_in, {0, 0, 0, BK, db, TILE, 0}};
  return gram_launch(c, A, B, G, c->nbo, c->d_in, s);
}

// C_j = U_j^T Y_j over the column-blocks j (contraction over d_out)
armor_status tc_colblock_gram(armor_ctx* c, const float* U, const float* Y, float* Cm, cudaStream_t s) {
  const int db = c->db;
  if (!ptr_ok(U) || !ptr_ok(Y) || !ptr_ok(Cm)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{U, c->d_in, c->d_out, c->d_in, {1, db, TILE, 0, 0, 0, BK}};   // Aop[m][k] = U[k][j*db + m]: M-major
  HostOp B{Y, c->d_in, c->d_out, c->d_in, {1, db, TILE, 0, 0, 0, BK}};
  return gram_launch(c, A, B, Cm, c->nbi, c->d_out, s);
}

// G_i = P_i T_i^T and G2_i = P2_i T_i^T in one launch (T read once)
armor_status tc_rowblock_gram_pair(armor_ctx* c, const float* P, const float* P2, const float* T, float* G, float* G2,
                                   cudaStream_t s) {
  const int db = c->db;
  if (!ptr_ok(P) || !ptr_ok(P2) || !ptr_ok(T) || !ptr_ok(G) || !ptr_ok(G2)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{P, c->d_in, c->d_out, c->d_in, {0, 0, 0, BK, db, TILE, 0}};
  HostOp B{T, c->d_in, c->d_out, c->d_in, {0, 0, 0, BK, db, TILE, 0}};
  return gram_pair_launch(c, A, B, P2, 1, G, G2, c->nbo, c->d_in, s);
}

// C_j = U_j^T U_j and C2_j = U_j^T Y_j in one launch (U and Y read once each); d_block = 128 (one tile per block: the
// chunk of U that is the M side of a tile is also its N side)
armor_status tc_colblock_gram_self_pair(armor_ctx* c, const float* U, const float* Y, float* Cm, float* Cm2, cudaStream_t s) {
  const int db = c->db;
  if (db != TILE) return ARMOR_ERR_UNSUPPORTED;
  if (!ptr_ok(U) || !ptr_ok(Y) || !ptr_ok(Cm) || !ptr_ok(Cm2)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{U, c->d_in, c->d_out, c->d_in, {1, db, TILE, 0, 0, 0, BK}};
  HostOp B{Y, c->d_in, c->d_out, c->d_in, {1, db, TILE, 0, 0, 0, BK}};
  return gram_pair_launch(c, A, B, nullptr, 2, Cm, Cm2, c->nbi, c->d_out, s);
}

// Y[j][i][:] = Z[j][i][:] * H[j-th block row, :]  for i < nbo: per column-block j a thin [nbo, d_block] x
// [d_block, d_in] product (the group-update guard).  Z and Y are stored with nbo_pad rows per j.
armor_status tc_select_rows_times_H(armor_ctx* c, const float* Z, const float* H, float* Y, int nbo_pad, cudaStream_t s) {
  const int db = c->db;
  if (!ptr_ok(Z) || !ptr_ok(H) || !ptr_ok(Y)) return ARMOR_ERR_UNSUPPORTED;
  HostOp A{Z, db, (int64_t)c->nbi * nbo_pad, db, {0, 0, 0, BK, nbo_pad, TILE, 0}};            // Aop[m][k] = Z[j][m][k]
  HostOp B{H, c->d_in, c->d_in, c->d_in, {1, 0, TILE, 0, db, 0, BK}};                         // Bop[n][k] = H[j*db + k][n]
  BParams p{};
  p.C = Y; p.D = nullptr; p.ldc = c->d_in; p.ldd = c->d_in;
  p.c_rows = (int64_t)c->nbi * nbo_pad; p.c_cols = c->d_in;
  p.r_b = nbo_pad; p.c_b = 0; p.r_s = 0;
  p.m_tiles = (c->nbo + TILE - 1) / TILE; p.n_tiles = (int)((c->d_in + TILE - 1) / TILE); p.batch = c->nbi;
  p.k_chunks = db / BK; p.n_split = 1; p.m_valid = c->nbo;
  p.alpha = 1.f; p.beta = 0.f;
  // reads H once, plus the thin operands
  return launch(c, A, B, p, ARMOR_KC_MASK_GUARD, 4.0 * (double)c->d_in * (double)c->d_in, s);
}
