// Tensor-core GEMM for sm_100a:  C[M][N] (+)= sum_k A[m][k] * B[n][k]   (fp32 storage, both operands K-major)
//
// Used for the dense contractions of the ARMOR iteration: the calibration Gram X^T X (Section 2 of the
// paper; both operands are the transposed, staged chunk of X) and the right-multiplications by the
// symmetric Gram, E.H, T.H and V.H (H[n][k] = H[k][n], so H itself is the K-major B operand).
//
// Design: persistent kernel, one CTA per SM, 192 threads:
//   warp 0   : TMA producer  (cp.async.bulk.tensor.2d, 128-byte swizzle, mbarrier complete_tx)
//   warp 1   : MMA issuer    (one thread issues tcgen05.mma kind::tf32, 128 x 256 x 8 per instruction,
//                             accumulators in tensor memory, two accumulator buffers of 256 columns)
//   warps 2-9: epilogue      (tcgen05.ld 32 lanes x 32 columns; the K segments of a tile are summed in registers,
//                             then one fused C-update / dot products; a symmetric product writes its lower
//                             triangle only, the caller mirrors it once at the end)
// passes == 3: every operand is given as a tf32-exact high part and an fp32 low part; the three products
// hi*hi, lo*hi, hi*lo are accumulated into the same fp32 accumulator (error-compensated tf32, fp32-grade).
// passes == 6: the same three products on fp16 high and low parts (kind::f16, twice the tf32 issue rate, half
// the operand bytes).  Two fp16 parts carry 22 significant bits like two tf32 parts, but only 5 exponent bits,
// so the caller scales rows of the operands by powers of two into the fp16 range beforehand and the epilogue
// multiplies the accumulator by the inverse scales (a per-row and a per-column vector): every scaling is
// exact, the result is fp32-grade.
// Every wait is bounded: a wait that runs out raises a status word and the CTA leaves through the common
// exit that frees its tensor memory.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 32;          // BK fp32 = 128 bytes = one swizzle row
constexpr int NTHREADS = 320;                       // TMA warp, MMA warp, eight epilogue warps
constexpr int RB = 8;                               // rows of C an epilogue lane keeps in flight
constexpr int EPI_COLS = 128;                       // accumulator columns per epilogue warp
constexpr int TB_LD = 17;                           // padded row length of an epilogue warp's 32 x 16 staging tile
constexpr uint32_t TMEM_COLS = 512;                 // two accumulator buffers of BN columns
constexpr int A_BYTES = BM * BK * 4;                // 16 KiB
constexpr int B_BYTES = BN * BK * 4;                // 32 KiB

struct Params {
  float* C; int64_t ldc;
  int64_t M, N, K;
  int m_tiles, n_tiles, n_tiles_total;
  int accumulate, symmetric_lower;
  int kt_seg;            // k-tiles accumulated in tensor memory before the epilogue folds them into C
  const float* d1; const float* d2;
  double* part1; double* part2;
  const float* row_scale; const float* col_scale;   // optional powers of two the accumulator is multiplied by
  int f16;               // 16-bit operands are fp16 (1) or bf16 (0)
  int32_t* status;
  // Tail split: tiles [split_first, n_tiles_total) are cut into split_parts pieces along K, each piece a work
  // item of its own that writes a 128 x 256 slab of partial sums; a second kernel adds the slabs.  This fills
  // the last, partly empty wave of tiles.
  int split_first, split_parts, n_items;
  float* slabs;
};

// K-major operand tile, rows of 128 bytes, 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                           // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset
  d |= (uint64_t)1 << 46;                           // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                           // 128-byte swizzle
  return d;
}

// tcgen05.mma with the accumulate flag set (the constant predicate costs no instruction)
template <bool F16>
__device__ __forceinline__ void umma_acc(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  if (F16)
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
  else
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
}

// fp32 accumulate, both operands K-major, M = 128, N = 256; operand format 0: fp16, 1: bf16 (both kind::f16),
// 2: tf32 (kind::tf32).
__device__ __forceinline__ uint32_t instr_desc(uint32_t fmt) {
  uint32_t d = 0;
  d |= 1u << 4;                   // D format: F32
  d |= fmt << 7;                  // A format
  d |= fmt << 10;                 // B format
  d |= (uint32_t)(BN >> 3) << 17; // N
  d |= (uint32_t)(BM >> 4) << 24; // M
  return d;
}

// tile index -> (m tile, n tile).  Groups of GROUP_M m tiles; inside a group m runs fastest, then n: the 148 tiles
// in flight are about 16 x 9, which minimises what a wave reads (16 A panels + 9 B panels, a B panel being twice
// an A panel) -- with m running over all m tiles every wave read up to 148 A panels, and on the large shapes
// (operands far beyond L2) the product became DRAM-bound.
constexpr int GROUP_M = 16;
__device__ __forceinline__ void tile_coords(const Params& p, int tile, int& mt, int& nt) {
  if (!p.symmetric_lower) {
    const int per_group = GROUP_M * p.n_tiles;
    const int g = tile / per_group, r = tile - g * per_group;
    const int gm = min(GROUP_M, p.m_tiles - g * GROUP_M);
    mt = g * GROUP_M + r % gm;
    nt = r / gm;
    return;
  }
  // only tiles that hold an element with column <= row: m tile >= 2 * n tile.  Same grouping: bands of GROUP_M
  // m tiles, inside a band the n tile is the outer index and m runs fastest
  int rem = tile;
  for (int m0 = 0; m0 < p.m_tiles; m0 += GROUP_M) {
    const int m1 = min(m0 + GROUP_M, p.m_tiles);
    for (nt = 0; 2 * nt < m1 && nt < p.n_tiles; ++nt) {
      const int lo = max(m0, 2 * nt);
      const int cnt = m1 - lo;
      if (rem < cnt) { mt = lo + rem; return; }
      rem -= cnt;
    }
  }
  mt = 0; nt = 0;   // not reached: tile < number of tiles
}

// work item -> tile, and its range of k-tiles
__device__ __forceinline__ void item_decode(const Params& p, int item, int kt_total, int& tile, int& part, int& kt_begin,
                                            int& kt_end) {
  if (item < p.split_first) {
    tile = item; part = -1; kt_begin = 0; kt_end = kt_total;
  } else {
    const int idx = item - p.split_first;
    tile = p.split_first + idx / p.split_parts;
    part = idx % p.split_parts;
    const int per = kt_total / p.split_parts;
    kt_begin = part * per; kt_end = kt_begin + per;
  }
}

// One epilogue warp's 32 rows x 128 columns of finished sums (lane = row) go out through shared memory, 16
// columns at a time, so that every store instruction writes two rows of 64 contiguous bytes.  Optional:
// power-of-two scales, C += (read-modify-write), lower triangle only, partial dot products with d1 / d2.
__device__ __forceinline__ void write_out(const float (&acc)[EPI_COLS], float* tilebuf, int lane, float* C, int64_t ldc,
                                          int64_t row_base, int64_t col_base, int64_t M, int64_t N, bool accum, bool sym,
                                          const float* rs, const float* cs, const float* d1, const float* d2, int64_t ldd,
                                          double& dot1, double& dot2) {
  if (row_base >= M) return;                                  // warp-uniform
  const int rr = lane >> 4, cc = lane & 15;
#pragma unroll
  for (int c16 = 0; c16 < EPI_COLS / 16; ++c16) {
    const int64_t col0 = col_base + c16 * 16;
    if (col0 >= N) continue;                                   // warp-uniform (N is a multiple of 32)
    if (sym && col0 > row_base + 31) continue;                 // chunk lies above the diagonal
#pragma unroll
    for (int i = 0; i < 16; ++i) tilebuf[lane * TB_LD + i] = acc[c16 * 16 + i];
    __syncwarp();
    const int64_t col = col0 + cc;
    const float cscale = cs ? cs[col] : 1.f;
    float f1 = 0.f, f2 = 0.f;
#pragma unroll 1
    for (int r0 = 0; r0 < 32; r0 += 2 * RB) {
      float x[RB], o[RB];
      bool keep[RB];
#pragma unroll
      for (int j = 0; j < RB; ++j) {
        const int r = r0 + 2 * j + rr;
        const int64_t grow = row_base + r;
        keep[j] = grow < M && (!sym || col <= grow);
        x[j] = tilebuf[r * TB_LD + cc];
        if (rs) x[j] *= (grow < M ? rs[grow] : 1.f) * cscale;
        o[j] = (accum && keep[j]) ? C[grow * ldc + col] : 0.f;
      }
      if (d1) {
#pragma unroll
        for (int j = 0; j < RB; ++j)
          if (keep[j]) f1 = fmaf(x[j] + o[j], d1[(row_base + r0 + 2 * j + rr) * ldd + col], f1);
      }
      if (d2) {
#pragma unroll
        for (int j = 0; j < RB; ++j)
          if (keep[j]) f2 = fmaf(x[j] + o[j], d2[(row_base + r0 + 2 * j + rr) * ldd + col], f2);
      }
#pragma unroll
      for (int j = 0; j < RB; ++j)
        if (keep[j]) C[(row_base + r0 + 2 * j + rr) * ldc + col] = x[j] + o[j];
    }
    dot1 += (double)f1;
    dot2 += (double)f2;
    __syncwarp();
  }
}

template <int PASSES>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapAlo,
               const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapBlo, const Params p) {
  constexpr bool SPLIT = (PASSES == 3 || PASSES == 6);   // operands come as high and low parts
  constexpr bool H16 = (PASSES == 0 || PASSES == 6);     // 16-bit operands (kind::f16)
  constexpr int STAGE_BYTES = (SPLIT ? 2 : 1) * (A_BYTES + B_BYTES);
  constexpr int STAGES = SPLIT ? 2 : 4;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment for the swizzled tiles
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 4];
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[2 * STAGES]), tempty0 = smem_u32(&bars[2 * STAGES + 2]);
  constexpr int BKE = H16 ? 64 : 32;                // elements of K per 128-byte row: 16-bit or fp32
  const int kt_total = (int)((p.K + BKE - 1) / BKE);

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
      for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
        int tile, part, kt_begin, kt_end, mt, nt;
        item_decode(p, item, kt_total, tile, part, kt_begin, kt_end);
        tile_coords(p, tile, mt, nt);
        for (int kt = kt_begin; kt < kt_end; ++kt) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, STAGE_BYTES);
          uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          tma_load_2d(dst, &mapA, kt * BKE, mt * BM, fb);
          dst += A_BYTES;
          if (SPLIT) { tma_load_2d(dst, &mapAlo, kt * BKE, mt * BM, fb); dst += A_BYTES; }
          tma_load_2d(dst, &mapB, kt * BKE, nt * BN, fb);
          dst += B_BYTES;
          if (SPLIT) tma_load_2d(dst, &mapBlo, kt * BKE, nt * BN, fb);
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
      const uint32_t idesc = instr_desc(H16 ? (p.f16 ? 0u : 1u) : 2u);
      const uint64_t d0 = smem_desc_k_sw128(smem_u32(smem));
      int stage = 0; uint32_t phase = 0;
      int local = 0;   // (tile, K segment) items handled so far: selects the accumulator buffer
      bool ok = true;
      for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
        int tile, part, kt_begin, kt_end;
        item_decode(p, item, kt_total, tile, part, kt_begin, kt_end);
        for (int kt0 = kt_begin; kt0 < kt_end && ok; kt0 += p.kt_seg, ++local) {
          const int as = local & 1;
          const uint32_t aphase = (uint32_t)(local >> 1) & 1u;
          if (!mbar_wait(tempty0 + 8 * as, aphase ^ 1, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t tacc = tmem_base + (uint32_t)(as * BN);
          const int kt1 = min(kt_end, kt0 + p.kt_seg);
          for (int kt = kt0; kt < kt1; ++kt) {
            if (!mbar_wait(full0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
            tc_fence_after();
            // One thread issues every MMA: the descriptors of stage 0 are formed once and only their address field
            // moves, and every MMA but a tile's first carries a constant accumulate flag, so that the instructions
            // around a tcgen05.mma stay well below the time it takes to execute.
            const uint64_t da = d0 + (uint64_t)(uint32_t)(stage * (STAGE_BYTES >> 4));
            const uint64_t dal = da + (A_BYTES >> 4);
            const uint64_t dbm = da + (((SPLIT ? 2 : 1) * A_BYTES) >> 4);
            const uint64_t dbl = dbm + (B_BYTES >> 4);
            const uint32_t acc = (uint32_t)(kt > kt0);
            if (PASSES == 3) {
              umma_tf32(tacc, dal, dbm, idesc, acc);
              umma_acc<false>(tacc, da, dbl, idesc);
              umma_acc<false>(tacc, da, dbm, idesc);
            } else if (PASSES == 6) {
              umma_bf16(tacc, dal, dbm, idesc, acc);
              umma_acc<true>(tacc, da, dbl, idesc);
              umma_acc<true>(tacc, da, dbm, idesc);
            } else if (PASSES == 0) {
              umma_bf16(tacc, da, dbm, idesc, acc);
            } else {
              umma_tf32(tacc, da, dbm, idesc, acc);
            }
#pragma unroll
            for (int k = 1; k < BK / 8; ++k) {
              const uint64_t ko = (uint64_t)(k * (32 >> 4));   // 8 fp32 (16 halves) of K: 32 bytes along the row
              if (SPLIT) {
                umma_acc<H16>(tacc, dal + ko, dbm + ko, idesc);
                umma_acc<H16>(tacc, da + ko, dbl + ko, idesc);
              }
              umma_acc<H16>(tacc, da + ko, dbm + ko, idesc);
            }
            umma_commit(empty0 + 8 * stage);   // frees the stage once these MMAs have read it
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (ok) umma_commit(tfull0 + 8 * as);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    // Eight warps: warp w reads TMEM lanes 32 (w % 4) .. and one half (128 columns) of the accumulator, one
    // row per lane.  The K segments of a tile are summed in registers (ordinary round-to-nearest adds), so the
    // accumulator buffer is handed back right after it has been read and C is touched once per tile.
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    float* tilebuf = reinterpret_cast<float*>(smem + (size_t)STAGES * STAGE_BYTES) + (warp - 2) * (32 * TB_LD);
    int local = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int tile, part, kt_begin, kt_end, mt, nt;
      item_decode(p, item, kt_total, tile, part, kt_begin, kt_end);
      tile_coords(p, tile, mt, nt);
      float acc[EPI_COLS];
#pragma unroll
      for (int i = 0; i < EPI_COLS; ++i) acc[i] = 0.f;
      for (int kt0 = kt_begin; kt0 < kt_end && ok; kt0 += p.kt_seg, ++local) {
        const int as = local & 1;
        const uint32_t aphase = (uint32_t)(local >> 1) & 1u;
        if (!mbar_wait(tfull0 + 8 * as, aphase, abortp, p.status)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < EPI_COLS / 32; ++ch) {
          uint32_t r[32];
          tmem_ld32(tmem_base + (uint32_t)(as * BN + half * EPI_COLS + ch * 32) + ((uint32_t)(q * 32) << 16), r);
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[ch * 32 + i] += __uint_as_float(r[i]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty0 + 8 * as);
      }
      if (!ok) break;
      if (part >= 0) {
        // a piece of a split tile: its partial sums go, plainly, to this item's slab
        float* slab = p.slabs + ((int64_t)(tile - p.split_first) * p.split_parts + part) * (BM * BN);
        double u1 = 0.0, u2 = 0.0;
        write_out(acc, tilebuf, lane, slab, BN, q * 32, half * EPI_COLS, BM, BN, false, false, nullptr, nullptr, nullptr,
                  nullptr, 0, u1, u2);
        continue;
      }
      double dot1 = 0.0, dot2 = 0.0;
      write_out(acc, tilebuf, lane, p.C, p.ldc, (int64_t)mt * BM + q * 32, (int64_t)nt * BN + half * EPI_COLS, p.M, p.N,
                p.accumulate != 0, p.symmetric_lower != 0, p.row_scale, p.col_scale, p.d1, p.d2, p.ldc, dot1, dot2);
      if (p.part1 || p.part2) {
        for (int o = 16; o > 0; o >>= 1) {
          dot1 += __shfl_down_sync(0xffffffffu, dot1, o);
          dot2 += __shfl_down_sync(0xffffffffu, dot2, o);
        }
        if (lane == 0) {
          if (p.part1) p.part1[(int64_t)tile * 8 + half * 4 + q] = dot1;
          if (p.part2) p.part2[(int64_t)tile * 8 + half * 4 + q] = dot2;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Adds the slabs of every split tile into C (+ what C held, if the product accumulates) and forms the tile's
// share of the fused dot products.  Four CTAs per split tile (32 rows each); fixed order.
__global__ void __launch_bounds__(256) tc_gemm_fixup_kernel(const Params p) {
  const int tile = p.split_first + blockIdx.x / 4, qq = blockIdx.x % 4;
  int mt, nt;
  tile_coords(p, tile, mt, nt);
  const float* slab0 = p.slabs + (int64_t)(blockIdx.x / 4) * p.split_parts * (BM * BN);
  double d1 = 0.0, d2 = 0.0;
  for (int e = threadIdx.x; e < 32 * BN / 4; e += 256) {
    const int r = qq * 32 + e / (BN / 4), c4 = (e % (BN / 4)) * 4;
    const int64_t grow = (int64_t)mt * BM + r, gcol = (int64_t)nt * BN + c4;
    if (grow >= p.M || gcol >= p.N) continue;
    float4 v = *reinterpret_cast<const float4*>(slab0 + (int64_t)r * BN + c4);
    for (int k = 1; k < p.split_parts; ++k) {
      const float4 w = *reinterpret_cast<const float4*>(slab0 + (int64_t)k * (BM * BN) + (int64_t)r * BN + c4);
      v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
    }
    if (p.row_scale) {
      const float rs = p.row_scale[grow];
      const float4 cs = *reinterpret_cast<const float4*>(p.col_scale + gcol);
      v.x *= rs * cs.x; v.y *= rs * cs.y; v.z *= rs * cs.z; v.w *= rs * cs.w;
    }
    float* cp = p.C + grow * p.ldc + gcol;
    if (p.accumulate) {
      const float4 o = *reinterpret_cast<const float4*>(cp);
      v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
    }
    *reinterpret_cast<float4*>(cp) = v;
    if (p.d1) {
      const float4 w = *reinterpret_cast<const float4*>(p.d1 + grow * p.ldc + gcol);
      d1 += (double)(v.x * w.x + v.y * w.y) + (double)(v.z * w.z + v.w * w.w);
    }
    if (p.d2) {
      const float4 w = *reinterpret_cast<const float4*>(p.d2 + grow * p.ldc + gcol);
      d2 += (double)(v.x * w.x + v.y * w.y) + (double)(v.z * w.z + v.w * w.w);
    }
  }
  __shared__ double red1[8], red2[8];
  for (int o = 16; o > 0; o >>= 1) {
    d1 += __shfl_down_sync(0xffffffffu, d1, o);
    d2 += __shfl_down_sync(0xffffffffu, d2, o);
  }
  if ((threadIdx.x & 31) == 0) { red1[threadIdx.x >> 5] = d1; red2[threadIdx.x >> 5] = d2; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t1 = 0.0, t2 = 0.0;
    for (int w = 0; w < 8; ++w) { t1 += red1[w]; t2 += red2[w]; }
    // eight slots per tile (the GEMM's eight epilogue warps); this kernel fills four and clears the rest
    if (p.part1) { p.part1[(int64_t)tile * 8 + qq] = t1; p.part1[(int64_t)tile * 8 + 4 + qq] = 0.0; }
    if (p.part2) { p.part2[(int64_t)tile * 8 + qq] = t2; p.part2[(int64_t)tile * 8 + 4 + qq] = 0.0; }
  }
}

// ------------------------------------------------------------------ host side
// [rows][K] fp32, leading dimension ld: box = BK x box_rows, 128-byte swizzle, zero fill out of bounds.
// bits16: 0 fp32 elements, 1 bf16, 2 fp16
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int64_t ld, int box_rows, int bits16 = 0) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * (bits16 ? 2 : 4)};
  cuuint32_t box[2] = {(cuuint32_t)(bits16 ? 64 : BK), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType dt = bits16 == 0 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : bits16 == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
  CUresult r = enc(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int PASSES>
armor_status launch_impl(armor_ctx* c, const TcGemm& g, Params p, cudaStream_t s) {
  CUtensorMap mA, mAlo, mB, mBlo;
  constexpr bool SPLIT = (PASSES == 3 || PASSES == 6);
  constexpr bool H16 = (PASSES == 0 || PASSES == 6);
  const int bits16 = H16 ? (g.fp16 ? 2 : 1) : 0;
  if (!make_map(&mA, g.A, g.M, g.K, g.lda, BM, bits16)) return ARMOR_ERR_CUDA;
  if (!make_map(&mB, g.B, g.N, g.K, g.ldb, BN, bits16)) return ARMOR_ERR_CUDA;
  if (SPLIT) {
    if (!make_map(&mAlo, g.Alo, g.M, g.K, g.lda, BM, bits16)) return ARMOR_ERR_CUDA;
    if (!make_map(&mBlo, g.Blo, g.N, g.K, g.ldb, BN, bits16)) return ARMOR_ERR_CUDA;
  } else {
    mAlo = mA;
    mBlo = mB;
  }
  constexpr int STAGE_BYTES = (SPLIT ? 2 : 1) * (A_BYTES + B_BYTES);
  constexpr int STAGES = SPLIT ? 2 : 4;
  constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024 + 8 * 32 * TB_LD * sizeof(float);
  static PerDeviceOnce attr;
  if (ensure_dynamic_smem(attr, c->device, tc_gemm_kernel<PASSES>, SMEM) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int n_sm = c->n_sm;
  // tail split: the tiles of the last, partly filled wave are cut along K so that their pieces fill the wave
  p.split_first = p.n_tiles_total; p.split_parts = 1; p.n_items = p.n_tiles_total; p.slabs = c->gemm_slabs;
  const int kt_total = (int)((p.K + (H16 ? 64 : BK) - 1) / (H16 ? 64 : BK));
  const int rem = p.n_tiles_total % n_sm;
  if (c->gemm_slabs && !p.symmetric_lower && rem > 0 && p.ldc % 4 == 0 && p.N % 4 == 0) {
    int parts = n_sm / rem;
    if (parts > 4) parts = 4;
    // a piece must be whole K segments (or lie inside one) so that issuer and epilogue agree on the segments
    while (parts > 1 && (kt_total % parts || kt_total / parts < 8 ||
                         ((kt_total / parts) % p.kt_seg && p.kt_seg < kt_total / parts)))
      --parts;
    if (parts > 1 && (int64_t)rem * parts <= c->gemm_slab_count) {
      p.split_first = p.n_tiles_total - rem;
      p.split_parts = parts;
      p.n_items = p.split_first + rem * parts;
    }
  }
  const int grid = p.n_items < n_sm ? p.n_items : n_sm;
  {
    KTimer kt(c, ARMOR_KC_GEMM, p.symmetric_lower ? (double)p.M * (double)(p.N + BM) * (double)p.K
                                                  : 2.0 * (double)p.M * (double)p.N * (double)p.K, s);
    tc_gemm_kernel<PASSES><<<grid, NTHREADS, SMEM, s>>>(mA, mAlo, mB, mBlo, p);
    if (p.split_parts > 1) {
      tc_gemm_fixup_kernel<<<4 * (p.n_tiles_total - p.split_first), 256, 0, s>>>(p);
      c->launches++;
    }
  }
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}

}  // namespace

bool tc_gemm_shape_ok(int64_t M, int64_t N, int64_t K) {
  return M > 0 && N > 0 && K > 0 && (N % 32 == 0) && (K % 4 == 0);
}

armor_status launch_tc_gemm(armor_ctx* c, const TcGemm& g, int* n_tiles, cudaStream_t s) {
  if (!tc_gemm_shape_ok(g.M, g.N, g.K)) return ARMOR_ERR_UNSUPPORTED;
  const bool h16 = (g.passes == 0 || g.passes == 6);
  if ((g.lda % (h16 ? 8 : 4)) || (g.ldb % (h16 ? 8 : 4)) || (g.ldc % 4)) return ARMOR_ERR_UNSUPPORTED;
  if ((g.row_scale == nullptr) != (g.col_scale == nullptr)) return ARMOR_ERR_INVALID_ARG;
  if (g.symmetric_lower && g.M != g.N) return ARMOR_ERR_INVALID_ARG;
  Params p{};
  p.C = g.C; p.ldc = g.ldc; p.M = g.M; p.N = g.N; p.K = g.K;
  p.m_tiles = (int)((g.M + BM - 1) / BM);
  p.n_tiles = (int)((g.N + BN - 1) / BN);
  if (g.symmetric_lower) {
    int tot = 0;
    for (int nt = 0; nt < p.n_tiles; ++nt) {
      const int cnt = p.m_tiles - 2 * nt;
      if (cnt > 0) tot += cnt;
    }
    p.n_tiles_total = tot;
  } else {
    p.n_tiles_total = p.m_tiles * p.n_tiles;
  }
  p.accumulate = g.accumulate; p.symmetric_lower = g.symmetric_lower;
  p.d1 = g.d1; p.d2 = g.d2; p.part1 = g.part1; p.part2 = g.part2;
  p.row_scale = g.row_scale; p.col_scale = g.col_scale; p.f16 = g.fp16;
  p.status = c->status;
  const int bke = h16 ? 64 : BK;
  p.kt_seg = g.k_segment > 0 ? (int)((g.k_segment + bke - 1) / bke) : (int)((g.K + bke - 1) / bke);
  if (p.kt_seg < 1) p.kt_seg = 1;
  if (n_tiles) *n_tiles = p.n_tiles_total;
  if (g.passes == 3) return launch_impl<3>(c, g, p, s);
  if (g.passes == 6) return launch_impl<6>(c, g, p, s);
  if (g.passes == 0) return launch_impl<0>(c, g, p, s);
  return launch_impl<1>(c, g, p, s);
}
