// The core product of the deployment form (Section 3.1: y = A (S (B x)), S the 2:4 sparse core) on the sparse
// tensor cores of sm_100a:  Z2[t][m] = sum_k S[m][k] * Z1[t][k]  with S given as its kept values (two of every
// four along k, bf16) plus the 2-bit positions of the kept values, Z1 bf16, fp32 accumulation and output.
//
// S is the A operand of tcgen05.mma.sp (kind::f16): each instruction multiplies a 128 x 32 slice of S, held in
// shared memory as 128 x 16 kept values, by a 32 x 128 slice of Z1^T; the positions come from tensor memory.
//
// Layout of the positions (what the instruction reads, M = 128, 16-bit operands): one 32-bit tensor-memory column
// per instruction; lane l = m0 + 8 k1 + 16 m2 (m0 < 8, k1 < 2, m2 < 8) holds, in its low half, the 16 bits of row
// m0 + 16 m2 for the k-half k1 (16 consecutive k: four groups, four bits each, the lower kept position in bits
// 0-1 and the higher one in bits 2-3 of the group's nibble) and, in its high half, the same for row m0 + 16 m2 + 8.
// Consecutive instructions along k use consecutive columns; the instruction is given the even column of the pair
// and the column's parity as the selector field of its descriptor.  compress_24_kernel writes the positions in
// exactly this order, 128 lanes x 4 columns (16 bytes per lane) per 128 x 128 block of S: 2 KiB that travel with
// the stage's operands by TMA and go from shared to tensor memory with one tcgen05.cp (128 lanes x 128 bits)
// issued by the MMA thread in front of the stage's four instructions -- the copy runs in the tensor-core pipe,
// in order with the MMAs.  (Writing the positions with tcgen05.st from other warps was measured first: every
// store waited about 1600 cycles behind the running MMAs and the kernel ran at a quarter of its rate.)
//
// Kernel: persistent, one CTA per SM, 192 threads: warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 epilogue
// (transposing store: lanes are rows m of S, columns are tokens).  128 x 128 output tiles, 128 k per stage
// (16 KiB of kept values + 32 KiB of Z1 + 2 KiB of positions), four stages, two accumulator buffers.  Every wait
// is bounded.
#include <cuda_bf16.h>

#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128, BN = 128, BKL = 128;        // BKL: logical k per stage (64 kept values = 128 bytes per row)
constexpr int NTHREADS = 192;
constexpr int STAGES = 4;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t META_COL0 = 256;                 // accumulators: columns 0-127 and 128-255
constexpr int A_BYTES = BM * 64 * 2;                // 16 KiB
constexpr int BH_BYTES = BN * 64 * 2;               // 16 KiB: one half (64 k) of the Z1 stage
constexpr int E_BYTES = 128 * 16;                   // positions of one stage
constexpr int STAGE_BYTES = A_BYTES + 2 * BH_BYTES + E_BYTES; // 50 KiB

struct SParams {
  float* Z; int64_t ldz;        // [N tokens][ldz], written transposed
  __nv_bfloat16* Zb;            // non-null: the output is written as bf16 here instead
  int64_t M, N, K;              // rows of S, tokens, logical k
  int m_tiles, n_tiles, k_tiles;
  int32_t* status;
};

__device__ __forceinline__ uint64_t smem_desc_k(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;                           // 128-byte swizzle
  return d;
}

// bf16 operands, fp32 accumulation, both K-major, sparse A; sel = parity of the position column
__device__ __forceinline__ uint32_t instr_desc_sp(uint32_t sel) {
  uint32_t d = sel & 3u;          // position selector
  d |= 1u << 2;                   // A is 2:4 sparse
  d |= 1u << 4;                   // D format: F32
  d |= 1u << 7;                   // A format: BF16
  d |= 1u << 10;                  // B format: BF16
  d |= (uint32_t)(BN >> 3) << 17;
  d |= (uint32_t)(BM >> 4) << 24;
  return d;
}

__device__ __forceinline__ void umma_bf16_sp(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t tmem_e,
                                             uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(tmem_e), "r"(idesc), "r"(acc)
      : "memory");
}

// Tile order: groups of GROUP_M row tiles of S; inside a group the row tile runs fastest, then the token tile.
// The CTAs running at one time then share a few row tiles of S (read from DRAM once) and a band of token tiles
// (Z1 stays in L2), instead of sweeping all of S for every token tile.
constexpr int GROUP_M = 8;
__device__ __forceinline__ void tile_to_mn(int tile, int m_tiles, int n_tiles, int& mt, int& nt) {
  const int per_group = GROUP_M * n_tiles;
  const int g = tile / per_group, r = tile - g * per_group;
  const int gm = min(GROUP_M, m_tiles - g * GROUP_M);
  mt = g * GROUP_M + r % gm;
  nt = r / gm;
}

// 128 rows of 16 bytes, packed (8-row groups 128 bytes apart), no swizzle: the positions of one stage
__device__ __forceinline__ uint64_t smem_desc_e(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(128 >> 4) << 16;
  d |= (uint64_t)(128 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// shared -> tensor memory, 128 lanes x 128 bits (four columns), in the tensor-core pipe
__device__ __forceinline__ void tmem_cp_e(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tmem_cp_e_pair(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}

// Epilogue store of 32 tokens of one row of S per lane (the output is [token][row], so a warp's 32 rows are
// contiguous for every token).  bf16: neighbouring lanes swap one value per pair of tokens so that every lane
// stores two adjacent rows (4 bytes) of one token -- as many store instructions per element as in fp32.
__device__ __forceinline__ void store_chunk(const SParams& p, const uint32_t (&r)[32], int64_t row, int64_t tok0, int lane) {
  if (p.Zb == nullptr) {
    if (row < p.M) {
#pragma unroll
      for (int cidx = 0; cidx < 32; ++cidx)
        if (tok0 + cidx < p.N) p.Z[(tok0 + cidx) * p.ldz + row] = __uint_as_float(r[cidx]);
    }
    return;
  }
  const bool odd = lane & 1;
  const int64_t row2 = row - (odd ? 1 : 0);                  // the even row of the lane pair (p.M is even)
#pragma unroll
  for (int cidx = 0; cidx < 32; cidx += 2) {
    const uint32_t give = odd ? r[cidx] : r[cidx + 1];
    const uint32_t got = __shfl_xor_sync(0xffffffffu, give, 1);
    const float lo = __uint_as_float(odd ? got : r[cidx]), hi = __uint_as_float(odd ? r[cidx + 1] : got);
    const int64_t tok = tok0 + cidx + (odd ? 1 : 0);
    if (row2 < p.M && tok < p.N) {
      const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
      *reinterpret_cast<__nv_bfloat162*>(p.Zb + tok * p.ldz + row2) = v;
    }
  }
}

__global__ void __launch_bounds__(NTHREADS, 1)
tc_sparse_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                 const __grid_constant__ CUtensorMap mapE, const SParams p) {
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
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int s = 0; s < 2; ++s) { mbar_init(tfull0 + 8 * s, 1); mbar_init(tempty0 + 8 * s, 4); }
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
        int mt, nt;
        tile_to_mn(tile, p.m_tiles, p.n_tiles, mt, nt);
        for (int kt = 0; kt < p.k_tiles; ++kt) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, STAGE_BYTES);
          const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          tma_load_2d(dst, &mapA, kt * 64, mt * BM, fb);                      // 64 kept values = 128 logical k
          tma_load_2d(dst + A_BYTES, &mapB, kt * BKL, nt * BN, fb);
          tma_load_2d(dst + A_BYTES + BH_BYTES, &mapB, kt * BKL + 64, nt * BN, fb);
          tma_load_2d(dst + A_BYTES + 2 * BH_BYTES, &mapE, 0, (mt * p.k_tiles + kt) * 128, fb);
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
          tmem_cp_e(tmem_base + META_COL0 + (uint32_t)(4 * stage), smem_desc_e(sb + 2 * BH_BYTES));
#pragma unroll
          for (int j = 0; j < 4; ++j) {                                        // 32 logical k per instruction
            const uint64_t da = smem_desc_k(sa + j * 32);                      // 16 kept values = 32 bytes
            const uint64_t dbm = smem_desc_k(sb + (j >> 1) * BH_BYTES + (j & 1) * 64);
            const uint32_t ecol = tmem_base + META_COL0 + (uint32_t)(4 * stage + j);
            umma_bf16_sp(tacc, da, dbm, ecol & ~1u, instr_desc_sp(ecol & 1u), (uint32_t)((kt > 0) | (j != 0)));
          }
          umma_commit(empty0 + 8 * stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit(tfull0 + 8 * as);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int q = warp & 3;
    int local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x, ++local) {
      int mt, nt;
        tile_to_mn(tile, p.m_tiles, p.n_tiles, mt, nt);
      const int as = local & 1;
      const uint32_t aphase = (uint32_t)(local >> 1) & 1u;
      if (!mbar_wait(tfull0 + 8 * as, aphase, abortp, p.status)) { ok = false; break; }
      tc_fence_after();
      const int64_t row = (int64_t)mt * BM + q * 32 + lane;                    // row of S = column of Z
#pragma unroll 1
      for (int ch = 0; ch < BN / 32; ++ch) {
        uint32_t r[32];
        tmem_ld32(tmem_base + (uint32_t)(as * BN + ch * 32) + ((uint32_t)(q * 32) << 16), r);
        const int64_t tok0 = (int64_t)nt * BN + ch * 32;
        store_chunk(p, r, row, tok0, lane);
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

// ---------------------------------------------------------------------------------------------------------
// The same product on pairs of CTAs (cta_group::2): a cluster of two CTAs works on a 256 x 256 output tile.
// Each CTA holds 128 rows of S (kept values in shared memory, positions in its own tensor memory) and half of
// the tile's tokens (128 rows of Z1); one instruction issued by the even CTA multiplies 256 x 32 of S by
// 32 x 256 of Z1^T, every SM reading only half of Z1's tile from its shared memory.  Per SM and 128 k this
// loads 16 KiB + 32 KiB for 128 x 256 outputs, half of what the one-CTA kernel above loads.
//   full[s]   (even CTA): armed by the even CTA's producer for the bytes of both CTAs; both CTAs' TMA loads
//             complete on it (cta_group::2 loads may signal the pair's other CTA)
//   empty[s], tfull (both CTAs): tcgen05.commit multicast to the pair
//   tempty    (even CTA): 8 arrivals, one per epilogue warp of either CTA
// The positions of both CTAs go from their shared to their tensor memory with one tcgen05.cp of the pair.
// One accumulator buffer of 256 columns (the positions need tensor-memory columns too).
constexpr int BN2 = 256;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(cluster_bar)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_sp_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t tmem_e,
                                                  uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(tmem_e), "r"(idesc), "r"(acc)
      : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ uint32_t instr_desc_sp_pair(uint32_t sel) {
  uint32_t d = sel & 3u;
  d |= 1u << 2;
  d |= 1u << 4;
  d |= 1u << 7;
  d |= 1u << 10;
  d |= (uint32_t)(BN2 >> 3) << 17;
  d |= (uint32_t)(256 >> 4) << 24;
  return d;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(NTHREADS, 1)
tc_sparse_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                      const __grid_constant__ CUtensorMap mapE, const SParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 2];
  __shared__ uint32_t tmem_base_holder;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);
  const uint32_t tfull = smem_u32(&bars[2 * STAGES]), tempty = smem_u32(&bars[2 * STAGES + 1]);
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_pairs = p.m_tiles >> 1;                       // 256-row tiles
  const int n_tiles_total = m_pairs * p.n_tiles;            // p.n_tiles counts 256-token tiles here

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(tfull, 1);
    mbar_init(tempty, 8);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                       // both CTAs' barriers exist before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; long long issued = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles_total && ok; tile += n_pairs) {
        int mt, nt;
        tile_to_mn(tile, m_pairs, p.n_tiles, mt, nt);
        const int row0 = mt * 256 + (int)rank * 128, tok0 = nt * BN2 + (int)rank * 128;
        for (int kt = 0; kt < p.k_tiles; ++kt) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abortp, p.status)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * STAGE_BYTES);
          const uint32_t fb = map_to_cta(full0 + 8 * stage, 0);
          const uint32_t dst = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          tma_load_2d_pair(dst, &mapA, kt * 64, row0, fb);
          tma_load_2d_pair(dst + A_BYTES, &mapB, kt * BKL, tok0, fb);
          tma_load_2d_pair(dst + A_BYTES + BH_BYTES, &mapB, kt * BKL + 64, tok0, fb);
          tma_load_2d_pair(dst + A_BYTES + 2 * BH_BYTES, &mapE, 0, ((2 * mt + (int)rank) * p.k_tiles + kt) * 128, fb);
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      // tail: the MMAs that read the stages issued last have finished (their commits reach both CTAs), so
      // nothing is in flight towards this CTA's shared memory when it leaves
      for (int back = 1; back <= STAGES && back <= issued; ++back) {
        int s = stage - back; uint32_t ph = phase;
        if (s < 0) { s += STAGES; ph ^= 1; }
        const long long t0 = clock64();
        while (!mbar_try(empty0 + 8 * s, ph) && clock64() - t0 < (ok ? WAIT_CYCLES : 20000000ll)) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles_total && ok; tile += n_pairs, ++local) {
        if (!mbar_wait(tempty, ((uint32_t)local & 1u) ^ 1u, abortp, p.status)) { ok = false; break; }
        tc_fence_after();
        for (int kt = 0; kt < p.k_tiles; ++kt) {
          if (!mbar_wait(full0 + 8 * stage, phase, abortp, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * STAGE_BYTES);
          const uint32_t sb = sa + A_BYTES;
          tmem_cp_e_pair(tmem_base + META_COL0 + (uint32_t)(4 * stage), smem_desc_e(sb + 2 * BH_BYTES));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint64_t da = smem_desc_k(sa + j * 32);
            const uint64_t dbm = smem_desc_k(sb + (j >> 1) * BH_BYTES + (j & 1) * 64);
            const uint32_t ecol = tmem_base + META_COL0 + (uint32_t)(4 * stage + j);
            umma_bf16_sp_pair(tmem_base, da, dbm, ecol & ~1u, instr_desc_sp_pair(ecol & 1u), (uint32_t)((kt > 0) | (j != 0)));
          }
          umma_commit_pair(empty0 + 8 * stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit_pair(tfull);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps (both CTAs)
    const int q = warp & 3;
    const uint32_t tempty_lead = map_to_cta(tempty, 0);
    int local = 0;
    bool ok = true;
    for (int tile = pair; tile < n_tiles_total && ok; tile += n_pairs, ++local) {
      int mt, nt;
        tile_to_mn(tile, m_pairs, p.n_tiles, mt, nt);
      if (!mbar_wait(tfull, (uint32_t)local & 1u, abortp, p.status)) { ok = false; break; }
      tc_fence_after();
      const int64_t row = (int64_t)mt * 256 + rank * 128 + q * 32 + lane;
#pragma unroll 1
      for (int ch = 0; ch < BN2 / 32; ++ch) {
        uint32_t r[32];
        tmem_ld32(tmem_base + (uint32_t)(ch * 32) + ((uint32_t)(q * 32) << 16), r);
        const int64_t tok0 = (int64_t)nt * BN2 + ch * 32;
        store_chunk(p, r, row, tok0, lane);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_lead);
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                       // neither CTA leaves while its partner may still signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// One thread per 32-bit word of positions: 2 rows x 16 k.  Writes the word and the eight pairs of kept values.
// A group whose mask byte keeps fewer than two positions is padded with unkept positions (their values are
// written as zeros); more than two kept positions cannot be represented: the first two are taken and the
// status word counts the group.
__global__ void __launch_bounds__(256)
compress_24_kernel(const float* __restrict__ S, const uint8_t* __restrict__ Mk, __nv_bfloat16* __restrict__ Sc,
                   uint32_t* __restrict__ E, int64_t d_out, int64_t d_in, int32_t* status) {
  const int64_t k_tiles = d_in / 128;
  const int64_t n_words = d_out * (d_in / 32);          // (d_out / 128) * k_tiles * 128 * 4
  const int64_t w = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (w >= n_words) return;
  const int k2 = (int)(w & 3), l = (int)((w >> 2) & 127);
  const int64_t blk = w >> 9;
  const int64_t kt = blk % k_tiles, mt = blk / k_tiles;
  const int m0 = l & 7, k1 = (l >> 3) & 1, m2 = l >> 4;
  const int64_t kbase = kt * 128 + k2 * 32 + k1 * 16;
  uint32_t word = 0;
  int bad = 0;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int64_t row = mt * 128 + m0 + 16 * m2 + 8 * h;
#pragma unroll
    for (int qd = 0; qd < 4; ++qd) {
      const int64_t g = kbase / 4 + qd;
      const unsigned m = Mk[row * (d_in / 4) + g] & 15u;
      const float4 v = *reinterpret_cast<const float4*>(S + row * d_in + 4 * g);
      const float vals[4] = {v.x, v.y, v.z, v.w};
      int i0 = -1, i1 = -1, cnt = 0;
#pragma unroll
      for (int pidx = 0; pidx < 4; ++pidx)
        if ((m >> pidx) & 1u) { if (cnt == 0) i0 = pidx; else if (cnt == 1) i1 = pidx; ++cnt; }
      if (cnt > 2) bad = 1;
      if (cnt < 2) {                                   // pad with unkept positions, keeping i0 < i1
        if (cnt == 0) { i0 = 0; i1 = 1; }
        else if (i0 < 3) i1 = i0 + 1;
        else { i1 = 3; i0 = 2; }
      }
      const float a = ((m >> i0) & 1u) ? vals[i0] : 0.f, b = ((m >> i1) & 1u) ? vals[i1] : 0.f;
      __nv_bfloat162 pr;
      pr.x = __float2bfloat16(a);
      pr.y = __float2bfloat16(b);
      *reinterpret_cast<__nv_bfloat162*>(Sc + row * (d_in / 2) + 2 * g) = pr;
      word |= (uint32_t)(i0 | (i1 << 2)) << (16 * h + 4 * qd);
    }
  }
  E[w] = word;
  if (bad) atomicAdd(&status[ST_SPARSE_BAD_GROUPS], 1);
}

bool make_map_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int64_t ld) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64, 128};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// positions: [rows of 16 bytes], box = 128 rows, no swizzle
bool make_map_e(CUtensorMap* map, const void* base, int64_t rows) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {4, (cuuint64_t)rows};
  cuuint64_t strides[1] = {16};
  cuuint32_t box[2] = {4, 128};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

int g_sparse_pairs = 1;   // 0: the one-CTA kernel only (tests compare the two)

bool tc_sparse_ok(const armor_ctx* c) {
  return c->cfg.n_keep == 2 && c->cfg.m_group == 4 && c->d_out % 128 == 0 && c->d_in % 128 == 0 &&
         c->cfg.precision != ARMOR_PREC_SIMT;
}

size_t tc_sparse_values_bytes(const armor_ctx* c) { return (size_t)c->d_out * (size_t)c->d_in; }   // bf16, half the entries

void launch_compress_24(armor_ctx* c, const float* S, const uint8_t* M, void* Sc, void* E, cudaStream_t s) {
  const int64_t n_words = c->d_out * (c->d_in / 32);
  KTimer kt(c, ARMOR_KC_FORWARD, (double)c->wn * 5.125, s);
  compress_24_kernel<<<(unsigned)((n_words + 255) / 256), 256, 0, s>>>(S, M, static_cast<__nv_bfloat16*>(Sc),
                                                                        static_cast<uint32_t*>(E), c->d_out, c->d_in,
                                                                        c->status);
  c->launches++;
}

// Z2[n][d_out] = Z1[n][d_in] * S^T with S given compressed (Sc, E); Z1 bf16; Z2 fp32, or bf16 if out_bf16.
armor_status launch_tc_sparse(armor_ctx* c, const void* Sc, const void* E, const void* z1_bf16, void* z2, bool out_bf16,
                              int64_t n, cudaStream_t s) {
  if (!tc_sparse_ok(c) || n <= 0) return ARMOR_ERR_UNSUPPORTED;
  CUtensorMap mA, mB, mE;
  if (!make_map_bf16(&mA, Sc, c->d_out, c->d_in / 2, c->d_in / 2)) return ARMOR_ERR_CUDA;
  if (!make_map_bf16(&mB, z1_bf16, n, c->d_in, c->d_in)) return ARMOR_ERR_CUDA;
  if (!make_map_e(&mE, E, (c->d_out / 128) * (c->d_in / 128) * 128)) return ARMOR_ERR_CUDA;
  SParams p{};
  p.Z = out_bf16 ? nullptr : static_cast<float*>(z2); p.Zb = out_bf16 ? static_cast<__nv_bfloat16*>(z2) : nullptr;
  p.ldz = c->d_out; p.M = c->d_out; p.N = n; p.K = c->d_in;
  p.m_tiles = (int)(c->d_out / BM); p.n_tiles = (int)((n + BN - 1) / BN); p.k_tiles = (int)(c->d_in / BKL);
  p.status = c->status;
  constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024;
  static PerDeviceOnce attr;
  if (ensure_dynamic_smem(attr, c->device, tc_sparse_kernel, SMEM) != ARMOR_OK) return ARMOR_ERR_CUDA;
  const int n_sm = c->n_sm;
  KTimer kt(c, ARMOR_KC_GEMM, 2.0 * (double)p.M * (double)p.N * (double)p.K, s);   // dense-equivalent flops
  if (g_sparse_pairs && c->d_out % 256 == 0 && n_sm >= 2) {
      static PerDeviceOnce attr2;
    if (ensure_dynamic_smem(attr2, c->device, tc_sparse_pair_kernel, SMEM) != ARMOR_OK) return ARMOR_ERR_CUDA;
    p.n_tiles = (int)((n + BN2 - 1) / BN2);
    const int tiles = (p.m_tiles / 2) * p.n_tiles;
    int pairs = n_sm / 2;
    if (tiles < pairs) pairs = tiles;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(NTHREADS); cfg.dynamicSmemBytes = SMEM; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, tc_sparse_pair_kernel, mA, mB, mE, p) != cudaSuccess) return ARMOR_ERR_CUDA;
  } else {
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < n_sm ? tiles : n_sm;
    tc_sparse_kernel<<<grid, NTHREADS, SMEM, s>>>(mA, mB, mE, p);
  }
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? ARMOR_OK : ARMOR_ERR_CUDA;
}
