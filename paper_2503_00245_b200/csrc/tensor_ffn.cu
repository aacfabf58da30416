// Tensor-core (prefill) path of the expert FFN: grouped GEMMs on the 5th-generation tensor cores.
//
// Tokens are grouped by expert (moe_permute), their rows gathered into a bf16 operand, and every expert's
// FFN becomes dense contractions  C[m, n] = sum_k A[m, k] * B_e[n, k]  over that expert's rows:
//
//   dense experts  (1) H = silu(X Wg) * (X Wu)   A = gathered x,  B = gate / up rows of gud   -> bf16 hidden
//                  (2) O = H Wd                  A = H,           B = down rows of gud (N-major) -> fp32 slots
//   Eq. 1 factors  (1) T = X [gL | uL]   (2) H = silu(Tg gR) * (Tu uR)   (3) V = H dL   (4) O = V dR
//
// Two CTAs on neighbouring SMs (a cluster of 2) compute one tile of 256 rows x up to 256 columns with
// tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of A and HALF of the tile's B rows, the tensor
// cores of the pair exchange the B halves, and each CTA ends up with the accumulators of its 128 rows
// (128 TMEM lanes x N columns).  Per flop a CTA moves half the B bytes into shared memory and reads a third
// fewer operand bytes out of it than a single CTA computing 256 x 256 on its own, and the tile takes 256 of the
// 512 TMEM columns, so the accumulators are double-buffered: the epilogue of tile i runs under the MMAs of
// tile i + 1.  Roles in each CTA:
//   warp 0     TMA producer: 64-wide K slices of A and B into a ring of shared-memory stages (128-byte swizzle);
//              both CTAs' copies complete on the LEADER's (rank 0) stage barrier;
//   warp 1     allocates tensor memory (both CTAs); in the leader one thread issues the MMAs for the pair
//              (M = 256, N <= 256, K = 16 per instruction) and commits to both CTAs' barriers;
//   warps 2-9  epilogue: tcgen05.ld the accumulators (one TMEM lane = one output row per thread), apply
//              SiLU * mul or nothing, convert, store the rows that belong to the expert.
// Tiles are handed out statically (pair p takes tiles p, p + pairs, ...): both CTAs of a pair derive the same
// sequence without talking to each other.
// Ragged groups: a tile may read rows of the next expert (or zeros past the end); they are never stored.
// K and N tails are zero-filled by TMA.  All waits are bounded; an expired wait sets the ctx's status word.
// No copy in this file uses cluster multicast: every CTA fetches what it needs with its own loads.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"

namespace cosmoe {

namespace {

constexpr int kBM = 128;  // rows per CTA and tile (TMEM lanes)
constexpr int kBK = 64;   // K elements per stage (128 bytes of bf16 = one swizzle row)
constexpr int kEpiWarps = 8;  // two per quarter of the TMEM lanes, splitting the columns
constexpr int kThreadsGG = (2 + kEpiWarps) * 32;
constexpr int kTmemCols = 512;  // two accumulator buffers of 256 columns
constexpr int kAccCols = 256;
constexpr int kMaxStagesGG = 6;
constexpr int kPairRows = 2 * kBM;  // rows of a pair's tile

enum Epi { EPI_SWIGLU = 0, EPI_BF16_PAIR = 1, EPI_BF16 = 2, EPI_F32 = 3 };
// How the B operand of a tile is laid out and shared between the two CTAs of a pair (rank 0 / rank 1):
enum BMode {
  B_PAIR = 0,    // interleaved matrix, columns [0, bn) = sub-row 0 (rank 0 loads them), [bn, 2 bn) = sub-row 1 (rank 1)
  B_DUAL = 1,    // the same columns, but sub-row 1 meets a second A operand: two MMAs of N = bn, each rank loads half of both
  B_SINGLE = 2,  // one sub-row, K-major: rank r loads rows [n0 + r bn/2, n0 + (r+1) bn/2)
  B_NMAJOR = 3   // one sub-row stored [k][n] (the down rows of gud): rank r loads its bn/2 columns in 64-column boxes
};

struct GGParams {
  const int32_t* offsets;  // [E+1] slot ranges per expert
  int E;
  int K;         // contraction length
  int n_total;   // output columns (per sub-row in B_PAIR / B_DUAL)
  int n_store;   // columns stored, >= n_total: the columns between are written as zeros (accumulators of B rows that do
                 // not exist), so that a consumer may read the padded width
  int bn;        // output columns per tile (per sub-row in B_PAIR / B_DUAL: <= 128; else <= 256)
  int bmode;
  int b_sub;     // sub-row of the interleaved matrix that B_SINGLE / B_NMAJOR tiles read
  int k_wrap;    // > 0: the B operand's k coordinate wraps at k_wrap (A = [hi | lo] halves of a split operand)
  int split;     // bf16 epilogues also store the rounding remainder: value = hi + lo, lo at column offset out_off_lo
  int epi;
  void* out;
  long long ld_out;    // elements
  long long out_off2;  // EPI_BF16_PAIR: column offset of the second half
  long long out_off_lo;  // split: column offset of the remainders
  int ksplit;             // the contraction is cut into this many parts, each a work item of its own ...
  long long plane_elems;  // ... writing its partial sums plane_elems further on in `out` (EPI_F32 only)
  int n_stages;
  DeviceState* st;
};

// ---- PTX wrappers ------------------------------------------------------------------------------------
// Tiled loads whose completion may be counted on a barrier of the other CTA of the pair (cta_group::2); the
// data always lands in the issuing CTA's own shared memory.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], "
      "[%4];" ::"r"(smem_u32(dst)),
      "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, "
      "%5}], [%6];" ::"r"(smem_u32(dst)),
      "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory object in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(const void* smem_ptr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(smem_ptr)), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// The barrier at this shared-memory offset gets one arrival IN BOTH CTAs of the pair when every MMA this thread
// has issued so far has completed.  (A multicast of barrier arrivals, not of data: no copy in this file is multicast.)
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                   smem_u32(bar)),
               "h"((unsigned short)3)
               : "memory");
}
// `acc` == 0: the product overwrites the accumulator; otherwise it is added.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor (128-byte swizzle).  K-major tiles: rows of 128 bytes, 8-row groups 1024
// bytes apart (stride byte offset), the leading offset is not used.  N-major tiles: 64 columns (128 bytes) per
// k-row, 8-k-row groups 1024 bytes apart (stride), 64-column blocks `lbo` bytes apart (leading).
// The start address sits in the low 14 bits (in units of 16 bytes), so stepping through a stage or through the
// ring is an addition to the low word.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= 1ull << 46;  // descriptor version of this architecture
  d |= 2ull << 61;  // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K- or N-major, M = 256 over the pair, N = n.
__device__ __forceinline__ uint32_t instr_desc(int n, bool b_nmajor) {
  uint32_t d = 0;
  d |= 1u << 4;   // accumulator format: fp32
  d |= 1u << 7;   // A: bf16
  d |= 1u << 10;  // B: bf16
  d |= (b_nmajor ? 1u : 0u) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(kPairRows >> 4) << 24;
  return d;
}

struct SmemGG {
  uint64_t full[kMaxStagesGG];   // leader's: both CTAs' operands of the stage have landed
  uint64_t empty[kMaxStagesGG];  // own: the MMAs have finished reading this CTA's stage
  uint64_t accum_full[2];        // own: all MMAs of the tile in accumulator buffer b have completed
  uint64_t accum_empty[2];       // leader's: the epilogue warps of both CTAs have read buffer b out of TMEM
  uint32_t tmem_base;
  int abort;
  int tile_prefix[MOE_MAX_EXPERTS + 1];  // 256-row tiles per expert, exclusive scan
};

struct Tile {
  int e, m0, m_end, n0, ks;
};

// idx-th tile of this launch: row-tile major, column tile minor (pairs that run side by side share the A rows
// and sweep the expert's B columns, which then sit in L2 for the expert's other row tiles).
__device__ __forceinline__ bool decode_tile(const GGParams& P, const SmemGG& sm, int idx, int n_tiles, Tile& t) {
  const int per_row = n_tiles * P.ksplit;
  const int mt = idx / per_row, rem = idx - mt * per_row;
  const int nt = rem / P.ksplit;
  t.ks = rem - nt * P.ksplit;
  if (mt >= sm.tile_prefix[P.E]) return false;
  int e = 0;
  while (sm.tile_prefix[e + 1] <= mt) ++e;
  t.e = e;
  t.m0 = P.offsets[e] + (mt - sm.tile_prefix[e]) * kPairRows;
  t.m_end = P.offsets[e + 1];
  t.n0 = nt * P.bn;
  return true;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

__global__ void __launch_bounds__(kThreadsGG, 1)
    grouped_gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                        const __grid_constant__ CUtensorMap map_b, const GGParams P) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // stage layout: [A 16 KB][A' 16 KB, B_DUAL only][B <= 16 KB], all 1024-byte aligned (swizzle atoms); identical
  // in both CTAs, because the MMA addresses the pair's operands by one shared-memory offset
  const uint32_t a_bytes = kBM * kBK * 2;
  const uint32_t n_a = P.bmode == B_DUAL ? 2u : 1u;
  const uint32_t b_rows = (P.bmode == B_PAIR || P.bmode == B_DUAL) ? (uint32_t)P.bn : (uint32_t)P.bn / 2u;  // per CTA
  const uint32_t b_bytes = b_rows * kBK * 2;
  const uint32_t stage_bytes = n_a * a_bytes + 128u * kBK * 2u;
  unsigned char* stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemGG& sm = *reinterpret_cast<SmemGG*>(stages + (size_t)P.n_stages * stage_bytes);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = P.n_stages;
  const int num_kb = (P.K + kBK - 1) / kBK;
  const int n_tiles = (P.n_total + P.bn - 1) / P.bn;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  pdl_launch_dependents();
  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.empty[i], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sm.accum_full[b], 1);
      mbar_init(&sm.accum_empty[b], 2 * kEpiWarps);
    }
    sm.abort = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {  // one warp of each CTA of the pair
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  // everything above touches only this CTA's shared memory and TMEM; the expert offsets and the operands may
  // come from the kernel before
  pdl_wait();
  if (tid == 0) {
    int run = 0;
    for (int i = 0; i < P.E; ++i) {
      sm.tile_prefix[i] = run;
      const int rows = P.offsets[i + 1] - P.offsets[i];
      run += rows > 0 ? (rows + kPairRows - 1) / kPairRows : 0;
    }
    sm.tile_prefix[P.E] = run;
  }
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();  // the other CTA's barriers are initialised before anything is counted on them
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  Tile t;

  if (warp == 0) {
    // ================================================================= TMA producer (both CTAs)
    if (lane == 0) {
      int it = 0;              // k-blocks issued so far, over all tiles
      uint32_t slot = 0, par = 1;  // ring position; parity of the `empty` phase the slot's next fill waits for
      bool ok = true;
      const uint32_t tx_pair = 2u * (n_a * a_bytes + b_bytes);  // bytes both CTAs bring in per stage
      const uint32_t full0 = map_to_rank(&sm.full[0], 0u);      // the leader's stage barriers, 8 bytes apart
      const int half_bn = P.bn / 2;
      for (int idx = pair; ok && decode_tile(P, sm, idx, n_tiles, t); idx += n_pairs) {
        const int kb0 = t.ks * num_kb / P.ksplit, kb1 = (t.ks + 1) * num_kb / P.ksplit;
        const int a_row = t.m0 + (int)rank * kBM;
        int k0 = kb0 * kBK;
        int kB = P.k_wrap > 0 ? k0 % P.k_wrap : k0;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          if (it >= NS && !mbar_wait(&sm.empty[slot], par)) {
            flag_error(P.st, MOE_ERR_TIMEOUT, 0x400u);
            sm.abort = 1;
            ok = false;
            break;
          }
          unsigned char* st_a0 = stages + (size_t)slot * stage_bytes;
          unsigned char* st_b = st_a0 + n_a * a_bytes;
          const uint32_t bar = full0 + 8u * slot;
          if (rank == 0) mbar_arrive_expect_tx(&sm.full[slot], tx_pair);
          tma_load_2d(st_a0, &map_a0, k0, a_row, bar);
          if (P.bmode == B_PAIR) {
            tma_load_4d(st_b, &map_b, kB, (int)rank, t.n0, t.e, bar);
          } else if (P.bmode == B_DUAL) {
            const int nr = t.n0 + (int)rank * half_bn;
            tma_load_2d(st_a0 + a_bytes, &map_a1, k0, a_row, bar);
            tma_load_4d(st_b, &map_b, kB, 0, nr, t.e, bar);
            tma_load_4d(st_b + (size_t)half_bn * kBK * 2, &map_b, kB, 1, nr, t.e, bar);
          } else if (P.bmode == B_SINGLE) {
            tma_load_4d(st_b, &map_b, kB, P.b_sub, t.n0 + (int)rank * half_bn, t.e, bar);
          } else {
            const int nc = t.n0 + (int)rank * half_bn;
            for (int j = 0; j < P.bn / 128; ++j)
              tma_load_4d(st_b + (size_t)j * 64 * kBK * 2, &map_b, nc + 64 * j, P.b_sub, kB, t.e, bar);
          }
          k0 += kBK, kB += kBK;
          if (P.k_wrap > 0 && kB >= P.k_wrap) kB -= P.k_wrap;
          if (++slot == (uint32_t)NS) slot = 0, par ^= 1u;
        }
      }
      if (!ok && rank == 0) {  // copies in flight (both CTAs' complete on these barriers) must land before the pair goes away
        for (int j = max(0, it - NS); j < it; ++j) (void)mbar_wait(&sm.full[j % NS], (j / NS) & 1);
      }
    }
  } else if (warp == 1) {
    // ================================================================= MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      // One thread feeds the tensor cores of both SMs, so its instruction stream is kept short: the ring position
      // is a counter, not a division, and the operand descriptors are a constant high word plus a low word that
      // steps through the stage (K-major operands: 32 bytes per 16 k-values; N-major: 16 k-rows of 128 bytes).
      const int n_mma = P.bmode == B_PAIR ? 2 * P.bn : P.bn;
      const uint32_t idesc = instr_desc(n_mma, P.bmode == B_NMAJOR);
      const uint64_t hi_k = smem_desc(0, 16, 1024) & 0xffffffff00000000ull;
      const uint64_t hi_b = (P.bmode == B_NMAJOR ? smem_desc(0, 64 * kBK * 2, 1024) : smem_desc(0, 16, 1024)) & 0xffffffff00000000ull;
      const uint32_t lo_b_lbo = (P.bmode == B_NMAJOR ? (uint32_t)(64 * kBK * 2 >> 4) : 1u) << 16;
      const uint32_t b_step = P.bmode == B_NMAJOR ? (2048u >> 4) : (32u >> 4);
      const uint32_t stage0 = smem_u32(stages) >> 4, stage_step = stage_bytes >> 4;
      const uint32_t b_off = (n_a * a_bytes) >> 4, a1_off = a_bytes >> 4, b1_off = ((uint32_t)(P.bn / 2) * kBK * 2) >> 4;
      uint32_t slot = 0, par = 0, st_lo = stage0;
      int tile_i = 0;
      bool ok = true;
      for (int idx = pair; ok && decode_tile(P, sm, idx, n_tiles, t); idx += n_pairs, ++tile_i) {
        const int buf = tile_i & 1;
        if (tile_i >= 2) {  // the accumulators two tiles back must have left this buffer, in both CTAs
          if (!mbar_wait(&sm.accum_empty[buf], ((tile_i >> 1) - 1) & 1)) {
            flag_error(P.st, MOE_ERR_TIMEOUT, 0x403u);
            sm.abort = 1;
            break;
          }
          tc_fence_after();
        }
        const uint32_t d_tmem = tmem + (uint32_t)(buf * kAccCols);
        const int kb0 = t.ks * num_kb / P.ksplit, kb1 = (t.ks + 1) * num_kb / P.ksplit;
        uint32_t acc = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(&sm.full[slot], par)) {
            flag_error(P.st, MOE_ERR_TIMEOUT, 0x401u);
            sm.abort = 1;
            ok = false;
            break;
          }
          tc_fence_after();
          const uint64_t da = hi_k | (uint64_t)(st_lo | (1u << 16));
          const uint64_t db = hi_b | (uint64_t)((st_lo + b_off) | lo_b_lbo);
          if (P.bmode == B_DUAL) {
            const uint64_t da1 = da + a1_off, db1 = db + b1_off;
#pragma unroll
            for (uint32_t kk = 0; kk < kBK / 16; ++kk) {
              tc_mma_bf16(d_tmem, da + 2u * kk, db + 2u * kk, idesc, acc | kk);
              tc_mma_bf16(d_tmem + (uint32_t)P.bn, da1 + 2u * kk, db1 + 2u * kk, idesc, acc | kk);
            }
          } else {
#pragma unroll
            for (uint32_t kk = 0; kk < kBK / 16; ++kk) tc_mma_bf16(d_tmem, da + 2u * kk, db + b_step * kk, idesc, acc | kk);
          }
          acc = 1;
          tc_commit_pair(&sm.empty[slot]);  // both CTAs' producers may refill the stage once these MMAs have read it
          st_lo += stage_step;
          if (++slot == (uint32_t)NS) slot = 0, par ^= 1u, st_lo = stage0;
        }
        if (ok) tc_commit_pair(&sm.accum_full[buf]);
      }
    }
  } else {
    // ================================================================= epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;  // TMEM lanes 32q .. 32q+31 are the only ones this warp may read
    const int cpar = (warp - 2) >> 2;  // which of the two warps of this quarter: it takes every other 32-column chunk
    const uint32_t acce_bar[2] = {map_to_rank(&sm.accum_empty[0], 0u), map_to_rank(&sm.accum_empty[1], 0u)};
    int tile_i = 0;
    for (int idx = pair; decode_tile(P, sm, idx, n_tiles, t); idx += n_pairs, ++tile_i) {
      const int buf = tile_i & 1;
      if (!mbar_wait(&sm.accum_full[buf], (tile_i >> 1) & 1)) {
        if (lane == 0) flag_error(P.st, MOE_ERR_TIMEOUT, 0x402u);
        break;
      }
      tc_fence_after();
      const int ncols = min(P.bn, P.n_store - t.n0);  // columns of this tile to store (multiple of 8)
      const int row = t.m0 + (int)rank * kBM + 32 * q + lane;
      const bool row_ok = row < t.m_end;
      const uint32_t tbase = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kAccCols);
      if (P.epi == EPI_SWIGLU || P.epi == EPI_BF16_PAIR) {
        __nv_bfloat16* out = (__nv_bfloat16*)P.out + (size_t)row * P.ld_out + t.n0;
        for (int c = 32 * cpar; c < P.bn; c += 64) {
          uint32_t g[32], u[32];
          tc_ld32(tbase + c, g);
          tc_ld32(tbase + P.bn + c, u);
          tc_wait_ld();
          if (!row_ok) continue;
          if (P.epi == EPI_SWIGLU) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (c + 8 * v < ncols) {
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  o[j] = pack_bf16x2(silu_mul(__uint_as_float(g[8 * v + 2 * j]), __uint_as_float(u[8 * v + 2 * j])),
                                     silu_mul(__uint_as_float(g[8 * v + 2 * j + 1]), __uint_as_float(u[8 * v + 2 * j + 1])));
                *reinterpret_cast<uint4*>(out + c + 8 * v) = make_uint4(o[0], o[1], o[2], o[3]);
              }
            }
          } else {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (c + 8 * v < ncols) {
                uint32_t o[4], p[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  o[j] = pack_bf16x2(__uint_as_float(g[8 * v + 2 * j]), __uint_as_float(g[8 * v + 2 * j + 1]));
                  p[j] = pack_bf16x2(__uint_as_float(u[8 * v + 2 * j]), __uint_as_float(u[8 * v + 2 * j + 1]));
                }
                *reinterpret_cast<uint4*>(out + c + 8 * v) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(out + P.out_off2 + c + 8 * v) = make_uint4(p[0], p[1], p[2], p[3]);
                if (P.split) {
                  uint32_t ol[4], pl[4];
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    ol[j] = pack_bf16x2(__uint_as_float(g[8 * v + 2 * j]) - __uint_as_float(o[j] << 16),
                                        __uint_as_float(g[8 * v + 2 * j + 1]) - __uint_as_float(o[j] & 0xffff0000u));
                    pl[j] = pack_bf16x2(__uint_as_float(u[8 * v + 2 * j]) - __uint_as_float(p[j] << 16),
                                        __uint_as_float(u[8 * v + 2 * j + 1]) - __uint_as_float(p[j] & 0xffff0000u));
                  }
                  *reinterpret_cast<uint4*>(out + P.out_off_lo + c + 8 * v) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                  *reinterpret_cast<uint4*>(out + P.out_off2 + P.out_off_lo + c + 8 * v) =
                      make_uint4(pl[0], pl[1], pl[2], pl[3]);
                }
              }
            }
          }
        }
      } else {
        for (int c = 32 * cpar; c < P.bn; c += 64) {
          uint32_t a[32];
          tc_ld32(tbase + c, a);
          tc_wait_ld();
          if (!row_ok) continue;
          if (P.epi == EPI_F32) {
            float* out = (float*)P.out + (size_t)t.ks * P.plane_elems + (size_t)row * P.ld_out + t.n0 + c;
#pragma unroll
            for (int v = 0; v < 8; ++v)
              if (c + 4 * v < ncols)
                *reinterpret_cast<uint4*>(out + 4 * v) = make_uint4(a[4 * v], a[4 * v + 1], a[4 * v + 2], a[4 * v + 3]);
          } else {
            __nv_bfloat16* out = (__nv_bfloat16*)P.out + (size_t)row * P.ld_out + t.n0 + c;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (c + 8 * v < ncols) {
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  o[j] = pack_bf16x2(__uint_as_float(a[8 * v + 2 * j]), __uint_as_float(a[8 * v + 2 * j + 1]));
                *reinterpret_cast<uint4*>(out + 8 * v) = make_uint4(o[0], o[1], o[2], o[3]);
                if (P.split) {
                  uint32_t ol[4];
#pragma unroll
                  for (int j = 0; j < 4; ++j)
                    ol[j] = pack_bf16x2(__uint_as_float(a[8 * v + 2 * j]) - __uint_as_float(o[j] << 16),
                                        __uint_as_float(a[8 * v + 2 * j + 1]) - __uint_as_float(o[j] & 0xffff0000u));
                  *reinterpret_cast<uint4*>(out + P.out_off_lo + 8 * v) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                }
              }
            }
          }
        }
      }
      // the accumulators are in registers / memory now: hand the buffer back to the leader's MMA thread
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acce_bar[buf]);
    }
  }
  // ---- teardown: every role gets here in bounded time; neither CTA leaves while the other may still count on
  // its barriers or read its operands
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
  }
}

// ---- host: tensor maps --------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    fn = (EncodeTiledFn)p;
  }
  return fn;
}

// rank-2 map over a row-major bf16 matrix [rows][ld], columns [0, cols): box 64 x 128
int make_map_a(CUtensorMap* m, const void* base, long long rows, long long cols, long long ld) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return MOE_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {kBK, kBM};
  const cuuint32_t es[2] = {1, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MOE_OK : MOE_ERR_CUDA;
}
// rank-4 map over an interleaved matrix [S][rows][nsub][inner]: coordinates (inner, sub, row, slot)
int make_map_b(CUtensorMap* m, const void* base, long long inner, int nsub, long long rows, int slots, int box_inner,
               int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return MOE_ERR_CUDA;
  const cuuint64_t dims[4] = {(cuuint64_t)inner, (cuuint64_t)nsub, (cuuint64_t)rows, (cuuint64_t)slots};
  const cuuint64_t strides[3] = {(cuuint64_t)inner * 2, (cuuint64_t)inner * nsub * 2,
                                 (cuuint64_t)inner * nsub * rows * 2};
  const cuuint32_t box[4] = {(cuuint32_t)box_inner, 1, (cuuint32_t)box_rows, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MOE_OK : MOE_ERR_CUDA;
}

// Pairs of CTAs the device can hold at once (one CTA per SM; a pair sits on two SMs of one cluster).
void pair_launch_config(cudaLaunchConfig_t& lc, cudaLaunchAttribute* attr, int ctas, size_t smem, cudaStream_t s) {
  lc = cudaLaunchConfig_t{};
  lc.gridDim = dim3(ctas), lc.blockDim = dim3(kThreadsGG), lc.dynamicSmemBytes = smem, lc.stream = s;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr, lc.numAttrs = 2;
}

// Pairs of CTAs the device can hold at once (one CTA per SM; a pair sits on two SMs of one cluster).
int max_pairs(moe_ctx* ctx, size_t smem) {
  cudaLaunchConfig_t lc;
  cudaLaunchAttribute attr[2];
  pair_launch_config(lc, attr, ctx->sm_count & ~1, smem, nullptr);
  lc.numAttrs = 1;  // the cluster shape alone decides the occupancy
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, grouped_gemm_kernel, &lc) != cudaSuccess || n < 1) {
    (void)cudaGetLastError();
    n = ctx->sm_count / 2;
  }
  return std::max(1, std::min(n, ctx->sm_count / 2));
}

int launch_gg(moe_ctx* ctx, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b, GGParams P,
              int n_slots, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  P.E = c.n_experts;
  P.st = ctx->d_state;
  if (P.n_store < P.n_total) P.n_store = P.n_total;
  if (P.ksplit < 1) P.ksplit = 1;
  const int n_tiles = (P.n_total + P.bn - 1) / P.bn;
  const size_t stage_bytes = (size_t)kBM * kBK * 2 * (P.bmode == B_DUAL ? 2 : 1) + 128 * kBK * 2;
  P.n_stages = P.bmode == B_DUAL ? 4 : kMaxStagesGG;
  const size_t smem = P.n_stages * stage_bytes + sizeof(SmemGG) + 1024 + 128;
  if ((long long)smem > ctx->max_smem_optin) return MOE_ERR_UNSUPPORTED;
  MOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const long long m_tiles = (n_slots + kPairRows - 1) / kPairRows + c.n_experts;  // upper bound
  const int pairs = (int)std::min<long long>(m_tiles * n_tiles * P.ksplit, max_pairs(ctx, smem));
  cudaLaunchConfig_t lc;
  cudaLaunchAttribute attr[2];
  pair_launch_config(lc, attr, 2 * pairs, smem, s);
  MOE_CUDA_TRY(cudaLaunchKernelEx(&lc, grouped_gemm_kernel, a0, a1, b, P));
  ctx->launches++;
  return MOE_OK;
}

// Output columns per tile: the largest of 64, 128, ... `cap` that is not mostly padding.
int pick_bn(int n_total, int cap, int floor_bn = 64) {
  int bn = cap;
  while (bn > floor_bn && bn / 2 >= n_total) bn /= 2;
  return bn;
}

}  // namespace

int launch_tensor_ffn(moe_ctx* ctx, const void* x, int T, const moe_weights* w, const int32_t* offsets,
                      const int32_t* perm, char* ws, const WsLayout& L, float* out_slots, int* out_planes,
                      cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  if (w->expert_slot) return MOE_ERR_UNSUPPORTED;  // the tensor path reads experts in place (slot == expert)
  const int d = c.d_model, f = c.d_ff, r = c.wd_rank, E = c.n_experts;
  const int n_slots = T * c.top_k;
  if (out_planes) *out_planes = 1;
  void* xperm = ws + L.xperm;
  void* hidden = ws + L.hidden;
  int rc = launch_gather_rows(ctx, x, perm, n_slots, xperm, s);
  if (rc != MOE_OK) return rc;
  CUtensorMap ma, ma1, mb;
  GGParams P{};
  P.offsets = offsets;
  if (r == 0) {
    // (1) hidden = silu(X Wg) * (X Wu): the tile's 128 gate rows come in through one CTA, its 128 up rows through the other
    if ((rc = make_map_a(&ma, xperm, n_slots, d, d)) != MOE_OK) return rc;
    if ((rc = make_map_b(&mb, w->gud, d, 3, f, E, kBK, 128)) != MOE_OK) return rc;
    P.K = d, P.n_total = f, P.bn = 128, P.bmode = B_PAIR, P.b_sub = 0, P.epi = EPI_SWIGLU;
    P.out = hidden, P.ld_out = f, P.out_off2 = 0;
    if ((rc = launch_gg(ctx, ma, ma, mb, P, n_slots, s)) != MOE_OK) return rc;
    // (2) out_slots = hidden Wd   (B = down rows of gud: [k = hidden unit][n = model column], n contiguous)
    if ((rc = make_map_a(&ma, hidden, n_slots, f, f)) != MOE_OK) return rc;
    if ((rc = make_map_b(&mb, w->gud, d, 3, f, E, 64, kBK)) != MOE_OK) return rc;
    P.K = f, P.n_total = d, P.bn = pick_bn(d, 256, 128), P.bmode = B_NMAJOR, P.b_sub = 2;
    P.epi = EPI_F32, P.out = out_slots, P.ld_out = d, P.out_off2 = 0;
    if (out_planes && n_slots <= kKSplitMaxSlots) {
      // short prefill: too few tiles for the SMs, and every tile streams a long run of weights.  The caller
      // sums planes: cut the contraction so that every pair streams a part, each part into its own plane.
      const int m_est = std::max((n_slots + kPairRows - 1) / kPairRows, std::min(E, n_slots));
      const long long tiles = (long long)m_est * ((d + P.bn - 1) / P.bn);
      int ks = (int)((ctx->sm_count / 2) / std::max<long long>(tiles, 1));
      ks = std::min(std::min(ks, kKSplitMax), (f + kBK - 1) / kBK);
      if (ks > 1) {
        P.ksplit = ks, P.plane_elems = (long long)n_slots * d;
        *out_planes = ks;
      }
    }
    return launch_gg(ctx, ma, ma, mb, P, n_slots, s);
  }
  // The rank-r intermediates t and v are kept as hi + lo pairs of bf16 (value = hi + lo): the GEMMs that
  // consume them run over K = 2 * rp with the weight slices repeated, so the intermediates carry ~16 mantissa
  // bits and the chain's only bf16 roundings are those of the dense path (hidden activations, output).
  // rp = r rounded up to the K step: the columns [r, rp) of an intermediate are stored as zeros and meet
  // weight rows past the end of the matrix (zero-filled by the loads), so any rank that is a multiple of 8 works.
  const int rp = (r + kBK - 1) / kBK * kBK;
  const int tw = 2 * rp;  // stored width of one intermediate: hi | lo
  void* mid_a = ws + L.mid_a;  // [n_slots][2*tw]: t_g (hi | lo) | t_u (hi | lo)
  void* mid_b = ws + L.mid_b;  // [n_slots][tw]:   v (hi | lo)
  // (1) T = X [gL | uL]
  if ((rc = make_map_a(&ma, xperm, n_slots, d, d)) != MOE_OK) return rc;
  P.bn = pick_bn(r, 128);
  if ((rc = make_map_b(&mb, w->wd_a, d, 2, r, E, kBK, P.bn)) != MOE_OK) return rc;
  P.K = d, P.n_total = r, P.bmode = B_PAIR, P.b_sub = 0, P.epi = EPI_BF16_PAIR;
  P.k_wrap = 0, P.split = 1, P.out = mid_a, P.ld_out = 2 * tw, P.out_off2 = tw, P.out_off_lo = rp, P.n_store = rp;
  if ((rc = launch_gg(ctx, ma, ma, mb, P, n_slots, s)) != MOE_OK) return rc;
  // (2) hidden = silu(Tg gR) * (Tu uR): two A operands, each CTA brings half of the gate and half of the up rows
  if ((rc = make_map_a(&ma, mid_a, n_slots, tw, 2 * tw)) != MOE_OK) return rc;
  if ((rc = make_map_a(&ma1, (const __nv_bfloat16*)mid_a + tw, n_slots, tw, 2 * tw)) != MOE_OK) return rc;
  if ((rc = make_map_b(&mb, w->wd_b, r, 2, f, E, kBK, 64)) != MOE_OK) return rc;
  P.K = tw, P.n_total = f, P.bn = 128, P.bmode = B_DUAL, P.b_sub = 0, P.epi = EPI_SWIGLU;
  P.k_wrap = rp, P.split = 0, P.out = hidden, P.ld_out = f, P.out_off2 = 0, P.out_off_lo = 0, P.n_store = 0;
  if ((rc = launch_gg(ctx, ma, ma1, mb, P, n_slots, s)) != MOE_OK) return rc;
  // (3) V = hidden dL
  if ((rc = make_map_a(&ma, hidden, n_slots, f, f)) != MOE_OK) return rc;
  P.bn = pick_bn(r, 256);
  if ((rc = make_map_b(&mb, w->wd_c, f, 1, r, E, kBK, P.bn / 2)) != MOE_OK) return rc;
  P.K = f, P.n_total = r, P.bmode = B_SINGLE, P.b_sub = 0, P.epi = EPI_BF16;
  P.k_wrap = 0, P.split = 1, P.out = mid_b, P.ld_out = tw, P.out_off2 = 0, P.out_off_lo = rp, P.n_store = rp;
  if ((rc = launch_gg(ctx, ma, ma, mb, P, n_slots, s)) != MOE_OK) return rc;
  // (4) out_slots = V dR
  if ((rc = make_map_a(&ma, mid_b, n_slots, tw, tw)) != MOE_OK) return rc;
  P.bn = pick_bn(d, 256);
  if ((rc = make_map_b(&mb, w->wd_d, r, 1, d, E, kBK, P.bn / 2)) != MOE_OK) return rc;
  P.K = tw, P.n_total = d, P.bmode = B_SINGLE, P.b_sub = 0, P.epi = EPI_F32;
  P.k_wrap = rp, P.split = 0, P.out = out_slots, P.ld_out = d, P.out_off2 = 0, P.out_off_lo = 0, P.n_store = 0;
  return launch_gg(ctx, ma, ma, mb, P, n_slots, s);
}

}  // namespace cosmoe
