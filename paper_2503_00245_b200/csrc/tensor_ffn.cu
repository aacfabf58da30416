// Tensor-core (prefill) path of the expert FFN: grouped GEMMs on the 5th-generation tensor cores.
//
// Tokens are grouped by expert (moe_permute), their rows gathered into a bf16 operand, and every expert's
// FFN becomes dense contractions  C[m, n] = sum_k A[m, k] * B_e[n, k]  over that expert's rows:
//
//   dense experts  (1) H = silu(X Wg) * (X Wu)   A = gathered x,  B = gate / up rows of gud   -> bf16 hidden
//                  (2) O = H Wd                  A = H,           B = down rows of gud (N-major) -> fp32 slots
//   Eq. 1 factors  (1) T = X [gL | uL]   (2) H = silu(Tg gR) * (Tu uR)   (3) V = H dL   (4) O = V dR
//
// One CTA computes one tile of up to 256 rows x 256 columns: two 128-row halves with their own accumulators
// share every B slice (128 flop per operand byte moved from L2, against 85 for a 128-row tile); a tile whose
// second half would be empty (the ragged end of an expert's rows) runs one half.  Roles:
//   warp 0     TMA producer: 64-wide K slices of A and B into a ring of shared-memory stages (128-byte swizzle);
//   warp 1     allocates tensor memory and issues tcgen05.mma (M = 128, N <= 256, K = 16 per instruction) with
//              fp32 accumulators in TMEM; a commit releases each stage back to the producer;
//   warps 2-5  epilogue: tcgen05.ld the accumulators (one TMEM lane = one output row per thread), apply
//              SiLU * mul or nothing, convert, store the rows that belong to the expert.
// Ragged groups: a tile may read rows of the next expert (or zeros past the end); they are never stored.
// K and N tails are zero-filled by TMA.  All waits are bounded; an expired wait sets the ctx's status word.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"

namespace cosmoe {

namespace {

constexpr int kBM = 128;  // rows per tile (TMEM lanes)
constexpr int kBK = 64;   // K elements per stage (128 bytes of bf16 = one swizzle row)
constexpr int kTileQueue = 8;  // tile indices in flight between the producer and the other roles
constexpr int kEpiWarps = 8;  // two per quarter of the TMEM lanes, splitting the columns
constexpr int kThreadsGG = (2 + kEpiWarps) * 32;
constexpr int kTmemCols = 512;  // two accumulators of 256 columns
constexpr int kMaxStagesGG = 4;
constexpr int kTileRows = 2 * kBM;  // rows per tile when the A operand is single (two halves)

enum Epi { EPI_SWIGLU = 0, EPI_BF16_PAIR = 1, EPI_BF16 = 2, EPI_F32 = 3 };

struct GGParams {
  const int32_t* offsets;  // [E+1] slot ranges per expert
  int E;
  int K;         // contraction length
  int n_total;   // output columns (per half when `pair`)
  int bn;        // output columns per tile (per half when `pair`): <= 128 when pair, <= 256 otherwise
  int pair;      // B tile = two halves (sub-rows 0 and 1 of an interleaved matrix): accumulator columns [0,bn) and [128,128+bn)
  int dual_a;    // the second half has its own A operand
  int b_nmajor;  // B is stored [k][n] (n contiguous): the down rows of gud
  int b_sub;     // sub-row of the interleaved matrix that single / N-major tiles read
  int tile_rows; // rows per tile: 256 (two halves) or 128
  int k_wrap;    // > 0: the B operand's k coordinate wraps at k_wrap (A = [hi | lo] halves of a split operand)
  int split;     // bf16 epilogues also store the rounding remainder: value = hi + lo, lo at column offset out_off_lo
  int epi;
  void* out;
  long long ld_out;    // elements
  long long out_off2;  // EPI_BF16_PAIR: column offset of the second half
  long long out_off_lo;  // split: column offset of the remainders
  int ctr_idx;            // which word of DeviceState::tile_ctr hands out this launch's tiles (the other is cleared)
  int single_a;           // 128-row tiles, one A operand: the stage has no A' part
  int ksplit;             // the contraction is cut into this many parts, each a work item of its own ...
  long long plane_elems;  // ... writing its partial sums plane_elems further on in `out` (EPI_F32 only)
  int n_stages;
  DeviceState* st;
};

// ---- PTX wrappers ------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
          "r"(smem_u32(dst)),
      "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], "
      "[%6];" ::"r"(smem_u32(dst)),
      "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)acc)
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
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= 1ull << 46;  // descriptor version of this architecture
  d |= 2ull << 61;  // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K- or N-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc(int n, bool b_nmajor) {
  uint32_t d = 0;
  d |= 1u << 4;   // accumulator format: fp32
  d |= 1u << 7;   // A: bf16
  d |= 1u << 10;  // B: bf16
  d |= (b_nmajor ? 1u : 0u) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(kBM >> 4) << 24;
  return d;
}

struct SmemGG {
  uint64_t full[kMaxStagesGG];
  uint64_t empty[kMaxStagesGG];
  uint64_t accum_full;   // all MMAs of the current tile have completed
  uint64_t accum_empty;  // the epilogue has read the accumulators out of TMEM (all epilogue warps arrive)
  uint64_t tq_full[kTileQueue];   // the producer has put a tile index into tq[i]
  uint64_t tq_empty[kTileQueue];  // the MMA thread and every epilogue warp have read it
  int tq[kTileQueue];
  uint32_t tmem_base;
  int abort;
  int tile_prefix[MOE_MAX_EXPERTS + 1];  // row tiles per expert, exclusive scan
};

struct Tile {
  int e, m0, m_end, halves, n0, ks;
};

// idx-th tile of this launch: row-tile major, column tile minor (CTAs that run side by side share the A rows
// and sweep the expert's B columns, which then sit in L2 for the expert's other row tiles).
__device__ __forceinline__ bool decode_tile(const GGParams& P, const SmemGG& sm, int idx, int n_tiles, Tile& t) {
  const int per_row = n_tiles * P.ksplit;
  const int mt = idx / per_row, rem = idx - mt * per_row;
  const int nt = rem / P.ksplit;
  t.ks = rem - nt * P.ksplit;
  if (mt >= sm.tile_prefix[P.E]) return false;
  int e = 0;
  while (sm.tile_prefix[e + 1] <= mt) ++e;
  const int tile_rows = P.tile_rows;
  t.e = e;
  t.m0 = P.offsets[e] + (mt - sm.tile_prefix[e]) * tile_rows;
  t.m_end = P.offsets[e + 1];
  t.halves = (!P.dual_a && tile_rows > kBM && t.m_end - t.m0 > kBM) ? 2 : 1;
  t.n0 = nt * P.bn;
  return true;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// Persistent: CTA c takes tiles c, c + gridDim.x, ...; the TMA producer runs ahead into the next tile while
// the epilogue of the current one drains TMEM.
__global__ void __launch_bounds__(kThreadsGG, 1)
    grouped_gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                        const __grid_constant__ CUtensorMap map_b, const GGParams P) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // stage layout: [A 16 KB][A' 16 KB][B 32 KB], all 1024-byte aligned (swizzle atoms).  A' is the second
  // 128-row half of the tile, or the second operand (dual_a, 128-row tiles)
  const uint32_t a_bytes = kBM * kBK * 2, b_bytes = 256 * kBK * 2;
  // (tiles of one 128-row half with a single A operand leave A' out: stages of 48 KB, one more of them)
  const uint32_t n_a = P.single_a ? 1u : 2u;
  const uint32_t stage_bytes = n_a * a_bytes + b_bytes;
  unsigned char* stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemGG& sm = *reinterpret_cast<SmemGG*>(stages + (size_t)P.n_stages * stage_bytes);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = P.n_stages;
  const int num_kb = (P.K + kBK - 1) / kBK;
  const int n_tiles = (P.n_total + P.bn - 1) / P.bn;

  pdl_launch_dependents();
  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.empty[i], 1);
    }
    for (int i = 0; i < kTileQueue; ++i) {
      mbar_init(&sm.tq_full[i], 1);
      mbar_init(&sm.tq_empty[i], 1 + kEpiWarps);
    }
    mbar_init(&sm.accum_full, 1);
    mbar_init(&sm.accum_empty, kEpiWarps);
    sm.abort = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // everything above touches only this CTA's shared memory and TMEM; the expert offsets and the operands may
  // come from the kernel before
  pdl_wait();
  if (tid == 0) {
    if (blockIdx.x == 0) P.st->tile_ctr[P.ctr_idx ^ 1] = 0u;  // for the next GEMM of the chain (it starts after this one ends)
    int run = 0;
    for (int i = 0; i < P.E; ++i) {
      sm.tile_prefix[i] = run;
      const int rows = P.offsets[i + 1] - P.offsets[i];
      run += rows > 0 ? (rows + P.tile_rows - 1) / P.tile_rows : 0;
    }
    sm.tile_prefix[P.E] = run;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  Tile t;

  if (warp == 0) {
    // ================================================================= TMA producer
    if (lane == 0) {
      int it = 0;  // k-blocks issued so far, over all tiles
      bool ok = true;
      // Tiles are drawn from a counter in global memory (the CTAs' tiles differ in cost: one or two halves, operands
      // found in L2 or not) and passed on to the MMA thread and the epilogue warps through a small queue.
      for (int ti = 0; ok; ++ti) {
        const int qs = ti % kTileQueue;
        if (ti >= kTileQueue && !mbar_wait(&sm.tq_empty[qs], ((ti / kTileQueue) - 1) & 1)) {
          flag_error(P.st, MOE_ERR_TIMEOUT, 0x404u);
          sm.abort = 1;
          ok = false;
          break;
        }
        const int idx = (int)atomicAdd(&P.st->tile_ctr[P.ctr_idx], 1u);
        sm.tq[qs] = idx;
        mbar_arrive(&sm.tq_full[qs]);
        if (!decode_tile(P, sm, idx, n_tiles, t)) break;  // past the last tile: the others stop on it too
        const uint32_t tx = a_bytes * (P.dual_a ? 2 : t.halves) +
                            (P.pair ? 2u * 128u * kBK * 2u : (uint32_t)P.bn * kBK * 2u);
        const int kb0 = t.ks * num_kb / P.ksplit, kb1 = (t.ks + 1) * num_kb / P.ksplit;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % NS;
          if (it >= NS && !mbar_wait(&sm.empty[s], ((it / NS) - 1) & 1)) {
            flag_error(P.st, MOE_ERR_TIMEOUT, 0x400u);
            sm.abort = 1;
            ok = false;
            break;
          }
          unsigned char* st_a0 = stages + (size_t)s * stage_bytes;
          unsigned char* st_a1 = st_a0 + a_bytes;
          unsigned char* st_b = st_a0 + n_a * a_bytes;
          const int k0 = kb * kBK;
          const int kB = P.k_wrap > 0 ? k0 % P.k_wrap : k0;
          mbar_arrive_expect_tx(&sm.full[s], tx);
          tma_load_2d(st_a0, &map_a0, k0, t.m0, &sm.full[s]);
          if (P.dual_a)
            tma_load_2d(st_a1, &map_a1, k0, t.m0, &sm.full[s]);
          else if (t.halves == 2)
            tma_load_2d(st_a1, &map_a0, k0, t.m0 + kBM, &sm.full[s]);
          if (P.b_nmajor) {
            for (int j = 0; j < P.bn / 64; ++j)
              tma_load_4d(st_b + (size_t)j * 64 * kBK * 2, &map_b, t.n0 + 64 * j, P.b_sub, kB, t.e, &sm.full[s]);
          } else if (P.pair) {
            tma_load_4d(st_b, &map_b, kB, 0, t.n0, t.e, &sm.full[s]);
            tma_load_4d(st_b + 128 * kBK * 2, &map_b, kB, 1, t.n0, t.e, &sm.full[s]);
          } else {
            tma_load_4d(st_b, &map_b, kB, P.b_sub, t.n0, t.e, &sm.full[s]);
          }
        }
      }
      if (!ok) {  // copies in flight must land before the CTA goes away
        for (int j = max(0, it - NS); j < it; ++j) (void)mbar_wait(&sm.full[j % NS], (j / NS) & 1);
      }
    }
  } else if (warp == 1) {
    // ================================================================= MMA issuer
    if (lane == 0) {
      const uint32_t idesc_pairhalf = instr_desc(128, false);
      const uint32_t idesc_single = instr_desc(P.pair ? 256 : P.bn, P.b_nmajor != 0);
      int it = 0, tile_i = 0;
      bool ok = true;
      for (;; ++tile_i) {
        const int qs = tile_i % kTileQueue;
        if (!ok) break;
        if (!mbar_wait(&sm.tq_full[qs], (tile_i / kTileQueue) & 1)) {
          flag_error(P.st, MOE_ERR_TIMEOUT, 0x405u);
          sm.abort = 1;
          break;
        }
        const int idx = sm.tq[qs];
        mbar_arrive(&sm.tq_empty[qs]);
        if (!decode_tile(P, sm, idx, n_tiles, t)) break;
        if (tile_i > 0) {  // the previous tile's accumulators must have left TMEM
          if (!mbar_wait(&sm.accum_empty, (tile_i - 1) & 1)) {
            flag_error(P.st, MOE_ERR_TIMEOUT, 0x403u);
            sm.abort = 1;
            ok = false;
            break;
          }
          tc_fence_after();
        }
        const int kb0 = t.ks * num_kb / P.ksplit, kb1 = (t.ks + 1) * num_kb / P.ksplit;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % NS;
          if (!mbar_wait(&sm.full[s], (it / NS) & 1)) {
            flag_error(P.st, MOE_ERR_TIMEOUT, 0x401u);
            sm.abort = 1;
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t a0 = smem_u32(stages + (size_t)s * stage_bytes);
          const uint32_t a1 = a0 + a_bytes;
          const uint32_t b = a0 + n_a * a_bytes;
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk) {
            const bool acc = (kb > kb0) || (kk > 0);
            const uint64_t da0 = smem_desc(a0 + kk * 32, 16, 1024);
            if (P.b_nmajor) {
              const uint64_t db = smem_desc(b + kk * 2048, 64 * kBK * 2, 1024);
              tc_mma_bf16(tmem, da0, db, idesc_single, acc);
              if (t.halves == 2) tc_mma_bf16(tmem + 256, smem_desc(a1 + kk * 32, 16, 1024), db, idesc_single, acc);
            } else if (P.dual_a) {
              const uint64_t da1 = smem_desc(a1 + kk * 32, 16, 1024);
              const uint64_t db0 = smem_desc(b + kk * 32, 16, 1024);
              const uint64_t db1 = smem_desc(b + 128 * kBK * 2 + kk * 32, 16, 1024);
              tc_mma_bf16(tmem, da0, db0, idesc_pairhalf, acc);
              tc_mma_bf16(tmem + 128, da1, db1, idesc_pairhalf, acc);
            } else {
              const uint64_t db = smem_desc(b + kk * 32, 16, 1024);
              tc_mma_bf16(tmem, da0, db, idesc_single, acc);
              if (t.halves == 2) tc_mma_bf16(tmem + 256, smem_desc(a1 + kk * 32, 16, 1024), db, idesc_single, acc);
            }
          }
          tc_commit(&sm.empty[s]);  // arrives when the MMAs above have finished reading this stage
        }
        if (ok) tc_commit(&sm.accum_full);
      }
    }
  } else {
    // ================================================================= epilogue (warps 2..9)
    const int q = warp & 3;  // TMEM lanes 32q .. 32q+31 are the only ones this warp may read
    const int cpar = (warp - 2) >> 2;  // which of the two warps of this quarter: it takes every other 32-column chunk
    int tile_i = 0;
    for (;; ++tile_i) {
      const int qs = tile_i % kTileQueue;
      if (!mbar_wait(&sm.tq_full[qs], (tile_i / kTileQueue) & 1)) {
        if (lane == 0) flag_error(P.st, MOE_ERR_TIMEOUT, 0x406u);
        break;
      }
      const int idx = sm.tq[qs];
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.tq_empty[qs]);
      if (!decode_tile(P, sm, idx, n_tiles, t)) break;
      if (!mbar_wait(&sm.accum_full, tile_i & 1)) {
        if (lane == 0) flag_error(P.st, MOE_ERR_TIMEOUT, 0x402u);
        break;
      }
      tc_fence_after();
      const int ncols = min(P.bn, P.n_total - t.n0);  // valid columns of this tile (multiple of 8)
      for (int hf = 0; hf < t.halves; ++hf) {
        const int row = t.m0 + hf * kBM + 32 * q + lane;
        const bool row_ok = row < t.m_end;
        const uint32_t tbase = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(hf * 256);
        if (P.epi == EPI_SWIGLU || P.epi == EPI_BF16_PAIR) {
          __nv_bfloat16* out = (__nv_bfloat16*)P.out + (size_t)row * P.ld_out + t.n0;
          for (int c = 32 * cpar; c < P.bn; c += 64) {
            uint32_t g[32], u[32];
            tc_ld32(tbase + c, g);
            tc_ld32(tbase + 128 + c, u);
            tc_wait_ld();
            if (!row_ok) continue;
            if (P.epi == EPI_SWIGLU) {
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                if (c + 8 * v < ncols) {
                  uint32_t o[4];
#pragma unroll
                  for (int j = 0; j < 4; ++j)
                    o[j] = pack_bf16x2(
                        silu_mul(__uint_as_float(g[8 * v + 2 * j]), __uint_as_float(u[8 * v + 2 * j])),
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
      }
      // the accumulators are in registers / memory now: hand TMEM back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.accum_empty);
    }
  }
  // ---- teardown: every role gets here in bounded time
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
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

int launch_gg(moe_ctx* ctx, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b, GGParams P,
              int n_slots, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  P.E = c.n_experts;
  P.st = ctx->d_state;
  const int n_tiles = (P.n_total + P.bn - 1) / P.bn;
  // 256-row tiles read every B slice once for up to 256 rows of an expert (half the operand traffic per flop,
  // and an expert with 129..256 rows is one tile instead of two); problems whose 256-row tiles would leave SMs
  // without work keep 128-row tiles.  A cut contraction (ksplit) multiplies the work items.
  P.tile_rows = kBM;
  if (P.ksplit < 1) P.ksplit = 1;
  const long long m256 = std::max<long long>((n_slots + kTileRows - 1) / kTileRows, std::min(c.n_experts, n_slots));
  if (!P.dual_a && (m256 * n_tiles >= ctx->sm_count || P.ksplit > 1)) P.tile_rows = kTileRows;
  P.single_a = (P.tile_rows == kBM && !P.dual_a) ? 1 : 0;
  P.n_stages = P.single_a ? 4 : 3;
  const size_t stage_bytes = (size_t)kBM * kBK * 2 * (P.single_a ? 1 : 2) + 256 * kBK * 2;
  const size_t smem = P.n_stages * stage_bytes + sizeof(SmemGG) + 1024 + 128;
  if ((long long)smem > ctx->max_smem_optin) return MOE_ERR_UNSUPPORTED;
  const long long m_tiles = (n_slots + P.tile_rows - 1) / P.tile_rows + c.n_experts;  // upper bound
  const int grid = (int)std::min<long long>(m_tiles * n_tiles * P.ksplit, ctx->sm_count);
  MOE_CUDA_TRY(cudaFuncSetAttribute(grouped_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  MOE_CUDA_TRY(launch_pdl(grouped_gemm_kernel, dim3(grid), dim3(kThreadsGG), smem, s, a0, a1, b, P));
  MOE_CUDA_TRY(cudaGetLastError());
  ctx->launches++;
  return MOE_OK;
}

int pick_bn(int n_total, int cap) {
  int bn = cap;
  while (bn > 64 && bn / 2 >= n_total) bn /= 2;
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
    // (1) hidden = silu(X Wg) * (X Wu)
    if ((rc = make_map_a(&ma, xperm, n_slots, d, d)) != MOE_OK) return rc;
    if ((rc = make_map_b(&mb, w->gud, d, 3, f, E, kBK, 128)) != MOE_OK) return rc;
    P.K = d, P.n_total = f, P.bn = 128, P.pair = 1, P.dual_a = 0, P.b_nmajor = 0, P.b_sub = 0, P.epi = EPI_SWIGLU;
    P.out = hidden, P.ld_out = f, P.out_off2 = 0;
    P.ctr_idx = 0;
    if ((rc = launch_gg(ctx, ma, ma, mb, P, n_slots, s)) != MOE_OK) return rc;
    // (2) out_slots = hidden Wd   (B = down rows of gud: [k = hidden unit][n = model column], n contiguous)
    if ((rc = make_map_a(&ma, hidden, n_slots, f, f)) != MOE_OK) return rc;
    if ((rc = make_map_b(&mb, w->gud, d, 3, f, E, 64, kBK)) != MOE_OK) return rc;
    P.K = f, P.n_total = d, P.bn = pick_bn(d, 256), P.pair = 0, P.dual_a = 0, P.b_nmajor = 1, P.b_sub = 2;
    P.epi = EPI_F32, P.out = out_slots, P.ld_out = d, P.out_off2 = 0;
    if (out_planes && n_slots <= kKSplitMaxSlots) {
      // short prefill: too few tiles for the SMs, and every tile streams a long run of weights.  The caller
      // sums planes: cut the contraction so that every SM streams a part, each part into its own plane.
      const int m_est = std::max((n_slots + kBM - 1) / kBM, std::min(E, n_slots));
      const long long tiles = (long long)m_est * ((d + P.bn - 1) / P.bn);
      int ks = (int)(ctx->sm_count / std::max<long long>(tiles, 1));
      ks = std::min(std::min(ks, kKSplitMax), (f + kBK - 1) / kBK);
      if (ks > 1) {
        P.ksplit = ks, P.plane_elems = (long long)n_slots * d;
        *out_planes = ks;
      }
    }
    P.ctr_idx = 1;
    return launch_gg(ctx, ma, ma, mb, P, n_slots, s);
  }
  // The rank-r intermediates t and v are kept as hi + lo pairs of bf16 (value = hi + lo): the GEMMs that
  // consume them run over K = 2r with the weight slices repeated, so the intermediates carry ~16 mantissa
  // bits and the chain's only bf16 roundings are those of the dense path (hidden activations, output).
  const bool split = (r % kBK) == 0;
  const int tw = split ? 2 * r : r;  // stored width of one intermediate
  void* mid_a = ws + L.mid_a;  // [n_slots][2*tw]: t_g (hi | lo) | t_u (hi | lo)
  void* mid_b = ws + L.mid_b;  // [n_slots][tw]:   v (hi | lo)
  // (1) T = X [gL | uL]
  if ((rc = make_map_a(&ma, xperm, n_slots, d, d)) != MOE_OK) return rc;
  if ((rc = make_map_b(&mb, w->wd_a, d, 2, r, E, kBK, 128)) != MOE_OK) return rc;
  P.K = d, P.n_total = r, P.bn = 128, P.pair = 1, P.dual_a = 0, P.b_nmajor = 0, P.b_sub = 0, P.epi = EPI_BF16_PAIR;
  P.k_wrap = 0, P.split = split, P.out = mid_a, P.ld_out = 2 * tw, P.out_off2 = tw, P.out_off_lo = r;
  P.ctr_idx = 0;
  if ((rc = launch_gg(ctx, ma, ma, mb, P, n_slots, s)) != MOE_OK) return rc;
  // (2) hidden = silu(Tg gR) * (Tu uR)
  if ((rc = make_map_a(&ma, mid_a, n_slots, tw, 2 * tw)) != MOE_OK) return rc;
  if ((rc = make_map_a(&ma1, (const __nv_bfloat16*)mid_a + tw, n_slots, tw, 2 * tw)) != MOE_OK) return rc;
  if ((rc = make_map_b(&mb, w->wd_b, r, 2, f, E, kBK, 128)) != MOE_OK) return rc;
  P.K = tw, P.n_total = f, P.bn = 128, P.pair = 1, P.dual_a = 1, P.b_nmajor = 0, P.b_sub = 0, P.epi = EPI_SWIGLU;
  P.k_wrap = split ? r : 0, P.split = 0, P.out = hidden, P.ld_out = f, P.out_off2 = 0, P.out_off_lo = 0;
  P.ctr_idx = 1;
  if ((rc = launch_gg(ctx, ma, ma1, mb, P, n_slots, s)) != MOE_OK) return rc;
  // (3) V = hidden dL
  if ((rc = make_map_a(&ma, hidden, n_slots, f, f)) != MOE_OK) return rc;
  P.bn = pick_bn(r, 256);
  if ((rc = make_map_b(&mb, w->wd_c, f, 1, r, E, kBK, P.bn)) != MOE_OK) return rc;
  P.K = f, P.n_total = r, P.pair = 0, P.dual_a = 0, P.b_nmajor = 0, P.b_sub = 0, P.epi = EPI_BF16;
  P.k_wrap = 0, P.split = split, P.out = mid_b, P.ld_out = tw, P.out_off2 = 0, P.out_off_lo = r;
  P.ctr_idx = 0;
  if ((rc = launch_gg(ctx, ma, ma, mb, P, n_slots, s)) != MOE_OK) return rc;
  // (4) out_slots = V dR
  if ((rc = make_map_a(&ma, mid_b, n_slots, tw, tw)) != MOE_OK) return rc;
  P.bn = pick_bn(d, 256);
  if ((rc = make_map_b(&mb, w->wd_d, r, 1, d, E, kBK, P.bn)) != MOE_OK) return rc;
  P.K = tw, P.n_total = d, P.pair = 0, P.dual_a = 0, P.b_nmajor = 0, P.b_sub = 0, P.epi = EPI_F32;
  P.k_wrap = split ? r : 0, P.split = 0, P.out = out_slots, P.ld_out = d, P.out_off2 = 0, P.out_off_lo = 0;
  P.ctr_idx = 1;
  return launch_gg(ctx, ma, ma, mb, P, n_slots, s);
}

}  // namespace cosmoe
