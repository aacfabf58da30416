// Batch-1 decode of a layer with weight-decomposed experts (Eq. 1): ONE launch, no cooperative grid.
//
// Every expert matrix is a product L R, applied as (x L) R, so the layer is a chain of four matrix-vector
// products per selected expert, each needing the whole result of the one before:
//
//   t = x [gL | uL]   (2r values)      wd_a [S][r][2][d]   row (j, gate|up) . x
//   h_c = silu(t_g . gR_c) * (t_u . uR_c)   (f values)   wd_b [S][f][2][r]
//   v = h dL          (r values)       wd_c [S][r][f]      row j . h
//   y = sum_a w_a (v_a dR_a)  (d values)   wd_d [S][d][r]  row i . v
//
// The weights are few (6 r (d + f) bytes per expert), so what counts is the latency of the chain.  Every
// product is "one warp per output row, lanes along the row": each output is the work of one warp, written with a
// plain store -- no atomics, no finalisation, bit-identical from call to call.  The router (Eq. 2, Eq. 3) runs in
// every CTA's prologue.  Between the products the CTAs meet at an arrival counter in global memory that runs
// over launches (each meeting is the next gridDim.x arrivals), with a bounded wait: the grid is one CTA of 256
// threads per SM, so all of it is resident as soon as a predecessor has drained.
// Short rows (v = h dL has only k r of them) are cut into up to 8 segments whose partial sums are added, in
// order, by the reader.
#include "common.cuh"

namespace cosmoe {

namespace {

constexpr int kWdWarps = 8;
constexpr int kWdThreads = kWdWarps * 32;
constexpr int kWdMaxD = 2048;     // x as fp32 in shared memory
constexpr int kWdMaxKR = 2048;    // top_k * r: t and v in shared memory
constexpr int kWdMaxSplit = 8;

struct WdParams {
  int k, E, d, f, r, x_is_bf16, renorm;
  const void* x;
  const uint16_t* w_router;
  const float* b_router;
  const int32_t* expert_slot;
  const uint16_t *wd_a, *wd_b, *wd_c, *wd_d;
  int32_t* topk_idx;
  float* topk_w;
  float *t, *h, *vpart;  // scratch: [k][2r], [k][f], [k][r][split]
  void* y;
  DeviceState* st;
  int split;  // segments per row of the third product
};

struct WdSmem {
  __align__(16) float x[kWdMaxD];   // (16-byte aligned: read as float4)
  __align__(16) float tg[kWdMaxKR];  // t de-interleaved; later v in tg
  __align__(16) float tu[kWdMaxKR];
  float rlog[kWdWarps][MOE_MAX_EXPERTS];
  int sel_e[MOE_MAX_TOPK];
  int sel_slot[MOE_MAX_TOPK];
  float sel_w[MOE_MAX_TOPK];
  int ok;
};

// All CTAs have passed their previous product.  Returns false (for the whole CTA) when the wait ran out.
__device__ __forceinline__ bool meet(DeviceState* st, WdSmem& sm) {
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned G = gridDim.x;
    // (the arrival is a release at GPU scope and the barrier above orders the CTA's stores before it; the wait
    // reads the counter with acquire loads: no separate fences)
    const unsigned long long old = atom_add_acq_rel64(&st->phase_total, 1ull);
    const unsigned long long target = old - old % G + G;
    int ok = 1;
    const long long t0 = clock64();
    while (ld_acquire64(&st->phase_total) < target) {
      if (clock64() - t0 > kWaitBudgetCycles) {
        flag_error(st, MOE_ERR_TIMEOUT, 0x500u);
        ok = 0;
        break;
      }
    }
    sm.ok = ok;
  }
  __syncthreads();
  return sm.ok != 0;
}

// dot of 8 bf16 weights with 8 fp32 values fetched from a 16-byte aligned place in shared memory as two float4
__device__ __forceinline__ float dot8s(const uint4& w, const float* v) {
  const float4 a = reinterpret_cast<const float4*>(v)[0], b = reinterpret_cast<const float4*>(v)[1];
  float f[8];
  unpack8(w, f);
  float acc = f[0] * a.x;
  acc = fmaf(f[1], a.y, acc), acc = fmaf(f[2], a.z, acc), acc = fmaf(f[3], a.w, acc);
  acc = fmaf(f[4], b.x, acc), acc = fmaf(f[5], b.y, acc), acc = fmaf(f[6], b.z, acc), acc = fmaf(f[7], b.w, acc);
  return acc;
}
// dot of 8 bf16 weights with 8 fp32 values (registers)
__device__ __forceinline__ float dot8f(const uint4& w, const float* v) {
  float f[8];
  unpack8(w, f);
  float a = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) a = fmaf(f[i], v[i], a);
  return a;
}

__global__ void __launch_bounds__(kWdThreads) wd_decode_kernel(const WdParams P) {
  extern __shared__ __align__(16) unsigned char wd_smem_raw[];
  WdSmem& sm = *reinterpret_cast<WdSmem*>(wd_smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = P.d, f = P.f, r = P.r, k = P.k, E = P.E;
  const int gw = blockIdx.x * kWdWarps + warp, n_warps = gridDim.x * kWdWarps;
  DeviceState* const st = P.st;
  pdl_launch_dependents();
  // the router's weights do not depend on any earlier kernel: this thread's rows (first eight experts) are fetched
  // before the dependency wait, not after the token row behind it
  uint4 wr0[kWdMaxD / kWdThreads];
  if ((E & 7) == 0) {
#pragma unroll
    for (int q = 0; q < kWdMaxD / kWdThreads; ++q)
      wr0[q] = __ldg(reinterpret_cast<const uint4*>(P.w_router + (size_t)min(tid + q * kWdThreads, d - 1) * E));
  }
  pdl_wait();

  // ---------------------------------------------------------------- token row, router (every CTA)
  for (int i = tid; i < d; i += kWdThreads)
    sm.x[i] = P.x_is_bf16 ? bf16_to_float(((const uint16_t*)P.x)[i]) : ((const float*)P.x)[i];
  __syncthreads();
  for (int e0 = 0; e0 < E; e0 += 8) {
    float a[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) a[j] = 0.f;
    if ((E & 7) == 0) {
      uint4 wr[kWdMaxD / kWdThreads];  // this thread's router rows, fetched in one round trip
#pragma unroll
      for (int q = 0; q < kWdMaxD / kWdThreads; ++q)
        wr[q] = e0 == 0 ? wr0[q]
                        : __ldg(reinterpret_cast<const uint4*>(P.w_router + (size_t)min(tid + q * kWdThreads, d - 1) * E + e0));
#pragma unroll
      for (int q = 0; q < kWdMaxD / kWdThreads; ++q) {
        const int i = tid + q * kWdThreads;
        float w[8];
        unpack8(wr[q], w);
        const float xv = i < d ? sm.x[i] : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) a[j] = fmaf(xv, w[j], a[j]);
      }
    } else {
      for (int i = tid; i < d; i += kWdThreads)
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (e0 + j < E) a[j] = fmaf(sm.x[i], bf16_to_float(__ldg(P.w_router + (size_t)i * E + e0 + j)), a[j]);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float v = warp_sum(a[j]);
      if (lane == 0 && e0 + j < E) sm.rlog[warp][e0 + j] = v;
    }
  }
  __syncthreads();
  if (warp == 0) {
    float l0 = 0.f, l1 = 0.f;
    if (lane < E) {
      for (int w = 0; w < kWdWarps; ++w) l0 += sm.rlog[w][lane];
      if (P.b_router) l0 += P.b_router[lane];
    }
    if (lane + 32 < E) {
      for (int w = 0; w < kWdWarps; ++w) l1 += sm.rlog[w][lane + 32];
      if (P.b_router) l1 += P.b_router[lane + 32];
    }
    warp_route_finish(l0, l1, E, k, P.renorm, lane, sm.sel_e, sm.sel_w, nullptr);
    __syncwarp();
    if (lane < k) {
      const int e = sm.sel_e[lane];
      const int sl = P.expert_slot ? P.expert_slot[e] : e;
      if (sl < 0) flag_error(st, MOE_ERR_STATE, 0x501u);
      sm.sel_slot[lane] = sl < 0 ? 0 : sl;
      if (blockIdx.x == 0) {
        if (P.topk_idx) P.topk_idx[lane] = e;
        if (P.topk_w) P.topk_w[lane] = sm.sel_w[lane];
      }
    }
  }
  __syncthreads();

  const int dc = d >> 3, rc = r >> 3, fc = f >> 3;

  // The selected experts' matrices are known now: every CTA asks for its share of all four to be brought into
  // L2 (fire and forget), in the order the chain needs them, so that the DRAM transfer runs in the background
  // of the chain instead of once per product behind a meeting.
  if (tid < 4 * k) {
    const int which = tid / k, a = tid - which * k;  // which-major: all experts' wd_a first
    const size_t per_expert[4] = {(size_t)2 * r * d * 2, (size_t)f * 2 * r * 2, (size_t)r * f * 2, (size_t)d * r * 2};
    const uint16_t* const base[4] = {P.wd_a, P.wd_b, P.wd_c, P.wd_d};
    const size_t bytes = per_expert[which];
    const size_t slice = ((bytes + gridDim.x - 1) / gridDim.x + 15) & ~(size_t)15;
    const size_t lo = (size_t)blockIdx.x * slice;
    if (lo < bytes) {
      const size_t n = bytes - lo < slice ? bytes - lo : slice;  // a multiple of 16: bytes is
      const unsigned char* src = reinterpret_cast<const unsigned char*>(base[which]) + (size_t)sm.sel_slot[a] * bytes + lo;
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"((uint32_t)n) : "memory");
    }
  }

  // ---------------------------------------------------------------- t = x [gL | uL]: k * 2r rows of d
  for (int row = gw; row < k * 2 * r; row += n_warps) {
    const int a = row / (2 * r), j2 = row - a * 2 * r;
    const uint4* wrow = reinterpret_cast<const uint4*>(P.wd_a + ((size_t)sm.sel_slot[a] * 2 * r + j2) * d);
    float acc = 0.f;
    for (int c0 = lane; c0 < dc; c0 += 32 * 4) {
      uint4 w[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) w[u] = __ldg(wrow + min(c0 + 32 * u, dc - 1));
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + 32 * u < dc) acc += dot8s(w[u], sm.x + (c0 + 32 * u) * 8);
    }
    acc = warp_sum(acc);
    if (lane == 0) P.t[row] = acc;
  }
  if (!meet(st, sm)) return;
  for (int i = tid; i < k * 2 * r; i += kWdThreads) {  // t[a][j][gate|up] -> tg[a][j], tu[a][j]
    const float v = __ldcg(P.t + i);
    const int a = i / (2 * r), j2 = i - a * 2 * r;
    ((j2 & 1) ? sm.tu : sm.tg)[a * r + (j2 >> 1)] = v;
  }
  __syncthreads();

  // ---------------------------------------------------------------- h_c: k * f units, rows (gR_c | uR_c) of 2r
  for (int u0 = gw; u0 < k * f; u0 += 4 * n_warps) {
    float g[4], up[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) g[q] = up[q] = 0.f;
    for (int c0 = lane; c0 < 2 * rc; c0 += 32) {
      const int part = c0 >= rc ? 1 : 0, cc = c0 - part * rc;
      uint4 w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int u = min(u0 + q * n_warps, k * f - 1);
        const int a = u / f, c = u - a * f;
        w[q] = __ldg(reinterpret_cast<const uint4*>(P.wd_b + ((size_t)sm.sel_slot[a] * f + c) * 2 * r) + c0);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int u = min(u0 + q * n_warps, k * f - 1);
        const int a = u / f;
        const float v = dot8s(w[q], (part ? sm.tu : sm.tg) + a * r + cc * 8);
        if (part) up[q] += v; else g[q] += v;
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float gs = warp_sum(g[q]), us = warp_sum(up[q]);
      const int u = u0 + q * n_warps;
      if (lane == 0 && u < k * f) P.h[u] = __fdividef(gs, 1.0f + __expf(-gs)) * us;
    }
  }
  if (!meet(st, sm)) return;

  // ---------------------------------------------------------------- v = h dL: k * r rows of f, in `split` segments
  {
    const int S = P.split, seg = ((fc + S - 1) / S);  // chunks per segment
    for (int item = gw; item < k * r * S; item += n_warps) {
      const int row = item / S, s = item - row * S;
      const int a = row / r, j = row - a * r;
      const uint4* wrow = reinterpret_cast<const uint4*>(P.wd_c + ((size_t)sm.sel_slot[a] * r + j) * f);
      const float* hv = P.h + (size_t)a * f;
      const int c_lo = s * seg, c_hi = min(fc, c_lo + seg);
      float acc = 0.f;
      for (int c0 = c_lo + lane; c0 < c_hi; c0 += 32 * 4) {
        uint4 w[4];
        float4 ha[4], hb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c = min(c0 + 32 * u, c_hi - 1);
          w[u] = __ldg(wrow + c);
          ha[u] = __ldcg(reinterpret_cast<const float4*>(hv) + 2 * c);
          hb[u] = __ldcg(reinterpret_cast<const float4*>(hv) + 2 * c + 1);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (c0 + 32 * u < c_hi) {
            const float hh[8] = {ha[u].x, ha[u].y, ha[u].z, ha[u].w, hb[u].x, hb[u].y, hb[u].z, hb[u].w};
            acc += dot8f(w[u], hh);
          }
        }
      }
      acc = warp_sum(acc);
      if (lane == 0) P.vpart[item] = acc;
    }
  }
  if (!meet(st, sm)) return;
  for (int i = tid; i < k * r; i += kWdThreads) {  // v[a][j] = its segments, in order
    float v = 0.f;
    for (int s = 0; s < P.split; ++s) v += __ldcg(P.vpart + (size_t)i * P.split + s);
    sm.tg[i] = v;
  }
  __syncthreads();

  // ---------------------------------------------------------------- y_i = sum_a w_a (v_a . dR_a[i]): d outputs
  const bool good = ld_acquire(&st->status) == 0u;
  for (int i = gw; i < d; i += n_warps) {
    float acc = 0.f;
    for (int q = lane; q < k * rc; q += 32) {
      const int a = q / rc, c = q - a * rc;
      const uint4 w = __ldg(reinterpret_cast<const uint4*>(P.wd_d + ((size_t)sm.sel_slot[a] * d + i) * r) + c);
      acc = fmaf(sm.sel_w[a], dot8s(w, sm.tg + a * r + c * 8), acc);
    }
    acc = warp_sum(acc);
    if (lane == 0 && good) {
      if (P.x_is_bf16)
        ((__nv_bfloat16*)P.y)[i] = __float2bfloat16_rn(acc);
      else
        ((float*)P.y)[i] = acc;
    }
  }
}


// =====================================================================================================
// The same chain for LARGE factors (tens of MB per token: the paper's rank, r = d / 2): bandwidth counts, so the
// weights go through a ring of shared-memory stages filled by bulk asynchronous copies, as in the dense
// streaming kernel, and only the meetings between the products remain of the grid-wide dependencies.
//   producer thread   walks the four products in order and brings this CTA's rows, a stage (<= 32 KB) at a
//                     time; the weights do not depend on the chain's values, so it runs ahead across the
//                     meetings as far as the ring allows and the DRAM latency of a product's first rows hides
//                     behind the meeting before it;
//   8 consumer warps  one output row per warp and stage (products 1, 2, 4: the input vector, at most 64 values per
//                     lane, sits in registers) or a quarter of a row (product 3, rows of f values: input in
//                     shared memory, four partial sums per row that the reader adds in order).
// Every value has one writer and a fixed summation order: results are bit-identical from call to call.
// =====================================================================================================
constexpr int kWsStages = 4;
constexpr int kWsStageBytes = 32768;
constexpr int kWsRows = 8;        // rows (outputs) per stage in products 1, 2 and 4
constexpr int kWsRowsC = 2;       // rows per stage in product 3
constexpr int kWsSeg = 4;         // partial sums per row of product 3
constexpr int kWsThreads = (kWdWarps + 1) * 32;
constexpr int kWsIn = 8;          // 16-byte chunks of the input vector per lane (registers)

struct WsSmem {
  uint64_t full[kWsStages], freeb[kWsStages];
  uint64_t cbar;  // barrier over the consumer warps
  __align__(16) float x[kWdMaxD];  // (16-byte aligned: the lanes fetch their slices of these vectors as float4)
  __align__(16) float tg[kWdMaxKR];
  __align__(16) float tu[kWdMaxKR];
  float rlog[kWdWarps][MOE_MAX_EXPERTS];
  int sel_e[MOE_MAX_TOPK];
  int sel_slot[MOE_MAX_TOPK];
  float sel_w[MOE_MAX_TOPK];
  int ok;
  volatile int abort;
};
constexpr int kWsHeader = (sizeof(WsSmem) + 127) / 128 * 128;

// Rows of product `ph` per expert, and this CTA's share [g0, g1) of all k * N of them (product 4: of the d outputs).
__device__ __forceinline__ int ws_rows(const WdParams& P, int ph) { return ph == 0 ? 2 * P.r : (ph == 1 ? P.f : (ph == 2 ? P.r : P.d)); }
__device__ __forceinline__ void ws_share(const WdParams& P, int ph, int& g0, int& g1) {
  const long long tot = ph == 3 ? P.d : (long long)P.k * ws_rows(P, ph);
  g0 = (int)(tot * blockIdx.x / gridDim.x);
  g1 = (int)(tot * (blockIdx.x + 1) / gridDim.x);
}

// Barrier over the consumer warps (the producer warp does not take part) with a bounded wait: an mbarrier, not
// bar.sync, so that a warp that gave up on an expired wait elsewhere cannot leave the others parked for ever.
__device__ __forceinline__ bool ws_sync(WsSmem& sm, unsigned& par) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(&sm.cbar);
  const bool ok = mbar_wait_spin(&sm.cbar, par);
  par ^= 1u;
  return ok;
}
// All CTAs have finished the product before.  False (for the whole CTA) when a wait ran out.
__device__ __forceinline__ bool ws_meet(DeviceState* st, WsSmem& sm, unsigned& par) {
  if (!ws_sync(sm, par)) return false;
  if (threadIdx.x == 0) {
    const unsigned G = gridDim.x;
    const unsigned long long old = atom_add_acq_rel64(&st->phase_total, 1ull);
    const unsigned long long target = old - old % G + G;
    int ok = 1;
    const long long t0 = clock64();
    while (ld_acquire64(&st->phase_total) < target) {
      if (clock64() - t0 > kWaitBudgetCycles || sm.abort) {
        flag_error(st, MOE_ERR_TIMEOUT, 0x510u);
        ok = 0;
        break;
      }
    }
    sm.ok = ok;
  }
  return ws_sync(sm, par) && sm.ok != 0;
}

// eight consecutive fp32 values of a 16-byte aligned vector
__device__ __forceinline__ void load8f(const float* src, float* dst) {
  const float4 a = reinterpret_cast<const float4*>(src)[0], b = reinterpret_cast<const float4*>(src)[1];
  dst[0] = a.x, dst[1] = a.y, dst[2] = a.z, dst[3] = a.w, dst[4] = b.x, dst[5] = b.y, dst[6] = b.z, dst[7] = b.w;
}
__device__ __forceinline__ void zero8f(float* dst) {
#pragma unroll
  for (int q = 0; q < 8; ++q) dst[q] = 0.f;
}

__global__ void __launch_bounds__(kWsThreads, 1) wd_stream_kernel(const WdParams P) {
  extern __shared__ __align__(128) unsigned char ws_smem_raw[];
  WsSmem& sm = *reinterpret_cast<WsSmem*>(ws_smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = P.d, f = P.f, r = P.r, k = P.k, E = P.E;
  float* const hs = reinterpret_cast<float*>(ws_smem_raw + kWsHeader);  // h of the selected experts, [k][f]
  unsigned char* const ring = ws_smem_raw + kWsHeader + (((size_t)k * f * 4 + 127) / 128) * 128;
  DeviceState* const st = P.st;
  pdl_launch_dependents();
  if (tid == kWdThreads) {
    for (int i = 0; i < kWsStages; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.freeb[i], kWdWarps);
    }
    mbar_init(&sm.cbar, kWdWarps);
    fence_mbar_init();
    fence_proxy_async_smem();
    sm.abort = 0;
  }
  uint4 wr0[kWdMaxD / kWdThreads];  // this thread's router rows (first eight experts): constants, fetched before the wait
  if ((E & 7) == 0 && warp < kWdWarps) {
#pragma unroll
    for (int q = 0; q < kWdMaxD / kWdThreads; ++q)
      wr0[q] = __ldg(reinterpret_cast<const uint4*>(P.w_router + (size_t)min(tid + q * kWdThreads, d - 1) * E));
  }
  pdl_wait();

  // ---------------------------------------------------------------- token row, router (every CTA)
  if (warp < kWdWarps)
    for (int i = tid; i < d; i += kWdThreads)
      sm.x[i] = P.x_is_bf16 ? bf16_to_float(((const uint16_t*)P.x)[i]) : ((const float*)P.x)[i];
  __syncthreads();
  if (warp < kWdWarps) {
    for (int e0 = 0; e0 < E; e0 += 8) {
      float a[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) a[j] = 0.f;
      if ((E & 7) == 0) {
        uint4 wr[kWdMaxD / kWdThreads];
#pragma unroll
        for (int q = 0; q < kWdMaxD / kWdThreads; ++q)
          wr[q] = e0 == 0 ? wr0[q]
                          : __ldg(reinterpret_cast<const uint4*>(P.w_router + (size_t)min(tid + q * kWdThreads, d - 1) * E + e0));
#pragma unroll
        for (int q = 0; q < kWdMaxD / kWdThreads; ++q) {
          const int i = tid + q * kWdThreads;
          float w[8];
          unpack8(wr[q], w);
          const float xv = i < d ? sm.x[i] : 0.f;
#pragma unroll
          for (int j = 0; j < 8; ++j) a[j] = fmaf(xv, w[j], a[j]);
        }
      } else {
        for (int i = tid; i < d; i += kWdThreads)
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (e0 + j < E) a[j] = fmaf(sm.x[i], bf16_to_float(__ldg(P.w_router + (size_t)i * E + e0 + j)), a[j]);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float v = warp_sum(a[j]);
        if (lane == 0 && e0 + j < E) sm.rlog[warp][e0 + j] = v;
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    float l0 = 0.f, l1 = 0.f;
    if (lane < E) {
      for (int w = 0; w < kWdWarps; ++w) l0 += sm.rlog[w][lane];
      if (P.b_router) l0 += P.b_router[lane];
    }
    if (lane + 32 < E) {
      for (int w = 0; w < kWdWarps; ++w) l1 += sm.rlog[w][lane + 32];
      if (P.b_router) l1 += P.b_router[lane + 32];
    }
    warp_route_finish(l0, l1, E, k, P.renorm, lane, sm.sel_e, sm.sel_w, nullptr);
    __syncwarp();
    if (lane < k) {
      const int e = sm.sel_e[lane];
      const int sl = P.expert_slot ? P.expert_slot[e] : e;
      if (sl < 0) flag_error(st, MOE_ERR_STATE, 0x511u);
      sm.sel_slot[lane] = sl < 0 ? 0 : sl;
      if (blockIdx.x == 0) {
        if (P.topk_idx) P.topk_idx[lane] = e;
        if (P.topk_w) P.topk_w[lane] = sm.sel_w[lane];
      }
    }
  }
  __syncthreads();
  const int dc = d >> 3, rc = r >> 3, fc = f >> 3;

  if (warp == kWdWarps) {
    // ================================================================= producer
    if (lane != 0) return;
    const uint64_t pol = l2_policy_evict_first();
    int n = 0, slot = 0;
    unsigned par = 1;  // parity of the freeb phase the slot's next fill waits for
    bool ok = true;
    auto acquire = [&]() -> bool {
      if (n >= kWsStages && !mbar_wait(&sm.freeb[slot], par)) {
        flag_error(st, MOE_ERR_TIMEOUT, 0x512u);
        sm.abort = 1;
        return false;
      }
      if (sm.abort) return false;
      fence_proxy_async_smem();
      return true;
    };
    auto advance = [&]() {
      ++n;
      if (++slot == kWsStages) slot = 0, par ^= 1u;
    };
    for (int ph = 0; ph < 4 && ok; ++ph) {
      const int N = ws_rows(P, ph);
      int g0, g1;
      ws_share(P, ph, g0, g1);
      if (ph < 3) {
        const int RS = ph == 2 ? kWsRowsC : kWsRows;
        const size_t rowlen = ph == 0 ? (size_t)d : (ph == 1 ? (size_t)2 * r : (size_t)f);
        const uint16_t* base = ph == 0 ? P.wd_a : (ph == 1 ? P.wd_b : P.wd_c);
        for (int a = 0; a < k && ok; ++a) {
          const int lo = max(g0, a * N) - a * N, hi = min(g1, (a + 1) * N) - a * N;
          const uint16_t* src = base + ((size_t)sm.sel_slot[a] * N) * rowlen;
          for (int r0 = lo; r0 < hi; r0 += RS) {
            const int nr = min(RS, hi - r0);
            if (!(ok = acquire())) break;
            const uint32_t bytes = (uint32_t)(nr * rowlen * 2);
            mbar_arrive_expect_tx(&sm.full[slot], bytes);
            bulk_g2s_hint(ring + (size_t)slot * kWsStageBytes, src + (size_t)r0 * rowlen, bytes, &sm.full[slot], pol);
            advance();
          }
        }
      } else {
        for (int r0 = g0; r0 < g1 && ok; r0 += kWsRows) {
          const int nr = min(kWsRows, g1 - r0);
          if (!(ok = acquire())) break;
          const uint32_t bytes = (uint32_t)(nr * r * 2);
          mbar_arrive_expect_tx(&sm.full[slot], bytes * (uint32_t)k);
          for (int a = 0; a < k; ++a)
            bulk_g2s_hint(ring + (size_t)slot * kWsStageBytes + (size_t)a * kWsRows * r * 2,
                          P.wd_d + ((size_t)sm.sel_slot[a] * d + r0) * r, bytes, &sm.full[slot], pol);
          advance();
        }
      }
    }
    if (!ok)  // copies in flight must land before this CTA's shared memory goes away
      for (int j = max(0, n - kWsStages); j < n; ++j) (void)mbar_wait(&sm.full[j % kWsStages], (unsigned)(j / kWsStages) & 1u);
    return;
  }

  // ===================================================================== consumers
  int slot = 0;
  unsigned par = 0;
  auto wait_stage = [&]() -> bool {
    if (mbar_wait(&sm.full[slot], par)) return true;
    if (lane == 0) {
      flag_error(st, MOE_ERR_TIMEOUT, 0x513u);
      sm.abort = 1;
    }
    return false;
  };
  auto release_stage = [&]() {
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.freeb[slot]);
    if (++slot == kWsStages) slot = 0, par ^= 1u;
  };
  unsigned cpar = 0;
  float in[kWsIn][8];  // this lane's slice of the current product's input vector

  // ---------------------------------------------------------------- t = x [gL | uL]: rows (j, gate | up) of d
  {
#pragma unroll
    for (int j = 0; j < kWsIn; ++j) {
      const int c = lane + 32 * j;
      if (c < dc)
        load8f(sm.x + c * 8, in[j]);
      else
        zero8f(in[j]);
    }
    const int N = 2 * r;
    int g0, g1;
    ws_share(P, 0, g0, g1);
    for (int a = 0; a < k; ++a) {
      const int lo = max(g0, a * N) - a * N, hi = min(g1, (a + 1) * N) - a * N;
      for (int r0 = lo; r0 < hi; r0 += kWsRows) {
        const int nr = min(kWsRows, hi - r0);
        if (!wait_stage()) return;
        if (warp < nr) {
          const uint4* row = reinterpret_cast<const uint4*>(ring + (size_t)slot * kWsStageBytes + (size_t)warp * d * 2);
          uint4 w[kWsIn];
#pragma unroll
          for (int j = 0; j < kWsIn; ++j) w[j] = row[min(lane + 32 * j, dc - 1)];
          float acc = 0.f;
#pragma unroll
          for (int j = 0; j < kWsIn; ++j) acc += dot8f(w[j], in[j]);  // chunks past the row meet zeros
          acc = warp_sum(acc);
          if (lane == 0) P.t[a * N + r0 + warp] = acc;
        }
        release_stage();
      }
    }
  }
  if (!ws_meet(st, sm, cpar)) return;
  {
    // t[a][j][gate|up] -> tg[a][j], tu[a][j]: four values (two gate / up pairs) per load, all of a thread's loads in
    // flight together
    constexpr int kT4 = 2 * kWdMaxKR / 4 / kWdThreads;
    // (every CTA reads the whole vector in the same order at the same moment: starting each at a different place was
    // slower -- the L2 serves many requests for one line better than requests spread over all of them)
    const int n4 = (k * 2 * r) >> 2;
    float4 v[kT4];
#pragma unroll
    for (int u = 0; u < kT4; ++u) {
      const int l4 = tid + u * kWdThreads, i4 = l4;
      v[u] = l4 < n4 ? __ldcg(reinterpret_cast<const float4*>(P.t) + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < kT4; ++u) {
      const int l4 = tid + u * kWdThreads, i4 = l4;
      if (l4 < n4) {
        const int i = 4 * i4, a = i / (2 * r), j = (i - a * 2 * r) >> 1;  // (r is a multiple of 8: a run of 4 stays inside one expert)
        sm.tg[a * r + j] = v[u].x, sm.tu[a * r + j] = v[u].y, sm.tg[a * r + j + 1] = v[u].z, sm.tu[a * r + j + 1] = v[u].w;
      }
    }
  }
  if (!ws_sync(sm, cpar)) return;

  // ---------------------------------------------------------------- h_c = silu(t_g . gR_c) * (t_u . uR_c): rows of 2r
  {
    int g0, g1;
    ws_share(P, 1, g0, g1);
    for (int a = 0; a < k; ++a) {
      const int lo = max(g0, a * f) - a * f, hi = min(g1, (a + 1) * f) - a * f;
      if (lo >= hi) continue;
      bool up[kWsIn];
#pragma unroll
      for (int j = 0; j < kWsIn; ++j) {
        const int c0 = lane + 32 * j;
        up[j] = c0 >= rc;
        const float* src = (up[j] ? sm.tu : sm.tg) + a * r + (c0 - (up[j] ? rc : 0)) * 8;
        if (c0 < 2 * rc)
          load8f(src, in[j]);
        else
          zero8f(in[j]);
      }
      for (int r0 = lo; r0 < hi; r0 += kWsRows) {
        const int nr = min(kWsRows, hi - r0);
        if (!wait_stage()) return;
        if (warp < nr) {
          const uint4* row = reinterpret_cast<const uint4*>(ring + (size_t)slot * kWsStageBytes + (size_t)warp * 2 * r * 2);
          uint4 w[kWsIn];
#pragma unroll
          for (int j = 0; j < kWsIn; ++j) w[j] = row[min(lane + 32 * j, 2 * rc - 1)];
          float g = 0.f, u = 0.f;
#pragma unroll
          for (int j = 0; j < kWsIn; ++j) {
            const float v = dot8f(w[j], in[j]);
            if (up[j]) u += v; else g += v;
          }
          g = warp_sum(g), u = warp_sum(u);
          if (lane == 0) P.h[a * f + r0 + warp] = __fdividef(g, 1.0f + __expf(-g)) * u;
        }
        release_stage();
      }
    }
  }
  if (!ws_meet(st, sm, cpar)) return;
  {
    const int n4 = (k * f) >> 2;
    for (int l0 = tid; l0 < n4; l0 += 8 * kWdThreads) {  // eight loads in flight per thread
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int l = l0 + u * kWdThreads, i = l;
        v[u] = l < n4 ? __ldcg(reinterpret_cast<const float4*>(P.h) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int l = l0 + u * kWdThreads, i = l;
        if (l < n4) reinterpret_cast<float4*>(hs)[i] = v[u];
      }
    }
  }
  if (!ws_sync(sm, cpar)) return;

  // ---------------------------------------------------------------- v = h dL: rows of f, four partial sums each
  {
    int g0, g1;
    ws_share(P, 2, g0, g1);
    const int segc = (fc + kWsSeg - 1) / kWsSeg;
    const int rr = warp >> 2, sg = warp & 3;
    for (int a = 0; a < k; ++a) {
      const int lo = max(g0, a * r) - a * r, hi = min(g1, (a + 1) * r) - a * r;
      const float* hv = hs + (size_t)a * f;
      for (int r0 = lo; r0 < hi; r0 += kWsRowsC) {
        const int nr = min(kWsRowsC, hi - r0);
        if (!wait_stage()) return;
        if (rr < nr) {
          const uint4* row = reinterpret_cast<const uint4*>(ring + (size_t)slot * kWsStageBytes + (size_t)rr * f * 2);
          const int c_lo = sg * segc, c_hi = min(fc, c_lo + segc);
          float acc = 0.f;
          for (int c = c_lo + lane; c < c_hi; c += 32) {
            const uint4 w = row[c];
            const float4 ha = reinterpret_cast<const float4*>(hv)[2 * c], hb = reinterpret_cast<const float4*>(hv)[2 * c + 1];
            const float hh[8] = {ha.x, ha.y, ha.z, ha.w, hb.x, hb.y, hb.z, hb.w};
            acc += dot8f(w, hh);
          }
          acc = warp_sum(acc);
          if (lane == 0) P.vpart[(size_t)(a * r + r0 + rr) * kWsSeg + sg] = acc;
        }
        release_stage();
      }
    }
  }
  if (!ws_meet(st, sm, cpar)) return;
  {
    constexpr int kV4 = kWdMaxKR / kWdThreads;  // v[a][j] = its partial sums, in order; all of a thread's loads in flight together
    const int nv = k * r;
    float4 p[kV4];
#pragma unroll
    for (int u = 0; u < kV4; ++u) {
      const int l = tid + u * kWdThreads, i = l;
      p[u] = l < nv ? __ldcg(reinterpret_cast<const float4*>(P.vpart) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < kV4; ++u) {
      const int l = tid + u * kWdThreads, i = l;
      if (l < nv) sm.tg[i] = ((p[u].x + p[u].y) + p[u].z) + p[u].w;
    }
  }
  if (!ws_sync(sm, cpar)) return;

  // ---------------------------------------------------------------- y_i = sum_a w_a (v_a . dR_a[i])
  {
    float wa[kWsIn];
    int off[kWsIn];
#pragma unroll
    for (int j = 0; j < kWsIn; ++j) {
      const int q = lane + 32 * j;  // chunk q of the k * r values of v: expert q / rc, chunk q % rc of its row
      const int a = min(q / rc, k - 1), c = q - a * rc;
      wa[j] = q < k * rc ? sm.sel_w[a] : 0.f;
      off[j] = q < k * rc ? (a * kWsRows * r * 2 + c * 16) : 0;
      if (q < k * rc)
        load8f(sm.tg + q * 8, in[j]);
      else
        zero8f(in[j]);
    }
    const bool good = ld_relaxed(&st->status) == 0u;  // (ordered behind the meeting's acquire; an acquire of its own would hold the rows back)
    int g0, g1;
    ws_share(P, 3, g0, g1);
    for (int r0 = g0; r0 < g1; r0 += kWsRows) {
      const int nr = min(kWsRows, g1 - r0);
      if (!wait_stage()) return;
      if (warp < nr) {
        const unsigned char* base = ring + (size_t)slot * kWsStageBytes + (size_t)warp * r * 2;
        float acc = 0.f;
#pragma unroll
        for (int j = 0; j < kWsIn; ++j) acc = fmaf(wa[j], dot8f(*reinterpret_cast<const uint4*>(base + off[j]), in[j]), acc);
        acc = warp_sum(acc);
        if (lane == 0 && good) {
          if (P.x_is_bf16)
            ((__nv_bfloat16*)P.y)[r0 + warp] = __float2bfloat16_rn(acc);
          else
            ((float*)P.y)[r0 + warp] = acc;
        }
      }
      release_stage();
    }
  }
}

}  // namespace

// Small factors (the chain's latency counts): wd_decode_kernel.  Large ones (bandwidth counts): wd_stream_kernel.
static bool wd_small(const moe_config& c) { return 6ll * c.wd_rank * (c.d_model + c.d_ff) * c.top_k <= (32ll << 20); }
static size_t wd_stream_smem(const moe_config& c) {
  return kWsHeader + (((size_t)c.top_k * c.d_ff * 4 + 127) / 128) * 128 + (size_t)kWsStages * kWsStageBytes + 128;
}

bool wd_decode_applies(const moe_config& c, int T) {
  if (T != 1 || c.wd_rank <= 0 || c.d_model > kWdMaxD || (long long)c.top_k * c.wd_rank > kWdMaxKR) return false;
  if (wd_small(c)) return true;
  // the streaming variant keeps the input vectors in registers (64 values per lane) and two rows of f values per stage
  return 2 * c.wd_rank <= 32 * 8 * kWsIn && c.d_model <= 32 * 8 * kWsIn && (size_t)kWsRowsC * c.d_ff * 2 <= (size_t)kWsStageBytes &&
         wd_stream_smem(c) <= 227u * 1024u;
}

int launch_wd_decode(moe_ctx* ctx, const void* x, const moe_weights* w, int32_t* topk_idx, float* topk_w, void* y,
                     float* t, float* h, float* vpart, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  if (!wd_decode_applies(c, 1)) return MOE_ERR_UNSUPPORTED;
  WdParams P{};
  P.k = c.top_k, P.E = c.n_experts, P.d = c.d_model, P.f = c.d_ff, P.r = c.wd_rank;
  P.x_is_bf16 = c.x_dtype == MOE_BF16, P.renorm = c.renorm;
  P.x = x, P.w_router = (const uint16_t*)w->w_router, P.b_router = w->b_router, P.expert_slot = w->expert_slot;
  P.wd_a = (const uint16_t*)w->wd_a, P.wd_b = (const uint16_t*)w->wd_b;
  P.wd_c = (const uint16_t*)w->wd_c, P.wd_d = (const uint16_t*)w->wd_d;
  P.topk_idx = topk_idx, P.topk_w = topk_w, P.t = t, P.h = h, P.vpart = vpart, P.y = y, P.st = ctx->d_state;
  const int grid = ctx->sm_count;  // one CTA per SM: the CTAs wait for each other, the grid must fit on the GPU at once
  if (!wd_small(c)) {
    const size_t smem = wd_stream_smem(c);
    if ((long long)smem > ctx->max_smem_optin) return MOE_ERR_UNSUPPORTED;
    MOE_CUDA_TRY(cudaFuncSetAttribute(wd_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    P.split = kWsSeg;
    MOE_CUDA_TRY(launch_pdl(wd_stream_kernel, dim3(grid), dim3(kWsThreads), smem, s, P));
    ctx->launches++;
    return MOE_OK;
  }
  const size_t smem = sizeof(WdSmem);
  MOE_CUDA_TRY(cudaFuncSetAttribute(wd_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int per_sm = 0;
  MOE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, wd_decode_kernel, kWdThreads, smem));
  if (per_sm < 1) return MOE_ERR_UNSUPPORTED;
  const int n_warps = grid * kWdWarps;
  int split = n_warps / (c.top_k * c.wd_rank);
  P.split = split < 1 ? 1 : (split > kWdMaxSplit ? kWdMaxSplit : split);
  MOE_CUDA_TRY(launch_pdl(wd_decode_kernel, dim3(grid), dim3(kWdThreads), smem, s, P));
  ctx->launches++;
  return MOE_OK;
}

}  // namespace cosmoe
