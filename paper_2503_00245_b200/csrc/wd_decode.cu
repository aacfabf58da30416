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
  float x[kWdMaxD];
  float tg[kWdMaxKR], tu[kWdMaxKR];  // t de-interleaved; later v in tg
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

// dot of 8 bf16 weights with 8 fp32 values
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
        wr[q] = __ldg(reinterpret_cast<const uint4*>(P.w_router + (size_t)min(tid + q * kWdThreads, d - 1) * E + e0));
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
        if (c0 + 32 * u < dc) acc += dot8f(w[u], sm.x + (c0 + 32 * u) * 8);
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
        const float v = dot8f(w[q], (part ? sm.tu : sm.tg) + a * r + cc * 8);
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
      acc = fmaf(sm.sel_w[a], dot8f(w, sm.tg + a * r + c * 8), acc);
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

}  // namespace

bool wd_decode_applies(const moe_config& c, int T) {
  // latency-bound regime only: with more than 32 MB of selected weights the streaming kernel with its TMA ring is faster
  const long long bytes = 6ll * c.wd_rank * (c.d_model + c.d_ff) * c.top_k;
  return T == 1 && c.wd_rank > 0 && c.d_model <= kWdMaxD && (long long)c.top_k * c.wd_rank <= kWdMaxKR &&
         bytes <= (32ll << 20);
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
  const size_t smem = sizeof(WdSmem);
  MOE_CUDA_TRY(cudaFuncSetAttribute(wd_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  // the CTAs wait for each other: the grid must fit on the GPU at once
  int per_sm = 0;
  MOE_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, wd_decode_kernel, kWdThreads, smem));
  if (per_sm < 1) return MOE_ERR_UNSUPPORTED;
  const int grid = ctx->sm_count;  // one CTA per SM: fewer arrivals at a meeting beat more warps per product
  const int n_warps = grid * kWdWarps;
  int split = n_warps / (c.top_k * c.wd_rank);
  P.split = split < 1 ? 1 : (split > kWdMaxSplit ? kWdMaxSplit : split);
  MOE_CUDA_TRY(launch_pdl(wd_decode_kernel, dim3(grid), dim3(kWdThreads), smem, s, P));
  ctx->launches++;
  return MOE_OK;
}

}  // namespace cosmoe
