// Router (logits + softmax + top-k + gate weights), token->expert grouping, row gather,
// gate-weighted combine and the one-off weight packing kernels.
#include "common.cuh"

namespace cosmoe {

// ------------------------------------------------------------------------------------ router
// Threads split the d axis and keep E partial logits each; shuffle trees finish them; one warp then
// does the E-wide softmax and the top-k with one or two experts per lane (E <= 64).
// Selection runs on the logits: softmax is monotonic, so top_k(W) = top_k(R) (Eq. 2, Eq. 3), and
// the logits carry more bits than the fp32 probabilities.  Ties go to the lower expert index.
template <typename XT>
__device__ __forceinline__ void load_x8(const XT* p, float* f);
template <>
__device__ __forceinline__ void load_x8<float>(const float* p, float* f) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  f[0] = a.x, f[1] = a.y, f[2] = a.z, f[3] = a.w, f[4] = b.x, f[5] = b.y, f[6] = b.z, f[7] = b.w;
}
template <>
__device__ __forceinline__ void load_x8<__nv_bfloat16>(const __nv_bfloat16* p, float* f) {
  unpack8(*reinterpret_cast<const uint4*>(p), f);
}

constexpr int kRouteWarps = 8;

// Partial logits of one token over the chunks [c_begin, c_end) step c_step of the d axis.  The token's
// chunks are fetched eight at a time before any arithmetic, so a warp pays one memory round trip per group.
template <typename XT, int EMAX>
__device__ __forceinline__ void route_partial(const XT* __restrict__ xr, const uint16_t* __restrict__ w_router, int E,
                                              int c_begin, int c_end, int c_step, float* acc) {
  const bool vec = (E % 8) == 0;
  for (int cb = c_begin; cb < c_end; cb += 8 * c_step) {
    float xv[8][8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int c = cb + u * c_step;
      if (c < c_end) {
        load_x8<XT>(xr + c * 8, xv[u]);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) xv[u][i] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int c = min(cb + u * c_step, c_end - 1);  // clamped rows meet zero inputs
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint16_t* wr = w_router + (size_t)(c * 8 + i) * E;
        if (vec) {
#pragma unroll
          for (int e8 = 0; e8 < EMAX / 8; ++e8) {
            if (e8 * 8 < E) {
              float wv[8];
              unpack8(__ldg(reinterpret_cast<const uint4*>(wr) + e8), wv);
#pragma unroll
              for (int j = 0; j < 8; ++j) acc[e8 * 8 + j] = fmaf(xv[u][i], wv[j], acc[e8 * 8 + j]);
            }
          }
        } else {
#pragma unroll
          for (int e = 0; e < EMAX; ++e)
            if (e < E) acc[e] = fmaf(xv[u][i], bf16_to_float(__ldg(wr + e)), acc[e]);
        }
      }
    }
  }
}

// Many tokens: one warp per token, lanes split the d axis.
template <typename XT, int EMAX>
__global__ void __launch_bounds__(kRouteWarps * 32)
    route_kernel(const XT* __restrict__ x, const uint16_t* __restrict__ w_router, const float* __restrict__ bias, int T,
                 int d, int E, int k, int renorm, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                 float* __restrict__ probs) {
  __shared__ float s_logit[kRouteWarps][EMAX];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int t = blockIdx.x * kRouteWarps + wib;
  if (t >= T) return;
  float acc[EMAX];
#pragma unroll
  for (int e = 0; e < EMAX; ++e) acc[e] = 0.f;
  route_partial<XT, EMAX>(x + (size_t)t * d, w_router, E, lane, d / 8, 32, acc);
#pragma unroll
  for (int e = 0; e < EMAX; ++e)
    if (e < E) acc[e] = warp_sum(acc[e]);
  if (lane == 0) {
#pragma unroll
    for (int e = 0; e < EMAX; ++e)
      if (e < E) s_logit[wib][e] = acc[e];
  }
  __syncwarp();
  const float l0 = lane < E ? s_logit[wib][lane] + (bias ? bias[lane] : 0.f) : 0.f;
  const float l1 = lane + 32 < E ? s_logit[wib][lane + 32] + (bias ? bias[lane + 32] : 0.f) : 0.f;
  warp_route_finish(l0, l1, E, k, renorm, lane, topk_idx + (size_t)t * k, topk_w + (size_t)t * k,
                    probs ? probs + (size_t)t * E : nullptr);
}

// Many tokens, 8 experts, a router matrix of at most 64 KB: every CTA first copies W_r into shared memory, its
// 16-byte rows (one input feature each) shifted by 16 bytes per 8 rows so that lanes reading rows 8 apart fall
// into different banks; then its warps walk the tokens, a lane taking 8 consecutive features per 16-byte load
// of x.  (The kernel above reads W_r through L1 with 32 cache lines per warp instruction.)
template <typename XT>
__global__ void __launch_bounds__(kRouteWarps * 32)
    route_smem_kernel(const XT* __restrict__ x, const uint16_t* __restrict__ w_router, const float* __restrict__ bias,
                      int T, int d, int k, int renorm, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                      float* __restrict__ probs) {
  constexpr int E = 8;
  extern __shared__ __align__(16) unsigned char s_w[];  // row r at byte 16 * (r + r / 8)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int r = threadIdx.x; r < d; r += blockDim.x)
    *reinterpret_cast<uint4*>(s_w + 16 * (r + (r >> 3))) = __ldg(reinterpret_cast<const uint4*>(w_router) + r);
  asm volatile("griddepcontrol.wait;" ::: "memory");  // x may come from the kernel before
  __syncthreads();
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int chunks = d >> 3;
  const float b0 = (bias && lane < E) ? bias[lane] : 0.f;
  for (int t = blockIdx.x * kRouteWarps + wib; t < T; t += gridDim.x * kRouteWarps) {
    const XT* xr = x + (size_t)t * d;
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int cb = lane; cb < chunks; cb += 32 * 8) {
      float xv[8][8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c = cb + 32 * u;
        if (c < chunks) {
          load_x8<XT>(xr + c * 8, xv[u]);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) xv[u][i] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c = min(cb + 32 * u, chunks - 1);  // clamped rows meet zero inputs
        const unsigned char* rows = s_w + 16 * (9 * c);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float wv[8];
          unpack8(*reinterpret_cast<const uint4*>(rows + 16 * i), wv);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[j] = fmaf(xv[u][i], wv[j], acc[j]);
        }
      }
    }
    float l0 = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const float v = warp_sum(acc[e]);
      if (lane == e) l0 = v;
    }
    l0 += b0;
    warp_route_finish(l0, 0.f, E, k, renorm, lane, topk_idx + (size_t)t * k, topk_w + (size_t)t * k,
                      probs ? probs + (size_t)t * E : nullptr);
  }
}

// Few tokens (decode): one CTA per token, all 256 threads split the d axis so the weight rows are
// fetched in a single round trip; warp 0 finishes.
template <typename XT, int EMAX>
__global__ void __launch_bounds__(kRouteWarps * 32)
    route_block_kernel(const XT* __restrict__ x, const uint16_t* __restrict__ w_router, const float* __restrict__ bias,
                       int T, int d, int E, int k, int renorm, int32_t* __restrict__ topk_idx,
                       float* __restrict__ topk_w, float* __restrict__ probs) {
  __shared__ float s_part[kRouteWarps][EMAX];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int t = blockIdx.x;
  float acc[EMAX];
#pragma unroll
  for (int e = 0; e < EMAX; ++e) acc[e] = 0.f;
  route_partial<XT, EMAX>(x + (size_t)t * d, w_router, E, threadIdx.x, d / 8, kRouteWarps * 32, acc);
#pragma unroll
  for (int e = 0; e < EMAX; ++e)
    if (e < E) acc[e] = warp_sum(acc[e]);
  if (lane == 0) {
#pragma unroll
    for (int e = 0; e < EMAX; ++e)
      if (e < E) s_part[wib][e] = acc[e];
  }
  __syncthreads();
  if (wib != 0) return;
  float l0 = 0.f, l1 = 0.f;
  if (lane < E) {
    for (int w = 0; w < kRouteWarps; ++w) l0 += s_part[w][lane];
    if (bias) l0 += bias[lane];
  }
  if (lane + 32 < E) {
    for (int w = 0; w < kRouteWarps; ++w) l1 += s_part[w][lane + 32];
    if (bias) l1 += bias[lane + 32];
  }
  warp_route_finish(l0, l1, E, k, renorm, lane, topk_idx + (size_t)t * k, topk_w + (size_t)t * k,
                    probs ? probs + (size_t)t * E : nullptr);
}

template <typename XT>
static int launch_route_t(moe_ctx* ctx, const void* x, int T, const moe_weights* w, int32_t* idx, float* wt,
                          float* probs, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  const dim3 block(kRouteWarps * 32);
  const bool few = T <= 64;
  const dim3 grid(few ? T : (T + kRouteWarps - 1) / kRouteWarps);
  const XT* xp = (const XT*)x;
  const uint16_t* wr = (const uint16_t*)w->w_router;
  const size_t staged = 18 * (size_t)c.d_model;  // bytes of the shifted copy of W_r (8 experts)
  if (!few && c.n_experts == 8 && staged <= 96 * 1024) {
    MOE_CUDA_TRY(cudaFuncSetAttribute(route_smem_kernel<XT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)staged));
    const int ctas = (T + kRouteWarps - 1) / kRouteWarps;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(ctas < 2 * ctx->sm_count ? ctas : 2 * ctx->sm_count), lc.blockDim = block;
    lc.dynamicSmemBytes = staged, lc.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr, lc.numAttrs = 1;
    MOE_CUDA_TRY(cudaLaunchKernelEx(&lc, route_smem_kernel<XT>, xp, wr, (const float*)w->b_router, T, c.d_model, c.top_k,
                                    c.renorm, idx, wt, probs));
    ctx->launches++;
    return MOE_OK;
  }
#define ROUTE_CASE(EM)                                                                                              \
  do {                                                                                                              \
    if (few)                                                                                                        \
      route_block_kernel<XT, EM><<<grid, block, 0, s>>>(xp, wr, w->b_router, T, c.d_model, c.n_experts, c.top_k,    \
                                                        c.renorm, idx, wt, probs);                                  \
    else                                                                                                            \
      route_kernel<XT, EM><<<grid, block, 0, s>>>(xp, wr, w->b_router, T, c.d_model, c.n_experts, c.top_k, c.renorm, \
                                                  idx, wt, probs);                                                  \
  } while (0)
  if (c.n_experts <= 8)
    ROUTE_CASE(8);
  else if (c.n_experts <= 16)
    ROUTE_CASE(16);
  else if (c.n_experts <= 32)
    ROUTE_CASE(32);
  else
    ROUTE_CASE(64);
#undef ROUTE_CASE
  MOE_CUDA_TRY(cudaGetLastError());
  ctx->launches++;
  return MOE_OK;
}

int launch_route(moe_ctx* ctx, const void* x, int T, const moe_weights* w, int32_t* idx, float* wt, float* probs,
                 cudaStream_t s) {
  if (ctx->cfg.x_dtype == MOE_F32) return launch_route_t<float>(ctx, x, T, w, idx, wt, probs, s);
  return launch_route_t<__nv_bfloat16>(ctx, x, T, w, idx, wt, probs, s);
}

// ------------------------------------------------------------------------------------ grouping
// One CTA: histogram of the T*k pairs by expert, exclusive scan, then a stable scatter that walks
// the pairs in order, 1024 at a time (rank inside a warp by match_any, across warps by a scan).
constexpr int kPermThreads = 1024;

__global__ void __launch_bounds__(kPermThreads)
    permute_kernel(const int32_t* __restrict__ topk_idx, int n, int E, int32_t* __restrict__ offsets,
                   int32_t* __restrict__ perm, int32_t* __restrict__ inv, DeviceState* st) {
  __shared__ int s_base[MOE_MAX_EXPERTS];
  __shared__ int s_wc[kPermThreads / 32][MOE_MAX_EXPERTS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();
  if (tid < MOE_MAX_EXPERTS) s_base[tid] = 0;
  __syncthreads();
  for (int p = tid; p < n; p += kPermThreads) {
    const int e = topk_idx[p];
    if (e < 0 || e >= E)
      flag_error(st, MOE_ERR_STATE, 0x100u);
    else
      atomicAdd(&s_base[e], 1);
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int e = 0; e < E; ++e) {
      const int c = s_base[e];
      offsets[e] = run;
      s_base[e] = run;
      run += c;
    }
    offsets[E] = run;
  }
  __syncthreads();
  for (int p0 = 0; p0 < n; p0 += kPermThreads) {
    for (int i = tid; i < (kPermThreads / 32) * MOE_MAX_EXPERTS; i += kPermThreads) (&s_wc[0][0])[i] = 0;
    __syncthreads();
    const int p = p0 + tid;
    int e = -1;
    if (p < n) {
      e = topk_idx[p];
      if (e < 0 || e >= E) e = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    if (e >= 0 && rank == 0) s_wc[warp][e] = __popc(peers);
    __syncthreads();
    if (tid < E) {
      int run = s_base[tid];
      for (int w = 0; w < kPermThreads / 32; ++w) {
        const int c = s_wc[w][tid];
        s_wc[w][tid] = run;
        run += c;
      }
      s_base[tid] = run;
    }
    __syncthreads();
    if (e >= 0) {
      const int slot = s_wc[warp][e] + rank;
      perm[slot] = p;
      inv[p] = slot;
    }
    __syncthreads();
  }
}

int launch_permute(moe_ctx* ctx, const int32_t* idx, int T, int32_t* offsets, int32_t* perm, int32_t* inv,
                   cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  MOE_CUDA_TRY(launch_pdl(permute_kernel, dim3(1), dim3(kPermThreads), 0, s, idx, T * c.top_k, c.n_experts, offsets, perm, inv,
                          ctx->d_state));
  ctx->launches++;
  return MOE_OK;
}

// ------------------------------------------------------------------------------------ gather
// xperm[s][:] = bf16(x[perm[s] / k][:])  (operand rows of the tensor-core path, grouped by expert)
template <typename XT>
__global__ void gather_rows_kernel(const XT* __restrict__ x, const int32_t* __restrict__ perm, int n_slots, int k,
                                   int d, uint4* __restrict__ out, DeviceState* st) {
  const int chunks = d / 8;
  const long long total = (long long)n_slots * chunks;
  pdl_launch_dependents();
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int s = (int)(i / chunks), c = (int)(i % chunks);
    const int t = perm[s] / k;
    float f[8];
    load_x8<XT>(x + (size_t)t * d + c * 8, f);
    uint4 o;
    o.x = pack_bf16x2(f[0], f[1]), o.y = pack_bf16x2(f[2], f[3]);
    o.z = pack_bf16x2(f[4], f[5]), o.w = pack_bf16x2(f[6], f[7]);
    out[i] = o;
  }
}

int launch_gather_rows(moe_ctx* ctx, const void* x, const int32_t* perm, int n_slots, void* xperm, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  const long long total = (long long)n_slots * (c.d_model / 8);
  const int block = 256;
  const int grid = (int)((total + block - 1) / block < 148 * 16 ? (total + block - 1) / block : 148 * 16);
  if (c.x_dtype == MOE_F32)
    MOE_CUDA_TRY(launch_pdl(gather_rows_kernel<float>, dim3(grid), dim3(block), 0, s, (const float*)x, perm, n_slots,
                            c.top_k, c.d_model, (uint4*)xperm, ctx->d_state));
  else
    MOE_CUDA_TRY(launch_pdl(gather_rows_kernel<__nv_bfloat16>, dim3(grid), dim3(block), 0, s, (const __nv_bfloat16*)x, perm,
                            n_slots, c.top_k, c.d_model, (uint4*)xperm, ctx->d_state));
  ctx->launches++;
  return MOE_OK;
}

// ------------------------------------------------------------------------------------ combine
// y[t][c] = sum_j w[t][j] * out_slots[inv[t*k+j]][c], j ascending, fp32, one rounding to the output type.
template <typename YT>
__global__ void combine_kernel(const float* __restrict__ out_slots, const float* __restrict__ wt,
                               const int32_t* __restrict__ inv, int T, int k, int d, int planes, YT* __restrict__ y) {
  const int quads = d / 4;
  const long long total = (long long)T * quads;
  pdl_launch_dependents();
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int t = (int)(i / quads), q = (int)(i % quads);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = 0; j < k; ++j) {
      const float w = wt[(size_t)t * k + j];
      const float* src = out_slots + (size_t)inv[(size_t)t * k + j] * d + q * 4;
      float4 o = *reinterpret_cast<const float4*>(src);
      for (int pl = 1; pl < planes; ++pl) {  // partial sums of a cut contraction, in order
        const float4 o2 = *reinterpret_cast<const float4*>(src + (size_t)pl * T * k * d);
        o.x += o2.x, o.y += o2.y, o.z += o2.z, o.w += o2.w;
      }
      acc.x = fmaf(w, o.x, acc.x), acc.y = fmaf(w, o.y, acc.y), acc.z = fmaf(w, o.z, acc.z), acc.w = fmaf(w, o.w, acc.w);
    }
    if constexpr (sizeof(YT) == 4) {
      *reinterpret_cast<float4*>(y + (size_t)t * d + q * 4) = acc;
    } else {
      uint2 o;
      o.x = pack_bf16x2(acc.x, acc.y), o.y = pack_bf16x2(acc.z, acc.w);
      *reinterpret_cast<uint2*>(y + (size_t)t * d + q * 4) = o;
    }
  }
}

int launch_combine(moe_ctx* ctx, const float* out_slots, const float* wt, const int32_t* inv, int T, void* y,
                   int planes, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  const long long total = (long long)T * (c.d_model / 4);
  const int block = 256;
  const int grid = (int)((total + block - 1) / block < 148 * 16 ? (total + block - 1) / block : 148 * 16);
  if (c.x_dtype == MOE_F32)
    MOE_CUDA_TRY(launch_pdl(combine_kernel<float>, dim3(grid), dim3(block), 0, s, out_slots, wt, inv, T, c.top_k, c.d_model,
                            planes, (float*)y));
  else
    MOE_CUDA_TRY(launch_pdl(combine_kernel<__nv_bfloat16>, dim3(grid), dim3(block), 0, s, out_slots, wt, inv, T, c.top_k,
                            c.d_model, planes, (__nv_bfloat16*)y));
  ctx->launches++;
  return MOE_OK;
}

// ------------------------------------------------------------------------------------ packing
// in [B][R][C] -> out[b][c][sub][r] with nsub interleaved row kinds: a tiled transpose.
__global__ void pack_transpose_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out, int R, int C,
                                      int nsub, int sub) {
  __shared__ uint16_t tile[32][33];
  const int b = blockIdx.z;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const uint16_t* src = in + (size_t)b * R * C;
  uint16_t* dst = out + (size_t)b * C * nsub * R;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    if (r < R && c < C) tile[i][threadIdx.x] = src[(size_t)r * C + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < R && c < C) dst[((size_t)c * nsub + sub) * R + r] = tile[threadIdx.x][i];
  }
}

// out[b][c][sub][:] = in[b][c][:]  (rows copied into an interleaved layout, 16 bytes per thread)
__global__ void pack_rows_kernel(const uint4* __restrict__ in, uint4* __restrict__ out, long long rows, int chunks,
                                 int nsub, int sub) {
  const long long total = rows * chunks;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / chunks;
    const int c = (int)(i - r * chunks);
    out[(r * nsub + sub) * chunks + c] = in[i];
  }
}

static int pack_one(const void* in, void* out, int B, int R, int C, int nsub, int sub, cudaStream_t s) {
  const dim3 grid((C + 31) / 32, (R + 31) / 32, B), block(32, 8);
  if (grid.y > 65535u || grid.z > 65535u) return MOE_ERR_UNSUPPORTED;
  pack_transpose_kernel<<<grid, block, 0, s>>>((const uint16_t*)in, (uint16_t*)out, R, C, nsub, sub);
  MOE_CUDA_TRY(cudaGetLastError());
  return MOE_OK;
}

}  // namespace cosmoe

using namespace cosmoe;

extern "C" {

int moe_pack_dense(int32_t d, int32_t f, int32_t n_experts, const void* w_gate, const void* w_up, const void* w_down,
                   void* gud_out, void* stream) {
  if (d <= 0 || f <= 0 || n_experts <= 0 || !w_gate || !w_up || !w_down || !gud_out) return MOE_ERR_INVALID_ARG;
  if (d % 8 || f % 8) return MOE_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  int rc = pack_one(w_gate, gud_out, n_experts, d, f, 3, 0, s);
  if (rc == MOE_OK) rc = pack_one(w_up, gud_out, n_experts, d, f, 3, 1, s);
  if (rc == MOE_OK) {
    pack_rows_kernel<<<148 * 8, 256, 0, s>>>((const uint4*)w_down, (uint4*)gud_out, (long long)n_experts * f, d / 8, 3, 2);
    MOE_CUDA_TRY(cudaGetLastError());
  }
  return rc;
}

int moe_pack_wd(int32_t d, int32_t f, int32_t r, int32_t n_experts, const void* gL, const void* gR, const void* uL,
                const void* uR, const void* dL, const void* dR, void* wd_a, void* wd_b, void* wd_c, void* wd_d,
                void* stream) {
  if (d <= 0 || f <= 0 || r <= 0 || n_experts <= 0 || !gL || !gR || !uL || !uR || !dL || !dR || !wd_a || !wd_b ||
      !wd_c || !wd_d)
    return MOE_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  int rc = pack_one(gL, wd_a, n_experts, d, r, 2, 0, s);
  if (rc == MOE_OK) rc = pack_one(uL, wd_a, n_experts, d, r, 2, 1, s);
  if (rc == MOE_OK) rc = pack_one(gR, wd_b, n_experts, r, f, 2, 0, s);
  if (rc == MOE_OK) rc = pack_one(uR, wd_b, n_experts, r, f, 2, 1, s);
  if (rc == MOE_OK) rc = pack_one(dL, wd_c, n_experts, f, r, 1, 0, s);
  if (rc == MOE_OK) rc = pack_one(dR, wd_d, n_experts, r, d, 1, 0, s);
  return rc;
}

}  // extern "C"
