// C boundary: contexts, validation, workspace layout and dispatch of the hot calls.
#include <new>

#include "common.cuh"

namespace cosmoe {

thread_local int g_last_cuda_error = 0;

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int validate_config(const moe_config* c) {
  if (!c) return MOE_ERR_INVALID_ARG;
  if (c->d_model <= 0 || c->d_ff <= 0 || c->n_experts <= 0 || c->top_k <= 0 || c->wd_rank < 0) return MOE_ERR_INVALID_ARG;
  if (c->d_model % 8 || c->d_ff % 8 || c->wd_rank % 8) return MOE_ERR_UNSUPPORTED;
  if (c->n_experts > MOE_MAX_EXPERTS || c->top_k > MOE_MAX_TOPK || c->top_k > c->n_experts) return MOE_ERR_UNSUPPORTED;
  if (c->x_dtype != MOE_F32 && c->x_dtype != MOE_BF16) return MOE_ERR_UNSUPPORTED;
  if (c->renorm != 0 && c->renorm != 1) return MOE_ERR_INVALID_ARG;
  if (c->path < MOE_PATH_AUTO || c->path > MOE_PATH_TENSOR) return MOE_ERR_INVALID_ARG;
  if (c->d_model > 16384 || c->d_ff > 65536 || c->wd_rank > 16384) return MOE_ERR_UNSUPPORTED;
  return MOE_OK;
}

WsLayout ws_layout(const moe_config& c, int T) {
  WsLayout L{};
  const size_t n = (size_t)T * c.top_k, A = 256;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, A);
    return o;
  };
  L.topk_idx = take(n * 4);
  L.topk_w = take(n * 4);
  L.offsets = take((size_t)(c.n_experts + 1) * 4);
  L.perm = take(n * 4);
  L.inv = take(n * 4);
  const bool stream_ok = T <= MOE_STREAM_MAX_TOKENS;
  const bool tensor_ok = true;
  L.vec_a = take(stream_ok ? n * 2 * (size_t)c.wd_rank * 4 : 0);
  L.vec_b = take(stream_ok ? n * (size_t)c.d_ff * 4 : 0);
  L.vec_c = take(stream_ok ? n * (size_t)c.wd_rank * 8 * 4 : 0);  // v, in up to 8 segments per value
  L.xperm = take(tensor_ok ? n * (size_t)c.d_model * 2 : 0);
  L.hidden = take(tensor_ok ? n * (size_t)c.d_ff * 2 : 0);
  const size_t rp = ((size_t)c.wd_rank + 63) / 64 * 64;            // the rank rounded up to the tensor path's K step
  L.mid_a = take(tensor_ok ? n * 4 * rp * 2 : 0);  // t_g, t_u as hi + lo bf16 pairs
  L.mid_b = take(tensor_ok ? n * 2 * rp * 2 : 0);  // v as a hi + lo pair
  L.out_slots = take(n * (size_t)c.d_model * 4 * (n <= (size_t)kKSplitMaxSlots ? kKSplitMax : 1));  // room for partial-sum planes
  L.total = off + A;
  return L;
}

static int pick_path(const moe_config& c, int T) {
  if (c.path != MOE_PATH_AUTO) return c.path;
  if (T > MOE_STREAM_MAX_TOKENS) return MOE_PATH_TENSOR;
  if (c.wd_rank == 0 && c.d_model > kDenseStreamMaxD) return MOE_PATH_TENSOR;  // the tensor path takes any width
  return MOE_PATH_STREAM;
}

static bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

static int check_weights(const moe_config& c, const moe_weights* w, bool need_router, bool need_experts) {
  if (!w) return MOE_ERR_INVALID_ARG;
  if (need_router && (!w->w_router || misaligned(w->w_router))) return MOE_ERR_INVALID_ARG;
  if (need_experts) {
    if (c.wd_rank == 0) {
      if (!w->gud || misaligned(w->gud)) return MOE_ERR_INVALID_ARG;
    } else {
      if (!w->wd_a || !w->wd_b || !w->wd_c || !w->wd_d) return MOE_ERR_INVALID_ARG;
      if (misaligned(w->wd_a) || misaligned(w->wd_b) || misaligned(w->wd_c) || misaligned(w->wd_d))
        return MOE_ERR_INVALID_ARG;
    }
  }
  return MOE_OK;
}

}  // namespace cosmoe

using namespace cosmoe;

extern "C" {

const char* moe_status_string(int status) {
  switch (status) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_UNSUPPORTED: return "unsupported shape, dtype or path";
    case MOE_ERR_WORKSPACE: return "workspace too small";
    case MOE_ERR_CUDA: return "CUDA runtime error";
    case MOE_ERR_TIMEOUT: return "a bounded wait expired";
    case MOE_ERR_STATE: return "invalid state";
    case MOE_ERR_NO_DEVICE: return "no usable CUDA device";
    default: return "unknown status";
  }
}

int moe_last_cuda_error(void) { return g_last_cuda_error; }

int moe_device_sm_count(void) {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return -MOE_ERR_NO_DEVICE;
  }
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return -MOE_ERR_NO_DEVICE;
  }
  return n;
}

int moe_create(const moe_config* cfg, moe_ctx** out) {
  if (!out) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate_config(cfg);
  if (rc != MOE_OK) return rc;
  int dev = 0, count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0) {
    (void)cudaGetLastError();
    return MOE_ERR_NO_DEVICE;
  }
  MOE_CUDA_TRY(cudaGetDevice(&dev));
  int major = 0, minor = 0;
  MOE_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  MOE_CUDA_TRY(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
  if (major != 10) return MOE_ERR_NO_DEVICE;  // kernels are built for sm_100a only
  moe_ctx* c = new (std::nothrow) moe_ctx();
  if (!c) return MOE_ERR_STATE;
  c->cfg = *cfg;
  c->device = dev;
  c->launches = 0;
  c->fin_wait_budget = 0;
  c->d_state = nullptr;
  c->h_state = nullptr;
  c->acc = nullptr;
  c->acc_elems = (cfg->wd_rank == 0 && cfg->d_model <= kDenseStreamMaxD)
                     ? (size_t)MOE_STREAM_MAX_TOKENS * cfg->top_k * cfg->d_model
                     : 0;
  cudaError_t e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e == cudaSuccess) e = cudaMalloc((void**)&c->d_state, sizeof(DeviceState));
  if (e == cudaSuccess) e = cudaMemset(c->d_state, 0, sizeof(DeviceState));
  if (e == cudaSuccess) e = cudaMallocHost((void**)&c->h_state, sizeof(DeviceState));
  if (e == cudaSuccess && c->acc_elems) e = cudaMalloc((void**)&c->acc, c->acc_elems * sizeof(long long));
  if (e == cudaSuccess && c->acc_elems) e = cudaMemset(c->acc, 0, c->acc_elems * sizeof(long long));
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    (void)cudaGetLastError();
    if (c->d_state) cudaFree(c->d_state);
    if (c->h_state) cudaFreeHost(c->h_state);
    if (c->acc) cudaFree(c->acc);
    delete c;
    return MOE_ERR_CUDA;
  }
  *out = c;
  return MOE_OK;
}

int moe_destroy(moe_ctx* ctx) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->d_state) cudaFree(ctx->d_state);
  if (ctx->h_state) cudaFreeHost(ctx->h_state);
  if (ctx->acc) cudaFree(ctx->acc);
  (void)cudaGetLastError();
  delete ctx;
  return MOE_OK;
}

int moe_check(moe_ctx* ctx, void* stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  MOE_CUDA_TRY(cudaMemcpyAsync(ctx->h_state, ctx->d_state, sizeof(DeviceState), cudaMemcpyDeviceToHost, s));
  MOE_CUDA_TRY(cudaStreamSynchronize(s));
  const unsigned st = ctx->h_state->status;
  if (st == 0) return MOE_OK;
  MOE_CUDA_TRY(cudaMemsetAsync(ctx->d_state, 0, sizeof(DeviceState), s));
  if (ctx->acc) MOE_CUDA_TRY(cudaMemsetAsync(ctx->acc, 0, ctx->acc_elems * sizeof(long long), s));
  MOE_CUDA_TRY(cudaStreamSynchronize(s));
  return st == MOE_ERR_TIMEOUT ? MOE_ERR_TIMEOUT : MOE_ERR_STATE;
}

int moe_workspace_bytes(const moe_config* cfg, int32_t T, size_t* bytes) {
  if (!bytes) return MOE_ERR_INVALID_ARG;
  int rc = validate_config(cfg);
  if (rc != MOE_OK) return rc;
  if (T < 0) return MOE_ERR_INVALID_ARG;
  *bytes = ws_layout(*cfg, T).total;
  return MOE_OK;
}

int moe_set_finaliser_wait(moe_ctx* ctx, long long cycles) {
  if (!ctx || cycles < 0) return MOE_ERR_INVALID_ARG;
  ctx->fin_wait_budget = cycles;
  return MOE_OK;
}

int moe_seed_arrival_counter(moe_ctx* ctx, unsigned long long value, void* stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  ctx->h_state->done_total = value;
  // one-token launches count arrivals in the accumulator words instead: a counter that is out of step with the
  // grid size makes them wait for one arrival more than a launch has
  ctx->h_state->tail_bias = (value % (unsigned long long)ctx->sm_count) != 0ull ? 1u : 0u;
  MOE_CUDA_TRY(cudaMemcpyAsync(&ctx->d_state->done_total, &ctx->h_state->done_total, sizeof(unsigned long long),
                               cudaMemcpyHostToDevice, s));
  MOE_CUDA_TRY(cudaMemcpyAsync(&ctx->d_state->tail_bias, &ctx->h_state->tail_bias, sizeof(unsigned int),
                               cudaMemcpyHostToDevice, s));
  MOE_CUDA_TRY(cudaStreamSynchronize(s));
  return MOE_OK;
}

int moe_launch_count(moe_ctx* ctx, uint64_t* launches) {
  if (!ctx || !launches) return MOE_ERR_INVALID_ARG;
  *launches = ctx->launches;
  return MOE_OK;
}

int moe_route(moe_ctx* ctx, const void* x, int32_t T, const moe_weights* w, int32_t* topk_idx, float* topk_w,
              float* probs, void* stream) {
  if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
  if (T == 0) return MOE_OK;
  if (!x || !topk_idx || !topk_w || misaligned(x)) return MOE_ERR_INVALID_ARG;
  int rc = check_weights(ctx->cfg, w, true, false);
  if (rc != MOE_OK) return rc;
  return launch_route(ctx, x, T, w, topk_idx, topk_w, probs, (cudaStream_t)stream);
}

int moe_permute(moe_ctx* ctx, const int32_t* topk_idx, int32_t T, int32_t* expert_offsets, int32_t* perm,
                int32_t* inv, void* stream) {
  if (!ctx || T < 0 || !expert_offsets) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!topk_idx || !perm || !inv)) return MOE_ERR_INVALID_ARG;
  return launch_permute(ctx, topk_idx, T, expert_offsets, perm, inv, (cudaStream_t)stream);
}

int moe_expert_ffn(moe_ctx* ctx, const void* x, int32_t T, const moe_weights* w, const int32_t* expert_offsets,
                   const int32_t* perm, float* out_slots, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
  if (T == 0) return MOE_OK;
  if (!x || !expert_offsets || !perm || !out_slots || !ws || misaligned(x) || misaligned(out_slots) || misaligned(ws))
    return MOE_ERR_INVALID_ARG;
  int rc = check_weights(ctx->cfg, w, false, true);
  if (rc != MOE_OK) return rc;
  const WsLayout L = ws_layout(ctx->cfg, T);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  const int path = pick_path(ctx->cfg, T);
  cudaStream_t s = (cudaStream_t)stream;
  if (path == MOE_PATH_STREAM) {
    if (T > MOE_STREAM_MAX_TOKENS) return MOE_ERR_UNSUPPORTED;
    if (ctx->cfg.wd_rank == 0)
      return launch_dense_stream(ctx, 1, x, T, w, nullptr, nullptr, expert_offsets, perm, nullptr, out_slots, s);
    return launch_stream_ffn(ctx, 1, x, T, w, nullptr, nullptr, expert_offsets, perm, nullptr, out_slots, (char*)ws, L,
                             s);
  }
  return launch_tensor_ffn(ctx, x, T, w, expert_offsets, perm, (char*)ws, L, out_slots, nullptr, s);
}

int moe_combine(moe_ctx* ctx, const float* out_slots, const float* topk_w, const int32_t* inv, int32_t T, void* y,
                void* stream) {
  if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
  if (T == 0) return MOE_OK;
  if (!out_slots || !topk_w || !inv || !y || misaligned(out_slots) || misaligned(y)) return MOE_ERR_INVALID_ARG;
  return launch_combine(ctx, out_slots, topk_w, inv, T, y, 1, (cudaStream_t)stream);
}

int moe_layer_forward(moe_ctx* ctx, const void* x, int32_t T, const moe_weights* w, void* y, int32_t* topk_idx,
                      float* topk_w, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
  if (T == 0) return MOE_OK;
  if (!x || !y || !ws || misaligned(x) || misaligned(y) || misaligned(ws)) return MOE_ERR_INVALID_ARG;
  int rc = check_weights(ctx->cfg, w, true, true);
  if (rc != MOE_OK) return rc;
  const WsLayout L = ws_layout(ctx->cfg, T);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  const int path = pick_path(ctx->cfg, T);
  if (path == MOE_PATH_STREAM && T > MOE_STREAM_MAX_TOKENS) return MOE_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  char* wsb = (char*)ws;
  int32_t* idx = topk_idx ? topk_idx : (int32_t*)(wsb + L.topk_idx);
  float* wt = topk_w ? topk_w : (float*)(wsb + L.topk_w);
  if (path == MOE_PATH_STREAM && ctx->cfg.wd_rank == 0 && dense_stream_fuses_route(ctx->cfg, T))  // router inside the expert kernel
    return launch_dense_stream(ctx, 0, x, T, w, idx, wt, nullptr, nullptr, y, nullptr, s);
  if (path == MOE_PATH_STREAM && wd_decode_applies(ctx->cfg, T))  // one launch, router included
    return launch_wd_decode(ctx, x, w, idx, wt, y, (float*)(wsb + L.vec_a), (float*)(wsb + L.vec_b),
                            (float*)(wsb + L.vec_c), s);
  rc = launch_route(ctx, x, T, w, idx, wt, nullptr, s);
  if (rc != MOE_OK) return rc;
  if (path == MOE_PATH_STREAM) {
    if (ctx->cfg.wd_rank == 0) return launch_dense_stream(ctx, 0, x, T, w, idx, wt, nullptr, nullptr, y, nullptr, s);
    return launch_stream_ffn(ctx, 0, x, T, w, idx, wt, nullptr, nullptr, y, nullptr, wsb, L, s);
  }
  int32_t* offsets = (int32_t*)(wsb + L.offsets);
  int32_t* perm = (int32_t*)(wsb + L.perm);
  int32_t* inv = (int32_t*)(wsb + L.inv);
  float* out_slots = (float*)(wsb + L.out_slots);
  rc = launch_permute(ctx, idx, T, offsets, perm, inv, s);
  if (rc != MOE_OK) return rc;
  int planes = 1;
  rc = launch_tensor_ffn(ctx, x, T, w, offsets, perm, wsb, L, out_slots, &planes, s);
  if (rc != MOE_OK) return rc;
  return launch_combine(ctx, out_slots, wt, inv, T, y, planes, s);
}

}  // extern "C"
