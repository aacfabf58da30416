// Host-resident experts (Eq. 8, Section 3.4.2): a per-layer cache of expert slots in device memory, filled
// from pinned host memory on routing, and the stacked decode step that uses it; plus the replacement metric
// of Eq. 4-5 on a routing trace.
//
// Bookkeeping is host code: per layer an LRU list over C slots; an expert selected in the current step is never
// the victim; with C == top_k this is exactly the rule of Eq. 8 (bring in what is selected, drop the rest).
// Evicted experts are dropped -- the host copy is the master -- so only host->device bytes move.
// Copies run on the object's own stream: it first waits for the compute stream (nobody may still be reading
// the victim's slot), copies the expert in chunks, updates the layer's expert->slot table in stream order, and
// the compute stream then waits for the copy stream's event.
#include <new>
#include <vector>

#include "common.cuh"

struct moe_offload {
  moe_config cfg;
  int n_layers, slots, E;
  std::vector<const void*> host_experts;    // [n_layers][E] pinned master copies (the pointers are copied on creation)
  unsigned char* device_slots;
  size_t slot_bytes;
  cudaStream_t copy_stream;
  cudaEvent_t ev_compute, ev_copy;
  std::vector<cudaEvent_t> layer_done;      // per layer: recorded after the layer's last kernel by the stacked steps
  std::vector<char> layer_done_set;
  std::vector<std::vector<int>> recency;    // per layer: resident experts, least recently used first
  std::vector<std::vector<int>> slot_of;    // per layer: expert -> slot or -1
  int32_t* d_tables;                        // device [n_layers][E]
  int32_t* h_tables;                        // pinned  [n_layers][E]
  int32_t* h_route;                         // pinned  [k] routing read-back of the stacked step
  uint64_t fetches, bytes, hits;
};

namespace cosmoe {
namespace {

constexpr size_t kCopyChunk = 8u << 20;  // host->device copies are issued in chunks of this size

// A prescribed expert set for one token: the gate weights are the router's probabilities of those experts,
// renormalised over the set (what the layer computes when it is told which experts to use).
struct ForcedSel {
  int32_t e[MOE_MAX_TOPK];
};
__global__ void forced_routing_kernel(const float* __restrict__ probs, int k, int renorm, ForcedSel f,
                                      int32_t* __restrict__ idx, float* __restrict__ wt) {
  const int lane = threadIdx.x;
  const float p = lane < k ? probs[f.e[lane]] : 0.f;
  const float sum = warp_sum(p);
  if (lane < k) {
    idx[lane] = f.e[lane];
    wt[lane] = renorm ? p / sum : p;
  }
}

// A layer's expert -> slot table, passed BY VALUE: every queued update carries its own copy, so a later call
// for the same layer cannot change what an earlier, still pending update writes.
struct SlotTable {
  int32_t slot[MOE_MAX_EXPERTS];
};
__global__ void slot_table_kernel(int32_t* __restrict__ table, int E, SlotTable t) {
  if ((int)threadIdx.x < E) table[threadIdx.x] = t.slot[threadIdx.x];
}

// u = h / sqrt(mean(h^2)) -> x (bf16 or fp32); one CTA
__global__ void rms_glue_kernel(const float* __restrict__ h, int d, void* __restrict__ x, int x_is_bf16) {
  __shared__ float s_part[32];
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) ss = fmaf(h[i], h[i], ss);
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += s_part[w];
  const float inv = rsqrtf(tot / (float)d);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = h[i] * inv;
    if (x_is_bf16)
      ((__nv_bfloat16*)x)[i] = __float2bfloat16_rn(v);
    else
      ((float*)x)[i] = v;
  }
}
// h += y
__global__ void residual_kernel(float* __restrict__ h, const void* __restrict__ y, int d, int y_is_bf16) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < d) h[i] += y_is_bf16 ? __bfloat162float(((const __nv_bfloat16*)y)[i]) : ((const float*)y)[i];
}

// Eq. 4: H = sum_b sum_t sum_e |[e in S(b,t+1)] - [e in S(b,t)]| = size of the symmetric difference of
// consecutive selections, summed.  A row is read as a SET of experts in [0, E): a repeated id counts once and an
// id outside the range not at all, exactly as in the 0/1 activity matrix the equation is written on.
__global__ void replacements_kernel(const int32_t* __restrict__ trace, int B, int T, int k, int E,
                                    unsigned long long* __restrict__ out) {
  unsigned long long local = 0;
  const long long pairs = (long long)B * (T - 1);
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < pairs;
       i += (long long)gridDim.x * blockDim.x) {
    const long long b = i / (T - 1), t = i % (T - 1);
    const int32_t* s0 = trace + (b * T + t) * k;
    const int32_t* s1 = s0 + k;
    int n0 = 0, n1 = 0, common = 0;
    for (int a = 0; a < k; ++a) {
      const int e0 = s0[a], e1 = s1[a];
      bool first0 = e0 >= 0 && e0 < E, first1 = e1 >= 0 && e1 < E;
      for (int c = 0; c < a; ++c) first0 &= (s0[c] != e0), first1 &= (s1[c] != e1);
      n0 += first0, n1 += first1;
      if (first0) {
        bool in1 = false;
        for (int c = 0; c < k; ++c) in1 |= (s1[c] == e0);
        common += in1;
      }
    }
    local += (unsigned long long)(n0 + n1 - 2 * common);
  }
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((threadIdx.x & 31) == 0 && local) atomicAdd(out, local);
}

// Expert balance of a routing trace (Section 3.3): per trace row b (a layer), how often each expert was
// selected.  One CTA per b; integer counts in shared memory, then to global.  Ids outside [0, E) are counted
// in bad_out instead.
__global__ void expert_histogram_kernel(const int32_t* __restrict__ trace, int T, int k, int E,
                                        unsigned long long* __restrict__ counts, unsigned long long* __restrict__ bad_out) {
  __shared__ unsigned int s_cnt[MOE_MAX_EXPERTS];
  __shared__ unsigned int s_bad;
  const int b = blockIdx.x;
  if (threadIdx.x < MOE_MAX_EXPERTS) s_cnt[threadIdx.x] = 0u;
  if (threadIdx.x == 0) s_bad = 0u;
  __syncthreads();
  const long long n = (long long)T * k;
  const int32_t* row = trace + (size_t)b * n;
  for (long long i = threadIdx.x; i < n; i += blockDim.x) {
    const int e = row[i];
    if (e >= 0 && e < E)
      atomicAdd(&s_cnt[e], 1u);
    else
      atomicAdd(&s_bad, 1u);
  }
  __syncthreads();
  if ((int)threadIdx.x < E) counts[(size_t)b * E + threadIdx.x] = s_cnt[threadIdx.x];
  if (threadIdx.x == 0 && s_bad) atomicAdd(bad_out, (unsigned long long)s_bad);
}
// delta[b] = 100 * mean_e | counts[b][e] / sum_e counts[b][e] - 1/E |;  delta[B] = mean over b.  fp64, one thread
// per b, the mean by thread 0 in b order.
__global__ void delta_uniform_kernel(const unsigned long long* __restrict__ counts, int B, int E, double* __restrict__ delta) {
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    double tot = 0.0;
    for (int e = 0; e < E; ++e) tot += (double)counts[(size_t)b * E + e];
    double acc = 0.0;
    for (int e = 0; e < E; ++e) acc += fabs((tot > 0.0 ? (double)counts[(size_t)b * E + e] / tot : 0.0) - 1.0 / (double)E);
    delta[b] = acc / (double)E * 100.0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double m = 0.0;
    for (int b = 0; b < B; ++b) m += delta[b];
    delta[B] = m / (double)B;
  }
}

}  // namespace
}  // namespace cosmoe

using namespace cosmoe;

extern "C" {

int moe_offload_create(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                       const void* const* host_experts, void* device_slots, size_t slot_bytes, moe_offload** out) {
  if (!out) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate_config(cfg);
  if (rc != MOE_OK) return rc;
  if (n_layers <= 0 || !host_experts || !device_slots || ((uintptr_t)device_slots & 15u)) return MOE_ERR_INVALID_ARG;
  if (cfg->wd_rank != 0) return MOE_ERR_UNSUPPORTED;
  if (slots_per_layer < cfg->top_k || slots_per_layer > cfg->n_experts) return MOE_ERR_INVALID_ARG;
  if (slot_bytes != (size_t)cfg->d_ff * 3 * cfg->d_model * 2) return MOE_ERR_INVALID_ARG;
  moe_offload* o = new (std::nothrow) moe_offload();
  if (!o) return MOE_ERR_STATE;
  o->cfg = *cfg;
  o->n_layers = n_layers, o->slots = slots_per_layer, o->E = cfg->n_experts;
  o->host_experts.assign(host_experts, host_experts + (size_t)n_layers * cfg->n_experts);
  o->device_slots = (unsigned char*)device_slots;
  o->slot_bytes = slot_bytes;
  o->fetches = o->bytes = o->hits = 0;
  o->copy_stream = nullptr, o->ev_compute = nullptr, o->ev_copy = nullptr;
  o->d_tables = nullptr, o->h_tables = nullptr, o->h_route = nullptr;
  const size_t tb = (size_t)n_layers * o->E * sizeof(int32_t);
  cudaError_t e = cudaStreamCreateWithFlags(&o->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&o->ev_compute, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&o->ev_copy, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMalloc((void**)&o->d_tables, tb);
  if (e == cudaSuccess) e = cudaMallocHost((void**)&o->h_tables, tb);
  if (e == cudaSuccess) e = cudaMallocHost((void**)&o->h_route, sizeof(int32_t) * MOE_MAX_TOPK);
  if (e == cudaSuccess) {
    o->layer_done.assign(n_layers, nullptr);
    o->layer_done_set.assign(n_layers, 0);
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l)
      e = cudaEventCreateWithFlags(&o->layer_done[l], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) {
    o->recency.assign(n_layers, std::vector<int>());
    o->slot_of.assign(n_layers, std::vector<int>(o->E, -1));
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
      for (int s = 0; s < o->slots && e == cudaSuccess; ++s) {  // slot s starts with expert s, expert 0 oldest
        o->recency[l].push_back(s);
        o->slot_of[l][s] = s;
        e = cudaMemcpyAsync(o->device_slots + ((size_t)l * o->slots + s) * slot_bytes,
                            host_experts[(size_t)l * o->E + s], slot_bytes, cudaMemcpyHostToDevice, o->copy_stream);
      }
      for (int x = 0; x < o->E; ++x) o->h_tables[(size_t)l * o->E + x] = o->slot_of[l][x];
    }
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(o->d_tables, o->h_tables, tb, cudaMemcpyHostToDevice, o->copy_stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(o->copy_stream);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    (void)cudaGetLastError();
    moe_offload_destroy(o);
    return MOE_ERR_CUDA;
  }
  *out = o;
  return MOE_OK;
}

int moe_offload_destroy(moe_offload* o) {
  if (!o) return MOE_ERR_INVALID_ARG;
  if (o->copy_stream) {
    cudaStreamSynchronize(o->copy_stream);
    cudaStreamDestroy(o->copy_stream);
  }
  if (o->ev_compute) cudaEventDestroy(o->ev_compute);
  if (o->ev_copy) cudaEventDestroy(o->ev_copy);
  for (cudaEvent_t ev : o->layer_done)
    if (ev) cudaEventDestroy(ev);
  if (o->d_tables) cudaFree(o->d_tables);
  if (o->h_tables) cudaFreeHost(o->h_tables);
  if (o->h_route) cudaFreeHost(o->h_route);
  (void)cudaGetLastError();
  delete o;
  return MOE_OK;
}

// by_layer_event: the caller is a stacked step, which records layer_done[layer] after the layer's kernels
static int ensure_impl(moe_offload* o, int32_t layer, const int32_t* sel, int32_t n, void* compute_stream,
                       bool by_layer_event) {
  if (!o || !sel || layer < 0 || layer >= o->n_layers || n <= 0 || n > o->slots) return MOE_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (sel[i] < 0 || sel[i] >= o->E) return MOE_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (sel[j] == sel[i]) return MOE_ERR_INVALID_ARG;
  }
  cudaStream_t cs = (cudaStream_t)compute_stream;
  std::vector<int>& rec = o->recency[layer];
  std::vector<int>& slot_of = o->slot_of[layer];
  bool waited = false, any = false;
  for (int i = 0; i < n; ++i) {
    const int e = sel[i];
    if (slot_of[e] >= 0) {
      o->hits++;
      for (size_t p = 0; p < rec.size(); ++p)
        if (rec[p] == e) {
          rec.erase(rec.begin() + p);
          break;
        }
      rec.push_back(e);
      continue;
    }
    int victim = -1;
    size_t vp = 0;
    for (size_t p = 0; p < rec.size() && victim < 0; ++p) {
      bool selected = false;
      for (int j = 0; j < n; ++j) selected |= (sel[j] == rec[p]);
      if (!selected) victim = rec[p], vp = p;
    }
    if (victim < 0) return MOE_ERR_STATE;
    if (!waited) {  // work already queued on the compute stream may still read the victim's slot
      if (by_layer_event && o->layer_done_set[layer]) {
        // the stacked steps record when a layer's kernels are done: only those read this layer's slots, so the
        // copy need not wait for the other layers' kernels queued since
        MOE_CUDA_TRY(cudaStreamWaitEvent(o->copy_stream, o->layer_done[layer], 0));
      } else {
        MOE_CUDA_TRY(cudaEventRecord(o->ev_compute, cs));
        MOE_CUDA_TRY(cudaStreamWaitEvent(o->copy_stream, o->ev_compute, 0));
      }
      waited = true;
    }
    const int slot = slot_of[victim];
    slot_of[victim] = -1;
    rec.erase(rec.begin() + vp);
    slot_of[e] = slot;
    rec.push_back(e);
    unsigned char* dst = o->device_slots + ((size_t)layer * o->slots + slot) * o->slot_bytes;
    const unsigned char* src = (const unsigned char*)o->host_experts[(size_t)layer * o->E + e];
    for (size_t off = 0; off < o->slot_bytes; off += kCopyChunk) {
      const size_t nb = o->slot_bytes - off < kCopyChunk ? o->slot_bytes - off : kCopyChunk;
      MOE_CUDA_TRY(cudaMemcpyAsync(dst + off, src + off, nb, cudaMemcpyHostToDevice, o->copy_stream));
    }
    o->fetches++;
    o->bytes += o->slot_bytes;
    any = true;
  }
  if (any) {
    SlotTable tab{};
    for (int x = 0; x < o->E; ++x) tab.slot[x] = slot_of[x];
    slot_table_kernel<<<1, MOE_MAX_EXPERTS, 0, o->copy_stream>>>(o->d_tables + (size_t)layer * o->E, o->E, tab);
    MOE_CUDA_TRY(cudaGetLastError());
    MOE_CUDA_TRY(cudaEventRecord(o->ev_copy, o->copy_stream));
    MOE_CUDA_TRY(cudaStreamWaitEvent(cs, o->ev_copy, 0));
  }
  return MOE_OK;
}

int moe_offload_ensure(moe_offload* o, int32_t layer, const int32_t* sel, int32_t n, void* compute_stream) {
  return ensure_impl(o, layer, sel, n, compute_stream, false);
}

int moe_offload_slot_table(moe_offload* o, int32_t layer, const int32_t** table) {
  if (!o || !table || layer < 0 || layer >= o->n_layers) return MOE_ERR_INVALID_ARG;
  *table = o->d_tables + (size_t)layer * o->E;
  return MOE_OK;
}

int moe_offload_resident(moe_offload* o, int32_t layer, int32_t* slots_host) {
  if (!o || !slots_host || layer < 0 || layer >= o->n_layers) return MOE_ERR_INVALID_ARG;
  for (int e = 0; e < o->E; ++e)
    if (o->slot_of[layer][e] >= 0) slots_host[o->slot_of[layer][e]] = e;
  return MOE_OK;
}

int moe_offload_stats(moe_offload* o, uint64_t* fetches, uint64_t* bytes, uint64_t* hits) {
  if (!o) return MOE_ERR_INVALID_ARG;
  if (fetches) *fetches = o->fetches;
  if (bytes) *bytes = o->bytes;
  if (hits) *hits = o->hits;
  return MOE_OK;
}

int moe_stack_decode_step(moe_offload* o, moe_ctx* ctx, const moe_weights* routers, float* h, int32_t* trace_host,
                          void* ws, size_t ws_bytes, void* stream) {
  if (!o || !ctx || !routers || !h || !ws) return MOE_ERR_INVALID_ARG;
  const moe_config& c = ctx->cfg;
  if (c.wd_rank != 0 || c.d_model != o->cfg.d_model || c.d_ff != o->cfg.d_ff || c.n_experts != o->E ||
      c.top_k != o->cfg.top_k)
    return MOE_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(c, 1);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  if ((size_t)c.d_ff * c.top_k * 2 < (size_t)c.d_model * 4) return MOE_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  char* wsb = (char*)ws;
  int32_t* idx = (int32_t*)(wsb + L.topk_idx);
  float* wt = (float*)(wsb + L.topk_w);
  void* u = wsb + L.hidden;               // the normalised input of the layer (x dtype; the region is >= 4*d bytes)
  void* y = wsb + L.out_slots;            // the layer's output (x dtype)
  const int d = c.d_model, k = c.top_k;
  const int xbf = c.x_dtype == MOE_BF16;
  for (int l = 0; l < o->n_layers; ++l) {
    rms_glue_kernel<<<1, 256, 0, s>>>(h, d, u, xbf);
    MOE_CUDA_TRY(cudaGetLastError());
    ctx->launches++;
    int rc = launch_route(ctx, u, 1, &routers[l], idx, wt, nullptr, s);
    if (rc != MOE_OK) return rc;
    // the host issues the copies, so it has to see the selection
    MOE_CUDA_TRY(cudaMemcpyAsync(o->h_route, idx, sizeof(int32_t) * k, cudaMemcpyDeviceToHost, s));
    MOE_CUDA_TRY(cudaStreamSynchronize(s));
    for (int j = 0; j < k; ++j) {
      if (trace_host) trace_host[(size_t)l * k + j] = o->h_route[j];
    }
    rc = ensure_impl(o, l, o->h_route, k, stream, true);
    if (rc != MOE_OK) return rc;
    moe_weights w = routers[l];
    w.gud = o->device_slots + (size_t)l * o->slots * o->slot_bytes;
    w.expert_slot = o->d_tables + (size_t)l * o->E;
    rc = launch_dense_stream(ctx, 2, u, 1, &w, idx, wt, nullptr, nullptr, y, nullptr, s);
    if (rc != MOE_OK) return rc;
    MOE_CUDA_TRY(cudaEventRecord(o->layer_done[l], s));
    o->layer_done_set[l] = 1;
    residual_kernel<<<(d + 255) / 256, 256, 0, s>>>(h, y, d, xbf);
    MOE_CUDA_TRY(cudaGetLastError());
    ctx->launches++;
  }
  return MOE_OK;
}

int moe_stack_decode_step_trace(moe_offload* o, moe_ctx* ctx, const moe_weights* routers, float* h,
                                const int32_t* sel_host, void* ws, size_t ws_bytes, void* stream) {
  if (!o || !ctx || !routers || !h || !ws || !sel_host) return MOE_ERR_INVALID_ARG;
  const moe_config& c = ctx->cfg;
  if (c.wd_rank != 0 || c.d_model != o->cfg.d_model || c.d_ff != o->cfg.d_ff || c.n_experts != o->E ||
      c.top_k != o->cfg.top_k)
    return MOE_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(c, 1);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  if ((size_t)c.d_ff * c.top_k * 2 < (size_t)c.d_model * 4 || (size_t)c.d_model * 2 < (size_t)c.n_experts * 4)
    return MOE_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  char* wsb = (char*)ws;
  int32_t* idx = (int32_t*)(wsb + L.topk_idx);
  float* wt = (float*)(wsb + L.topk_w);
  void* u = wsb + L.hidden;
  void* y = wsb + L.out_slots;
  float* probs = (float*)(wsb + L.xperm);  // [E] fp32; the region holds d bf16 values
  const int d = c.d_model, k = c.top_k;
  const int xbf = c.x_dtype == MOE_BF16;
  for (int l = 0; l < o->n_layers; ++l) {
    ForcedSel f{};
    for (int j = 0; j < k; ++j) f.e[j] = sel_host[(size_t)l * k + j];
    // the copies of this layer's misses are queued before its kernels: they run on the copy stream while the
    // compute stream is still busy with the layers before
    int rc = ensure_impl(o, l, f.e, k, stream, true);
    if (rc != MOE_OK) return rc;
    rms_glue_kernel<<<1, 256, 0, s>>>(h, d, u, xbf);
    MOE_CUDA_TRY(cudaGetLastError());
    rc = launch_route(ctx, u, 1, &routers[l], idx, wt, probs, s);
    if (rc != MOE_OK) return rc;
    forced_routing_kernel<<<1, 32, 0, s>>>(probs, k, c.renorm, f, idx, wt);
    MOE_CUDA_TRY(cudaGetLastError());
    moe_weights w = routers[l];
    w.gud = o->device_slots + (size_t)l * o->slots * o->slot_bytes;
    w.expert_slot = o->d_tables + (size_t)l * o->E;
    rc = launch_dense_stream(ctx, 2, u, 1, &w, idx, wt, nullptr, nullptr, y, nullptr, s);
    if (rc != MOE_OK) return rc;
    MOE_CUDA_TRY(cudaEventRecord(o->layer_done[l], s));
    o->layer_done_set[l] = 1;
    residual_kernel<<<(d + 255) / 256, 256, 0, s>>>(h, y, d, xbf);
    MOE_CUDA_TRY(cudaGetLastError());
    ctx->launches += 3;
  }
  // the per-layer staging of the slot tables is reused by the next step
  MOE_CUDA_TRY(cudaStreamSynchronize(s));
  return MOE_OK;
}

int moe_delta_uniform(const int32_t* trace, int32_t B, int32_t T, int32_t k, int32_t n_experts,
                      unsigned long long* counts_out, double* delta_out, unsigned long long* bad_out, void* stream) {
  if (!trace || !counts_out || !delta_out || !bad_out || B <= 0 || T <= 0 || k <= 0 || k > MOE_MAX_TOPK || n_experts <= 0 ||
      n_experts > MOE_MAX_EXPERTS || B > 1024)
    return MOE_ERR_INVALID_ARG;
  if ((long long)T * k >= (1ll << 32)) return MOE_ERR_UNSUPPORTED;  // 32-bit counters per CTA
  cudaStream_t s = (cudaStream_t)stream;
  MOE_CUDA_TRY(cudaMemsetAsync(bad_out, 0, sizeof(unsigned long long), s));
  expert_histogram_kernel<<<B, 256, 0, s>>>(trace, T, k, n_experts, counts_out, bad_out);
  MOE_CUDA_TRY(cudaGetLastError());
  delta_uniform_kernel<<<1, 256, 0, s>>>(counts_out, B, n_experts, delta_out);
  MOE_CUDA_TRY(cudaGetLastError());
  return MOE_OK;
}

int moe_expert_replacements(const int32_t* trace, int32_t B, int32_t T, int32_t k, int32_t n_experts,
                            unsigned long long* h_total_out, void* stream) {
  if (!trace || !h_total_out || B <= 0 || T <= 0 || k <= 0 || k > MOE_MAX_TOPK || n_experts <= 0)
    return MOE_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  MOE_CUDA_TRY(cudaMemsetAsync(h_total_out, 0, sizeof(unsigned long long), s));
  if (T < 2) return MOE_OK;
  const long long pairs = (long long)B * (T - 1);
  const int grid = (int)((pairs + 255) / 256 < 1184 ? (pairs + 255) / 256 : 1184);
  replacements_kernel<<<grid, 256, 0, s>>>(trace, B, T, k, n_experts, h_total_out);
  MOE_CUDA_TRY(cudaGetLastError());
  return MOE_OK;
}

}  // extern "C"
