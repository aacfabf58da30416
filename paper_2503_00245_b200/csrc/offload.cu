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
#include <algorithm>
#include <atomic>
#include <chrono>
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
  int32_t* h_route;                         // pinned, mapped: [0..k) the routing of the current layer, [k] its sequence number
  int32_t* h_route_dev;                     // the same memory as the device sees it
  int32_t route_seq;                        // sequence number the next routing kernel writes
  std::vector<cudaEvent_t> chunk_ev;        // one per chunk of the misses of a layer: recorded on the copy stream
  std::vector<int> chunk_row;               // a missing expert is copied (and computed) in runs of hidden units
  int n_chunks;                             // [chunk_row[c], chunk_row[c+1]): halves of what is left, so that few copies are
                                            // issued and the compute that trails the last one is short
  int fp8;                                  // the host copies are FP8 codes + row scales (half the link bytes)
  size_t blob_bytes;                        // bytes of one expert on the host: slot_bytes, or codes + scales
  unsigned char* staging;                   // device, fp8 only: [2][top_k] blobs as they arrive, before widening into the slot
                                            // (two sets, by layer parity: a layer's copies may run while the layer before is widened)
  cudaEvent_t staging_free[2];              // recorded on the compute stream after a set's last widening kernel
  char staging_used[2];
  uint64_t fetches, bytes, hits;
  // what the routed step spent where, summed over its calls (host wall time, seconds)
  double t_poll, t_issue;
  uint64_t polls;
};

namespace cosmoe {
namespace {

constexpr size_t kLastChunk = 4u << 20;  // a miss is copied in halves of what is left, down to about this size

// A layer's expert -> slot table, passed BY VALUE: every queued update carries its own copy, so a later call
// for the same layer cannot change what an earlier, still pending update writes.
struct SlotTable {
  int32_t slot[MOE_MAX_EXPERTS];
};
__global__ void slot_table_kernel(int32_t* __restrict__ table, int E, SlotTable t) {
  if ((int)threadIdx.x < E) table[threadIdx.x] = t.slot[threadIdx.x];
}

// Stacked decode, routed: u = h / rms(h) rounded to the type of x, the router on u (Eq. 2, Eq. 3), and the
// selection handed to the host through mapped pinned memory: the k expert ids, a system-scope fence, then the
// sequence number the host polls for.  One CTA; thread t takes the input features t, t + 256, ...
constexpr int kRouteThreads = 256;
constexpr int kRouteFeat = 8;  // features per thread: d <= 2048
__global__ void __launch_bounds__(kRouteThreads)
    rms_route_kernel(const float* __restrict__ h, int d, int E, int k, int renorm, const uint16_t* __restrict__ w_router,
                     const float* __restrict__ bias, void* __restrict__ u, int x_is_bf16, int32_t* __restrict__ idx,
                     float* __restrict__ wt, volatile int32_t* __restrict__ host_route, int32_t seq) {
  __shared__ float s_sum[kRouteThreads / 32];
  __shared__ float s_log[kRouteThreads / 32][MOE_MAX_EXPERTS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float hv[kRouteFeat], ss = 0.f;
#pragma unroll
  for (int j = 0; j < kRouteFeat; ++j) {
    const int i = tid + j * kRouteThreads;
    hv[j] = i < d ? h[i] : 0.f;
    ss = fmaf(hv[j], hv[j], ss);
  }
  ss = warp_sum(ss);
  if (lane == 0) s_sum[warp] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < kRouteThreads / 32; ++w) tot += s_sum[w];
  const float inv = rsqrtf(tot / (float)d);
#pragma unroll
  for (int j = 0; j < kRouteFeat; ++j) {
    const int i = tid + j * kRouteThreads;
    float v = hv[j] * inv;
    if (x_is_bf16) {
      const __nv_bfloat16 b = __float2bfloat16_rn(v);
      if (i < d) reinterpret_cast<__nv_bfloat16*>(u)[i] = b;
      v = __bfloat162float(b);  // the router sees what the experts see
    } else if (i < d) {
      reinterpret_cast<float*>(u)[i] = v;
    }
    hv[j] = i < d ? v : 0.f;
  }
  for (int e0 = 0; e0 < E; e0 += 8) {
    float a[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) a[q] = 0.f;
    if ((E & 7) == 0) {
#pragma unroll
      for (int j = 0; j < kRouteFeat; ++j) {
        const int i = min(tid + j * kRouteThreads, d - 1);
        float w[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(w_router + (size_t)i * E + e0)), w);
#pragma unroll
        for (int q = 0; q < 8; ++q) a[q] = fmaf(hv[j], w[q], a[q]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < kRouteFeat; ++j) {
        const int i = min(tid + j * kRouteThreads, d - 1);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (e0 + q < E) a[q] = fmaf(hv[j], bf16_to_float(__ldg(w_router + (size_t)i * E + e0 + q)), a[q]);
      }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float t = warp_sum(a[q]);
      if (lane == 0 && e0 + q < E) s_log[warp][e0 + q] = t;
    }
  }
  __syncthreads();
  if (warp != 0) return;
  float l0 = 0.f, l1 = 0.f;
  if (lane < E) {
    for (int w = 0; w < kRouteThreads / 32; ++w) l0 += s_log[w][lane];
    if (bias) l0 += bias[lane];
  }
  if (lane + 32 < E) {
    for (int w = 0; w < kRouteThreads / 32; ++w) l1 += s_log[w][lane + 32];
    if (bias) l1 += bias[lane + 32];
  }
  warp_route_finish(l0, l1, E, k, renorm, lane, idx, wt, nullptr);
  __syncwarp();
  if (lane < k) host_route[lane] = idx[lane];
  __threadfence_system();
  __syncwarp();
  if (lane == 0) host_route[k] = seq;
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

static int offload_create(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                          const void* const* host_experts, void* device_slots, size_t slot_bytes, int fp8, moe_offload** out);

int moe_offload_create(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                       const void* const* host_experts, void* device_slots, size_t slot_bytes, moe_offload** out) {
  return offload_create(cfg, n_layers, slots_per_layer, host_experts, device_slots, slot_bytes, 0, out);
}

int moe_offload_create_fp8(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                           const void* const* host_blobs, void* device_slots, size_t slot_bytes, moe_offload** out) {
  return offload_create(cfg, n_layers, slots_per_layer, host_blobs, device_slots, slot_bytes, 1, out);
}

// Copy of one expert's rows [r0, r1) from the host, on the copy stream.  bf16 host copies go straight into the
// device slot.  FP8 blobs (codes [f][3][d], then scales [f][3]) land in the staging area of miss number `m` of the
// layer (set layer & 1); widen_rows turns them into the slot's bf16 rows on whatever stream the caller orders
// behind the copy -- the compute stream in the stacked steps, so that the copy stream only ever copies.
static unsigned char* staging_of(moe_offload* o, int layer, int m) {
  return o->staging + ((size_t)(layer & 1) * o->cfg.top_k + m) * o->blob_bytes;
}
static int queue_rows(moe_offload* o, int layer, int e, int slot, int m, int r0, int r1) {
  const size_t d = (size_t)o->cfg.d_model, f = (size_t)o->cfg.d_ff;
  const unsigned char* src = (const unsigned char*)o->host_experts[(size_t)layer * o->E + e];
  if (!o->fp8) {
    unsigned char* dst = o->device_slots + ((size_t)layer * o->slots + slot) * o->slot_bytes;
    const size_t row_bytes = 3 * d * 2;
    MOE_CUDA_TRY(cudaMemcpyAsync(dst + (size_t)r0 * row_bytes, src + (size_t)r0 * row_bytes, (size_t)(r1 - r0) * row_bytes,
                                 cudaMemcpyHostToDevice, o->copy_stream));
    return MOE_OK;
  }
  unsigned char* stg = staging_of(o, layer, m);
  const size_t codes_bytes = f * 3 * d;
  if (r0 == 0)  // the scales of the whole expert go first (12 f bytes)
    MOE_CUDA_TRY(cudaMemcpyAsync(stg + codes_bytes, src + codes_bytes, f * 3 * sizeof(float), cudaMemcpyHostToDevice, o->copy_stream));
  MOE_CUDA_TRY(cudaMemcpyAsync(stg + (size_t)r0 * 3 * d, src + (size_t)r0 * 3 * d, (size_t)(r1 - r0) * 3 * d, cudaMemcpyHostToDevice,
                               o->copy_stream));
  return MOE_OK;
}
static int widen_rows(moe_offload* o, int layer, int slot, int m, int r0, int r1, cudaStream_t s) {
  if (!o->fp8) return MOE_OK;
  const size_t d = (size_t)o->cfg.d_model, f = (size_t)o->cfg.d_ff;
  unsigned char* stg = staging_of(o, layer, m);
  unsigned char* dst = o->device_slots + ((size_t)layer * o->slots + slot) * o->slot_bytes;
  return launch_fp8_dequant(stg + (size_t)r0 * 3 * d, reinterpret_cast<const float*>(stg + f * 3 * d) + (size_t)r0 * 3,
                            (long long)(r1 - r0) * 3, (int)d, dst + (size_t)r0 * 3 * d * 2, s);
}
// The staging set of `layer` is free again once the widening kernels queued on `s` so far have run.
static int staging_release(moe_offload* o, int layer, cudaStream_t s) {
  if (!o->fp8) return MOE_OK;
  MOE_CUDA_TRY(cudaEventRecord(o->staging_free[layer & 1], s));
  o->staging_used[layer & 1] = 1;
  return MOE_OK;
}

static int offload_create(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                          const void* const* host_experts, void* device_slots, size_t slot_bytes, int fp8, moe_offload** out) {
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
  o->fp8 = fp8, o->staging = nullptr;
  o->staging_free[0] = o->staging_free[1] = nullptr, o->staging_used[0] = o->staging_used[1] = 0;
  o->blob_bytes = fp8 ? (size_t)cfg->d_ff * 3 * cfg->d_model + (size_t)cfg->d_ff * 3 * sizeof(float) : slot_bytes;
  o->copy_stream = nullptr, o->ev_compute = nullptr, o->ev_copy = nullptr;
  o->d_tables = nullptr, o->h_tables = nullptr, o->h_route = nullptr, o->h_route_dev = nullptr;
  o->route_seq = 0, o->t_poll = o->t_issue = 0.0, o->polls = 0;
  {
    const size_t row_bytes = (size_t)3 * cfg->d_model * 2;
    const int min_rows = (int)std::max<size_t>(1, kLastChunk / row_bytes);
    o->chunk_row.assign(1, 0);
    for (int left = cfg->d_ff; left > 0;) {
      const int take = left <= 2 * min_rows ? left : left / 2;
      o->chunk_row.push_back(o->chunk_row.back() + take);
      left -= take;
    }
    o->n_chunks = (int)o->chunk_row.size() - 1;
  }
  const size_t tb = (size_t)n_layers * o->E * sizeof(int32_t);
  cudaError_t e = cudaStreamCreateWithFlags(&o->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&o->ev_compute, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&o->ev_copy, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMalloc((void**)&o->d_tables, tb);
  if (e == cudaSuccess) e = cudaMallocHost((void**)&o->h_tables, tb);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&o->h_route, sizeof(int32_t) * (MOE_MAX_TOPK + 1), cudaHostAllocMapped);
  if (e == cudaSuccess) {
    for (int j = 0; j <= MOE_MAX_TOPK; ++j) o->h_route[j] = -1;
    e = cudaHostGetDevicePointer((void**)&o->h_route_dev, o->h_route, 0);
  }
  if (e == cudaSuccess) {
    o->chunk_ev.assign((size_t)cfg->top_k * o->n_chunks, nullptr);
    for (size_t i = 0; i < o->chunk_ev.size() && e == cudaSuccess; ++i)
      e = cudaEventCreateWithFlags(&o->chunk_ev[i], cudaEventDisableTiming);
  }
  if (e == cudaSuccess && fp8) e = cudaMalloc((void**)&o->staging, (size_t)2 * cfg->top_k * o->blob_bytes);
  for (int i = 0; i < 2 && e == cudaSuccess && fp8; ++i) e = cudaEventCreateWithFlags(&o->staging_free[i], cudaEventDisableTiming);
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
        if (queue_rows(o, l, s, s, 0, 0, cfg->d_ff) != MOE_OK || widen_rows(o, l, s, 0, 0, cfg->d_ff, o->copy_stream) != MOE_OK)
          e = cudaErrorUnknown;
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
  for (cudaEvent_t ev : o->chunk_ev)
    if (ev) cudaEventDestroy(ev);
  if (o->staging) cudaFree(o->staging);
  for (int i = 0; i < 2; ++i)
    if (o->staging_free[i]) cudaEventDestroy(o->staging_free[i]);
  if (o->d_tables) cudaFree(o->d_tables);
  if (o->h_tables) cudaFreeHost(o->h_tables);
  if (o->h_route) cudaFreeHost(o->h_route);
  (void)cudaGetLastError();
  delete o;
  return MOE_OK;
}

// What a layer has to do for one step's selection: per selected expert its slot and whether it must be fetched.
struct LayerPlan {
  int n, n_miss;
  int e[MOE_MAX_TOPK], slot[MOE_MAX_TOPK];
  bool miss[MOE_MAX_TOPK];
};

// Bookkeeping only (host integers): hits touch the recency list, a miss takes the slot of the least recently
// used resident expert that is not selected in this step.  Nothing is queued.
static int plan_layer(moe_offload* o, int32_t layer, const int32_t* sel, int32_t n, LayerPlan& pl) {
  if (!o || !sel || layer < 0 || layer >= o->n_layers || n <= 0 || n > o->slots || n > MOE_MAX_TOPK) return MOE_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (sel[i] < 0 || sel[i] >= o->E) return MOE_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (sel[j] == sel[i]) return MOE_ERR_INVALID_ARG;
  }
  std::vector<int>& rec = o->recency[layer];
  std::vector<int>& slot_of = o->slot_of[layer];
  pl.n = n, pl.n_miss = 0;
  for (int i = 0; i < n; ++i) {
    const int e = sel[i];
    pl.e[i] = e;
    if (slot_of[e] >= 0) {
      o->hits++;
      for (size_t p = 0; p < rec.size(); ++p)
        if (rec[p] == e) {
          rec.erase(rec.begin() + p);
          break;
        }
      rec.push_back(e);
      pl.slot[i] = slot_of[e], pl.miss[i] = false;
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
    const int slot = slot_of[victim];
    slot_of[victim] = -1;
    rec.erase(rec.begin() + vp);
    slot_of[e] = slot;
    rec.push_back(e);
    pl.slot[i] = slot, pl.miss[i] = true, pl.n_miss++;
    o->fetches++;
    o->bytes += o->blob_bytes;
  }
  return MOE_OK;
}

// Work already queued on the compute stream may still read the victims' slots: the copy stream waits for it.
// by_layer_event: the caller is a stacked step, which records layer_done[layer] after the layer's kernels -- only
// those read this layer's slots, so the copies need not wait for the other layers' kernels queued since.
static int copies_wait_for_readers(moe_offload* o, int32_t layer, cudaStream_t cs, bool by_layer_event) {
  if (o->fp8 && o->staging_used[layer & 1])  // the staging set's last contents have been widened
    MOE_CUDA_TRY(cudaStreamWaitEvent(o->copy_stream, o->staging_free[layer & 1], 0));
  if (by_layer_event && o->layer_done_set[layer]) {
    MOE_CUDA_TRY(cudaStreamWaitEvent(o->copy_stream, o->layer_done[layer], 0));
  } else {
    MOE_CUDA_TRY(cudaEventRecord(o->ev_compute, cs));
    MOE_CUDA_TRY(cudaStreamWaitEvent(o->copy_stream, o->ev_compute, 0));
  }
  return MOE_OK;
}

// The layer's device table, rewritten in copy-stream order from a by-value copy of the host's bookkeeping.
static int queue_table_update(moe_offload* o, int32_t layer) {
  SlotTable tab{};
  for (int x = 0; x < o->E; ++x) tab.slot[x] = o->slot_of[layer][x];
  slot_table_kernel<<<1, MOE_MAX_EXPERTS, 0, o->copy_stream>>>(o->d_tables + (size_t)layer * o->E, o->E, tab);
  MOE_CUDA_TRY(cudaGetLastError());
  return MOE_OK;
}

static int ensure_impl(moe_offload* o, int32_t layer, const int32_t* sel, int32_t n, void* compute_stream,
                       bool by_layer_event, LayerPlan* plan_out = nullptr) {
  LayerPlan pl;
  int rc = plan_layer(o, layer, sel, n, pl);
  if (rc != MOE_OK) return rc;
  if (plan_out) *plan_out = pl;
  if (pl.n_miss == 0) return MOE_OK;
  cudaStream_t cs = (cudaStream_t)compute_stream;
  if ((rc = copies_wait_for_readers(o, layer, cs, by_layer_event)) != MOE_OK) return rc;
  for (int i = 0, m = 0; i < n; ++i) {
    if (!pl.miss[i]) continue;
    for (int cch = 0; cch < o->n_chunks; ++cch)
      if ((rc = queue_rows(o, layer, pl.e[i], pl.slot[i], m, o->chunk_row[cch], o->chunk_row[cch + 1])) != MOE_OK) return rc;
    ++m;
  }
  if ((rc = queue_table_update(o, layer)) != MOE_OK) return rc;
  MOE_CUDA_TRY(cudaEventRecord(o->ev_copy, o->copy_stream));
  MOE_CUDA_TRY(cudaStreamWaitEvent(cs, o->ev_copy, 0));
  for (int i = 0, m = 0; i < n; ++i) {  // 8-bit host copies: widened on the compute stream, behind the copies
    if (!pl.miss[i]) continue;
    if ((rc = widen_rows(o, layer, pl.slot[i], m, 0, o->cfg.d_ff, cs)) != MOE_OK) return rc;
    ++m;
  }
  return staging_release(o, layer, cs);
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

static int check_stack_args(moe_offload* o, moe_ctx* ctx, size_t ws_bytes) {
  const moe_config& c = ctx->cfg;
  if (c.wd_rank != 0 || c.d_model != o->cfg.d_model || c.d_ff != o->cfg.d_ff || c.n_experts != o->E ||
      c.top_k != o->cfg.top_k)
    return MOE_ERR_INVALID_ARG;
  if (c.d_model > kRouteThreads * kRouteFeat || c.d_model > kDenseStreamMaxD) return MOE_ERR_UNSUPPORTED;
  if (ws_bytes < ws_layout(c, 1).total) return MOE_ERR_WORKSPACE;
  if ((size_t)c.d_ff * c.top_k * 2 < (size_t)c.d_model * 4) return MOE_ERR_UNSUPPORTED;  // u lives in the hidden region
  return MOE_OK;
}

int moe_stack_decode_step(moe_offload* o, moe_ctx* ctx, const moe_weights* routers, float* h, int32_t* trace_host,
                          void* ws, size_t ws_bytes, void* stream) {
  if (!o || !ctx || !routers || !h || !ws) return MOE_ERR_INVALID_ARG;
  int rc = check_stack_args(o, ctx, ws_bytes);
  if (rc != MOE_OK) return rc;
  const moe_config& c = ctx->cfg;
  const WsLayout L = ws_layout(c, 1);
  cudaStream_t s = (cudaStream_t)stream;
  char* wsb = (char*)ws;
  int32_t* idx = (int32_t*)(wsb + L.topk_idx);
  float* wt = (float*)(wsb + L.topk_w);
  void* u = wsb + L.hidden;  // the normalised input of the layer (x dtype)
  const int d = c.d_model, k = c.top_k;
  const int xbf = c.x_dtype == MOE_BF16;
  using clk = std::chrono::steady_clock;
  for (int l = 0; l < o->n_layers; ++l) {
    // (1) u = h / rms(h), router, selection -> device buffers and the host's mapped words
    const int32_t seq = ++o->route_seq;
    rms_route_kernel<<<1, kRouteThreads, 0, s>>>(h, d, o->E, k, c.renorm, (const uint16_t*)routers[l].w_router,
                                                 routers[l].b_router, u, xbf, idx, wt, o->h_route_dev, seq);
    MOE_CUDA_TRY(cudaGetLastError());
    ctx->launches++;
    // (2) the host must see the selection before it can queue the copies: it polls the sequence word (bounded)
    const clk::time_point t0 = clk::now();
    volatile int32_t* hr = o->h_route;
    for (unsigned spin = 0; hr[k] != seq; ++spin) {
      if ((spin & 1023u) == 1023u) {
        if (cudaStreamQuery(s) != cudaErrorNotReady && hr[k] != seq) {  // the stream drained (or failed) without the word
          (void)cudaGetLastError();
          return MOE_ERR_STATE;
        }
        if (std::chrono::duration<double>(clk::now() - t0).count() > 10.0) return MOE_ERR_TIMEOUT;
      }
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    int32_t sel[MOE_MAX_TOPK];
    for (int j = 0; j < k; ++j) {
      sel[j] = hr[j];
      if (trace_host) trace_host[(size_t)l * k + j] = sel[j];
    }
    const clk::time_point t1 = clk::now();
    o->t_poll += std::chrono::duration<double>(t1 - t0).count();
    o->polls++;
    // (3) bookkeeping; the copies of the misses go out first, chunk by chunk, each chunk with its own event
    LayerPlan pl;
    if ((rc = plan_layer(o, l, sel, k, pl)) != MOE_OK) return rc;
    unsigned hit_mask = 0;
    int last_miss = -1;
    for (int j = 0; j < k; ++j) {
      if (pl.miss[j])
        last_miss = j;
      else
        hit_mask |= 1u << j;
    }
    if (pl.n_miss) {
      if ((rc = copies_wait_for_readers(o, l, s, true)) != MOE_OK) return rc;
      int m = 0;
      for (int j = 0; j < k; ++j) {
        if (!pl.miss[j]) continue;
        for (int cch = 0; cch < o->n_chunks; ++cch) {
          if ((rc = queue_rows(o, l, pl.e[j], pl.slot[j], m, o->chunk_row[cch], o->chunk_row[cch + 1])) != MOE_OK) return rc;
          MOE_CUDA_TRY(cudaEventRecord(o->chunk_ev[(size_t)m * o->n_chunks + cch], o->copy_stream));
        }
        ++m;
      }
      if ((rc = queue_table_update(o, l)) != MOE_OK) return rc;
    }
    // (4) the resident selected experts run while the missing ones are on their way; a missing expert is
    // consumed chunk by chunk, each launch waiting only for its own chunk's copy.  Every launch adds into the
    // same fixed-point accumulators; the last one converts them and adds the layer's output to h.
    moe_weights w = routers[l];
    w.gud = o->device_slots + (size_t)l * o->slots * o->slot_bytes;
    w.expert_slot = nullptr;
    DenseExtra ex{};
    for (int j = 0; j < MOE_MAX_TOPK; ++j) ex.slot_of_entry[j] = j < k ? pl.slot[j] : -1;
    ex.resid = h;
    if (hit_mask) {
      ex.sel_mask = hit_mask, ex.unit_lo = 0, ex.unit_cnt = 0, ex.finalize = pl.n_miss == 0;
      if ((rc = launch_dense_stream(ctx, 2, u, 1, &w, idx, wt, nullptr, nullptr, nullptr, nullptr, s, &ex)) != MOE_OK) return rc;
    }
    int m = 0;
    for (int j = 0; j < k; ++j) {
      if (!pl.miss[j]) continue;
      for (int cch = 0; cch < o->n_chunks; ++cch) {
        const int r0 = o->chunk_row[cch], r1 = o->chunk_row[cch + 1];
        MOE_CUDA_TRY(cudaStreamWaitEvent(s, o->chunk_ev[(size_t)m * o->n_chunks + cch], 0));
        if ((rc = widen_rows(o, l, pl.slot[j], m, r0, r1, s)) != MOE_OK) return rc;
        ex.sel_mask = 1u << j, ex.unit_lo = r0, ex.unit_cnt = r1 - r0;
        ex.finalize = (j == last_miss && cch == o->n_chunks - 1) ? 1 : 0;
        if ((rc = launch_dense_stream(ctx, 2, u, 1, &w, idx, wt, nullptr, nullptr, nullptr, nullptr, s, &ex)) != MOE_OK) return rc;
      }
      ++m;
    }
    if (pl.n_miss && (rc = staging_release(o, l, s)) != MOE_OK) return rc;
    MOE_CUDA_TRY(cudaEventRecord(o->layer_done[l], s));
    o->layer_done_set[l] = 1;
    o->t_issue += std::chrono::duration<double>(clk::now() - t1).count();
  }
  return MOE_OK;
}

int moe_stack_decode_step_trace(moe_offload* o, moe_ctx* ctx, const moe_weights* routers, float* h,
                                const int32_t* sel_host, void* ws, size_t ws_bytes, void* stream) {
  if (!o || !ctx || !routers || !h || !ws || !sel_host) return MOE_ERR_INVALID_ARG;
  int rc = check_stack_args(o, ctx, ws_bytes);
  if (rc != MOE_OK) return rc;
  const moe_config& c = ctx->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  const int k = c.top_k;
  for (int l = 0; l < o->n_layers; ++l) {
    // the copies of this layer's misses are queued before its kernel: they run on the copy stream while the
    // compute stream is still busy with the layers before
    LayerPlan pl;
    rc = ensure_impl(o, l, sel_host + (size_t)l * k, k, stream, true, &pl);
    if (rc != MOE_OK) return rc;
    // the whole layer is one launch: u = h / rms(h), the router's probabilities of the prescribed experts, the
    // experts, h += y
    moe_weights w = routers[l];
    w.gud = o->device_slots + (size_t)l * o->slots * o->slot_bytes;
    w.expert_slot = nullptr;
    DenseExtra ex{};
    for (int j = 0; j < MOE_MAX_TOPK; ++j) ex.slot_of_entry[j] = j < k ? pl.slot[j] : -1, ex.forced[j] = j < k ? pl.e[j] : 0;
    ex.finalize = 1, ex.resid = h, ex.h_in = h, ex.use_forced = 1;
    rc = launch_dense_stream(ctx, 0, h, 1, &w, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, s, &ex);
    if (rc != MOE_OK) return rc;
    MOE_CUDA_TRY(cudaEventRecord(o->layer_done[l], s));
    o->layer_done_set[l] = 1;
  }
  return MOE_OK;
}

int moe_offload_host_times(moe_offload* o, double* poll_s, double* issue_s, uint64_t* polls) {
  if (!o) return MOE_ERR_INVALID_ARG;
  if (poll_s) *poll_s = o->t_poll;
  if (issue_s) *issue_s = o->t_issue;
  if (polls) *polls = o->polls;
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
