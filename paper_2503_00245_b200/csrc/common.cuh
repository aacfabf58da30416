// Shared host/device helpers for the MoE layer kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cosmoe.h"

namespace cosmoe {

// ------------------------------------------------------------------ host side
extern thread_local int g_last_cuda_error;

#define MOE_CUDA_TRY(expr)                   \
  do {                                       \
    cudaError_t _e = (expr);                 \
    if (_e != cudaSuccess) {                 \
      ::cosmoe::g_last_cuda_error = (int)_e; \
      (void)cudaGetLastError();              \
      return MOE_ERR_CUDA;                   \
    }                                        \
  } while (0)

// Device-resident state of a ctx: status word written by kernels, grid barrier.
struct DeviceState {
  unsigned int status;  // 0 ok, else moe_status
  unsigned int detail;  // where it happened (kernel-specific code)
  unsigned int pad0[30];
  unsigned int bar_count;  // arrivals at the current grid barrier (own 128-byte line: it takes the atomics)
  unsigned int pad1[31];
  unsigned int bar_gen;  // generation, bumped by the last arriver (own line: it takes the polling)
  unsigned int pad2[31];
  // dense streaming path: CTAs that have added their partial outputs, over all launches since the state was last
  // cleared (never reset by the kernels: a launch's arrivals are numbered by the remainder modulo its grid size)
  unsigned long long done_total;
  // weight-decomposed decode kernel: arrivals at its meetings between the products, counted the same way
  unsigned long long phase_total;
  // dense streaming kernel, one token: next stage (4 hidden units) of each active expert that no CTA has taken yet;
  // the finalisers leave zeros
  unsigned int stage_ctr[MOE_MAX_TOPK];
  // dense streaming kernel, one token: added to the arrivals an accumulator word waits for (0; the diagnostics
  // hook sets 1, so that the wait runs out)
  unsigned int tail_bias;
  unsigned int pad3[19];
};

}  // namespace cosmoe

struct moe_ctx {
  moe_config cfg;
  int device;
  int sm_count;
  int max_smem_optin;
  cosmoe::DeviceState* d_state;  // device
  cosmoe::DeviceState* h_state;  // pinned host mirror for moe_check
  long long* acc;                // device: fixed-point output accumulators of the dense streaming path, kept zero
  size_t acc_elems;              //         between calls by the kernel itself (MOE_STREAM_MAX_TOKENS*top_k*d)
  unsigned long long launches;
  long long fin_wait_budget;     // cycles the dense streaming kernel's finalisers wait for the arrival counter (0 = default)
};

namespace cosmoe {

// Offsets (bytes) of the pieces of the caller's scratch buffer.
struct WsLayout {
  size_t topk_idx, topk_w, offsets, perm, inv;  // routing products when the caller does not ask for them
  size_t vec_a, vec_b, vec_c;                   // fp32 inter-phase vectors of the streaming path
  size_t xperm, hidden, mid_a, mid_b;           // bf16 operands of the tensor path
  size_t out_slots;                             // fp32 [T*k][d]
  size_t total;
};
WsLayout ws_layout(const moe_config& c, int T);

int validate_config(const moe_config* c);

// launchers implemented in the other translation units
int launch_route(moe_ctx* ctx, const void* x, int T, const moe_weights* w, int32_t* idx, float* wt, float* probs,
                 cudaStream_t s);
int launch_permute(moe_ctx* ctx, const int32_t* idx, int T, int32_t* offsets, int32_t* perm, int32_t* inv,
                   cudaStream_t s);
// out_slots may come as `planes` partial sums, one [T*k][d] plane after the other (summed in order).
constexpr int kDenseStreamMaxD = 2048;  // widest d_model the dense streaming kernel handles (token row in registers)
constexpr int kKSplitMax = 4;          // planes the tensor path may ask for ...
constexpr int kKSplitMaxSlots = 2048;  // ... when there are at most this many (token, choice) slots
int launch_combine(moe_ctx* ctx, const float* out_slots, const float* wt, const int32_t* inv, int T, void* y,
                   int planes, cudaStream_t s);
int launch_gather_rows(moe_ctx* ctx, const void* x, const int32_t* perm, int n_slots, void* xperm, cudaStream_t s);

// Streaming (decode) path.  mode 0: whole layer from topk (writes y); mode 1: FFN per slot from
// expert_offsets/perm (writes out_slots).
// Batch-1 decode with weight-decomposed experts in one launch (router included); t, h, vpart: fp32 scratch of
// k*2r, k*f and k*r*8 values.
bool wd_decode_applies(const moe_config& c, int T);
int launch_wd_decode(moe_ctx* ctx, const void* x, const moe_weights* w, int32_t* topk_idx, float* topk_w, void* y,
                     float* t, float* h, float* vpart, cudaStream_t s);
int launch_stream_ffn(moe_ctx* ctx, int mode, const void* x, int T, const moe_weights* w, const int32_t* topk_idx,
                      const float* topk_w, const int32_t* offsets, const int32_t* perm, void* y, float* out_slots,
                      char* ws, const WsLayout& L, cudaStream_t s);
// Dense experts, streaming path, one kernel (router fused when T == 1 and mode == 0; mode 2 = mode 0 with the
// routing always taken from topk_idx / topk_w).
// Optional extras of a single-token launch of the dense streaming kernel (the stacked decode steps use them).
struct DenseExtra {
  unsigned sel_mask;                 // routing given: which of the k routing entries this launch computes (0 = all)
  int slot_of_entry[MOE_MAX_TOPK];   // slot of the packed array that holds routing entry j's expert (-1: expert_slot table)
  int unit_lo, unit_cnt;             // hidden units [unit_lo, unit_lo + unit_cnt) of every expert only (unit_cnt 0 = all)
  int finalize;                      // 0: leave the partial sums in the accumulators for a later launch of the group
  float* resid;                      // fp32 [d]: the finalisers add the layer's output to it (h += y) instead of writing y
  const float* h_in;                 // fp32 [d]: the layer input is h / rms(h), computed in the prologue (router fused)
  int use_forced;                    // router fused: the expert set is prescribed, the gate weights are its probabilities
  int forced[MOE_MAX_TOPK];
};
bool dense_stream_fuses_route(const moe_config& c, int T);  // mode 0 computes the routing itself (else: run launch_route first)
int launch_dense_stream(moe_ctx* ctx, int mode, const void* x, int T, const moe_weights* w, int32_t* topk_idx,
                        float* topk_w, const int32_t* offsets, const int32_t* perm, void* y, float* out_slots,
                        cudaStream_t s, const DenseExtra* ex = nullptr);
// FP8 E4M3 codes with one fp32 scale per row of n values -> bf16 (csrc/fp8_store.cu).
int launch_fp8_dequant(const void* codes, const float* scales, long long rows, int n, void* w, cudaStream_t s);
// Tensor-core (prefill) path: out_slots from x gathered by perm.
int launch_tensor_ffn(moe_ctx* ctx, const void* x, int T, const moe_weights* w, const int32_t* offsets,
                      const int32_t* perm, char* ws, const WsLayout& L, float* out_slots, int* out_planes,
                      cudaStream_t s);

// ------------------------------------------------------------------ device side
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Longest any device-side wait may last before the kernel gives up and flags MOE_ERR_TIMEOUT,
// in SM clock cycles (about two seconds at the boost clock).  clock64() is used because it is cheap to
// read; %globaltimer is not.
constexpr long long kWaitBudgetCycles = 4000000000ll;

__device__ __forceinline__ void flag_error(DeviceState* st, unsigned code, unsigned detail) {
  if (atomicCAS(&st->status, 0u, code) == 0u) st->detail = detail;
}

// ---- programmatic dependent launch ---------------------------------------------------------------
// A kernel launched with launch_pdl may be scheduled while its predecessor in the stream is still running;
// it must not touch anything the predecessor reads or writes before pdl_wait(), which returns once the
// predecessor has completed and its writes are visible.  (Without the launch attribute both are no-ops.)
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t lc{};
  lc.gridDim = grid, lc.blockDim = block, lc.dynamicSmemBytes = smem, lc.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr, lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

// ---- mbarrier -----------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the budget ran out (the barrier never completed its phase).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > kWaitBudgetCycles) return false;
  }
}

// Same contract, but polls with the non-blocking test_wait: the waiter is never parked by the hardware.
// For short waits between warps of one CTA.
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_spin(uint64_t* bar, uint32_t parity) {
  if (mbar_test_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 1024; ++i)
      if (mbar_test_wait(bar, parity)) return true;
    if (clock64() - t0 > kWaitBudgetCycles) return false;
  }
}

// ---- bulk asynchronous copy global -> shared (TMA, no tensor map) ---------------
// src and dst 16-byte aligned, bytes a multiple of 16.  Completion is counted on `bar`.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst_smem)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// Same, with an L2 eviction-priority hint: evict_first for data that is read exactly once (streamed weights),
// so that it does not push the small reused operands out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::
          "r"(smem_u32(dst_smem)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// ---- acquire / release on global words -------------------------------------------
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_relaxed(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long atom_add_acq_rel64(unsigned long long* p, unsigned long long v) {
  unsigned long long old;
  asm volatile("atom.acq_rel.gpu.global.add.u64 %0, [%1], %2;" : "=l"(old) : "l"(p), "l"(v) : "memory");
  return old;
}
__device__ __forceinline__ unsigned atom_add_acq_rel(unsigned* p, unsigned v) {
  unsigned old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}

// Barrier over all CTAs of a co-resident (cooperative) grid.  Thread 0 of each CTA arrives; the
// wait is bounded.  Returns false (for the whole CTA) when the budget ran out.
__device__ __forceinline__ bool grid_barrier(DeviceState* st, unsigned n_ctas, int* smem_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    const unsigned gen = ld_acquire(&st->bar_gen);
    __threadfence();
    const unsigned old = atom_add_acq_rel(&st->bar_count, 1u);
    if (old == n_ctas - 1u) {
      st->bar_count = 0u;
      __threadfence();
      st_release(&st->bar_gen, gen + 1u);
    } else {
      const long long t0 = clock64();
      unsigned spins = 0;
      while (ld_acquire(&st->bar_gen) == gen) {
        if ((++spins & 255u) == 0u && clock64() - t0 > kWaitBudgetCycles) {
          ok = 0;
          break;
        }
      }
    }
    __threadfence();
    *smem_flag = ok;
  }
  __syncthreads();
  return *smem_flag != 0;
}

// ---- bf16 helpers ---------------------------------------------------------------------
// 8 bf16 packed in a uint4 -> 8 floats (exact).
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  f[0] = __uint_as_float(v.x << 16);
  f[1] = __uint_as_float(v.x & 0xffff0000u);
  f[2] = __uint_as_float(v.y << 16);
  f[3] = __uint_as_float(v.y & 0xffff0000u);
  f[4] = __uint_as_float(v.z << 16);
  f[5] = __uint_as_float(v.z & 0xffff0000u);
  f[6] = __uint_as_float(v.w << 16);
  f[7] = __uint_as_float(v.w & 0xffff0000u);
}
__device__ __forceinline__ float bf16_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

// fp32 -> unsigned key with the same order (-0 counts as +0; NaN is not ordered), and back
__device__ __forceinline__ unsigned f32_key(float v) {
  const unsigned b = __float_as_uint(v + 0.0f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float f32_unkey(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

// Softmax over E logits (Eq. 2), top-k (Eq. 3) and gate weights by one warp: lane l holds logit l (l0)
// and logit l + 32 (l1).  Selection runs on the logits (softmax is monotonic, and the logits carry more
// bits than fp32 probabilities); ties go to the lower expert index.  Lane j < k writes the j-th choice.
// (maxima go through the warp's integer reduction, one instruction instead of five shuffle rounds: this
// routine sits on the serial path of every decode launch)
// Registers only: lane j < k gets the j-th choice (my_idx) and its gate weight (my_w); every lane gets the set of
// selected experts as a bit mask.  One warp-wide maximum and one ballot per choice; the exponentials are those of
// the k selected logits only, unless the full softmax is asked for (probs_out) or the weights are not renormalised
// (then the softmax denominator over all E logits is needed).  Renormalised weights are formed the same way in
// either case, exp(l_j - m) / sum over the selected of exp(l_i - m) with m the largest logit, so they do not depend
// on whether the probabilities were asked for.
__device__ __forceinline__ void warp_route_top(float l0, float l1, int E, int k, int renorm, int lane,
                                               float* __restrict__ probs_out, int& my_idx, float& my_w,
                                               unsigned long long& selmask) {
  const unsigned FULL = 0xffffffffu;
  const bool has0 = lane < E, has1 = lane + 32 < E;
  const bool two = E > 32;  // (uniform) a lane holds a second logit
  unsigned key0 = has0 ? f32_key(l0) : 0u, key1 = has1 ? f32_key(l1) : 0u;  // 0: taken or absent (below every key)
  float m = 0.f, wtot = 0.f, my_pw = 0.f;
  my_idx = 0;
  selmask = 0ull;
  for (int j = 0; j < k; ++j) {
    // ties keep the lower index: within a lane expert `lane` is below `lane + 32`, across lanes every `lane`
    // candidate is below every `lane + 32` one, and the lowest lane is the lowest index
    const unsigned key = key0 >= key1 ? key0 : key1;
    const unsigned best = __reduce_max_sync(FULL, key);
    int win;
    if (!two) {
      win = __ffs(__ballot_sync(FULL, key0 == best)) - 1;
    } else {
      const unsigned b0 = __ballot_sync(FULL, key0 == best), b1 = __ballot_sync(FULL, key1 == best);
      win = b0 ? __ffs(b0) - 1 : 31 + __ffs(b1);
    }
    if (win == lane) key0 = 0u;
    if (win == lane + 32) key1 = 0u;
    const float bv = f32_unkey(best);
    if (j == 0) m = bv;
    const float pw = expf(bv - m);
    wtot += pw;
    selmask |= 1ull << win;
    if (lane == j) my_pw = pw, my_idx = win;
  }
  my_w = my_pw / wtot;
  if (probs_out || !renorm) {
    const float p0 = has0 ? expf(l0 - m) : 0.f, p1 = has1 ? expf(l1 - m) : 0.f;
    const float inv_sum = 1.0f / warp_sum(p0 + p1);
    if (probs_out) {
      if (has0) probs_out[lane] = p0 * inv_sum;
      if (has1) probs_out[lane + 32] = p1 * inv_sum;
    }
    if (!renorm) my_w = my_pw * inv_sum;
  }
}

__device__ __forceinline__ void warp_route_finish(float l0, float l1, int E, int k, int renorm, int lane,
                                                  int32_t* __restrict__ idx_out, float* __restrict__ w_out,
                                                  float* __restrict__ probs_out) {
  int my_idx;
  float my_w;
  unsigned long long selmask;
  warp_route_top(l0, l1, E, k, renorm, lane, probs_out, my_idx, my_w, selmask);
  if (lane < k) {
    idx_out[lane] = my_idx;
    w_out[lane] = my_w;
  }
}

// The same with the expert set prescribed (sel[0..k), distinct): the gate weights are the softmax probabilities
// (Eq. 2) of those experts, renormalised over the set when `renorm`.  Lane j < k writes the j-th entry.
__device__ __forceinline__ void warp_route_forced(float l0, float l1, int E, int k, int renorm, int lane,
                                                  const int* __restrict__ sel, int32_t* __restrict__ idx_out,
                                                  float* __restrict__ w_out) {
  const unsigned FULL = 0xffffffffu;
  const float NEG = -3.402823466e38f;
  const bool has0 = lane < E, has1 = lane + 32 < E;
  const float m = f32_unkey(__reduce_max_sync(FULL, f32_key(fmaxf(has0 ? l0 : NEG, has1 ? l1 : NEG))));
  const float p0 = has0 ? expf(l0 - m) : 0.f, p1 = has1 ? expf(l1 - m) : 0.f;
  const float inv_sum = 1.0f / warp_sum(p0 + p1);
  float my_w = 0.f, wtot = 0.f;
  int my_idx = 0;
  for (int j = 0; j < k; ++j) {
    const int e = sel[j];
    const float a = __shfl_sync(FULL, p0, e & 31), b = __shfl_sync(FULL, p1, e & 31);
    const float pw = (e < 32 ? a : b) * inv_sum;
    wtot += pw;
    if (lane == j) my_w = pw, my_idx = e;
  }
  if (lane < k) {
    idx_out[lane] = my_idx;
    w_out[lane] = renorm ? my_w / wtot : my_w;
  }
}

#endif  // __CUDACC__
}  // namespace cosmoe
