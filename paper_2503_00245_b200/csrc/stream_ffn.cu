// Streaming (decode) path of the expert FFN: T <= 16 tokens.
//
// The work is bandwidth: every selected expert's weights are read once.  All matrices are stored
// with one output neuron's weights contiguous ("rows"), so a phase is "for my rows: dot(row, input
// vector) for every token routed to that expert".  One cooperative kernel, one CTA per SM:
//
//   dense experts   phase 0: gate_up rows  . x        -> h = silu(g) * u      (global, fp32)
//                   phase 1: down_t rows   . h        -> y (gate-weighted) or out_slots
//   Eq. 1 factors   phase 0: wd_a rows . x -> t_g,t_u;  phase 1: wd_b rows . t -> h;
//                   phase 2: wd_c rows . h -> v;        phase 3: wd_d rows . v -> y / out_slots
//
// Rows of (active expert x phase matrix) are split evenly over the CTAs; the last phase splits the
// output rows instead so that a CTA owns its outputs for all experts and sums them itself (no
// atomics, fixed order).  Phases are separated by a bounded grid barrier.
//
// Inside a CTA the warps are specialised and talk through mbarriers only:
//   producer warp   walks the list of stages (a stage = a few consecutive rows, <= 32 KB) and
//                   brings each into a ring slot with one bulk asynchronous copy (TMA without a
//                   tensor map: the rows a CTA needs are one contiguous run of bytes), running ahead
//                   of the consumers -- across phase boundaries too, so DRAM stays busy while the
//                   grid barrier is crossed;
//   8 consumer warps   wait for a slot, take (row, segment) tasks, leave partial dot products;
//   epilogue warp   finishes each stage (sums partials, SiLU*mul, stores / accumulates y), frees
//                   the slot, crosses the grid barrier and loads input vectors for the next expert.
// Every role derives the same stage list from the routing by itself, so no descriptors are passed.
#include "common.cuh"

namespace cosmoe {

namespace {

constexpr int kWarps = 8;                       // consumer warps
constexpr int kProducerWarp = kWarps;
constexpr int kEpilogueWarp = kWarps + 1;
constexpr int kThreads = (kWarps + 2) * 32;
constexpr int kMaxSlotsPerGroup = 8;            // tokens of one expert handled per pass over its rows
constexpr int kMaxRowsPerStage = 32;
constexpr int kMaxTasks = 2 * kMaxRowsPerStage; // sub-rows x segments per stage, >= kWarps
constexpr int kMaxSlots = MOE_STREAM_MAX_TOKENS * MOE_MAX_TOPK;
constexpr int kMaxPhases = 4;
constexpr int kMaxStages = 8;
constexpr int kRegIters = 8;                    // chunks per lane the register-resident vector path holds

enum InKind { IN_X = 0, IN_PAIR = 1, IN_SLOT = 2 };
enum EpiKind { EPI_SWIGLU = 0, EPI_PAIR_RAW = 1, EPI_RAW = 2, EPI_FINAL = 3 };
enum DescKind { D_STAGE = 0, D_BARRIER = 1, D_END = 2 };

struct Phase {
  const uint16_t* mat;             // packed matrix of slot 0
  unsigned long long slot_stride;  // elements between expert slots
  int rows, cols, nsub;            // rows per expert, elements per sub-row, sub-rows per row (2 = interleaved pair)
  int in_kind, epi_kind;
  const float* in;                 // global fp32 source of the input vectors (IN_PAIR / IN_SLOT)
  float* out;                      // global fp32 destination (all but EPI_FINAL)
  int rows_per_stage;
  int segs;                        // segments a sub-row is cut into (power of two <= kWarps)
};

struct StreamParams {
  int T, k, E, d, mode, x_is_bf16, n_phases;
  const void* x;
  const int32_t* topk_idx;
  const float* topk_w;
  const int32_t* offsets;
  const int32_t* perm;
  const int32_t* expert_slot;
  void* y;
  float* out_slots;
  DeviceState* st;
  int stage_bytes, n_stages, vec_cap_floats, yacc_rows;
  Phase ph[kMaxPhases];
};

struct Desc {
  int kind, phase;
  int ai;           // active-expert ordinal
  int s0, ns;       // slot sub-range of that expert handled by this pass
  int row0, nrows;  // rows of the expert's matrix in this stage
  int first;        // first stage of a (expert, slot group) pass: input vectors change here
};

struct Smem {
  uint64_t full[kMaxStages];   // stage data landed (producer / TMA), or grid barrier crossed (epilogue warp)
  uint64_t done[kMaxStages];   // all consumer warps finished with the slot
  uint64_t freeb[kMaxStages];  // epilogue finished: slot and its partials may be reused
  uint64_t vec_ready;          // shared-memory input vectors of the current pass are in place
  int act_e[MOE_MAX_EXPERTS];
  int act_slot[MOE_MAX_EXPERTS];     // packed-array slot of the active expert
  int act_off[MOE_MAX_EXPERTS + 1];  // slot ranges, expert-ascending (same numbering as moe_permute)
  int slot_tok[kMaxSlots];
  float slot_w[kMaxSlots];
  int cursor[MOE_MAX_EXPERTS];
  int n_act;
  int flag;
  volatile int abort;
  float part[kMaxStages][kMaxTasks * kMaxSlotsPerGroup];
};
constexpr int kSmemHeaderBytes = (sizeof(Smem) + 127) / 128 * 128;

// ---- the stage list: a pure function of (routing, blockIdx), walked identically by every role ----
struct Gen {
  int phase, ai, ai_hi, grp, ngrp, row, ra, rb;
};

__device__ __forceinline__ void item_bounds(const StreamParams& P, const Smem& sm, int phase, int ai, int& ra, int& rb,
                                            int& ngrp) {
  const Phase& ph = P.ph[phase];
  const unsigned G = gridDim.x, c = blockIdx.x;
  if (phase == P.n_phases - 1) {
    ra = (int)((unsigned long long)c * ph.rows / G);
    rb = (int)((unsigned long long)(c + 1) * ph.rows / G);
  } else {
    const unsigned long long U = (unsigned long long)sm.n_act * ph.rows;
    const unsigned long long u0 = c * U / G, u1 = (c + 1) * U / G;
    const unsigned long long lo = (unsigned long long)ai * ph.rows, hi = lo + ph.rows;
    const unsigned long long a = u0 > lo ? u0 : lo, b = u1 < hi ? u1 : hi;
    ra = (int)(a - lo);
    rb = b > a ? (int)(b - lo) : ra;
  }
  const int ne = sm.act_off[ai + 1] - sm.act_off[ai];
  ngrp = (ne + kMaxSlotsPerGroup - 1) / kMaxSlotsPerGroup;
}

__device__ __forceinline__ void gen_setup_phase(const StreamParams& P, const Smem& sm, Gen& g) {
  const Phase& ph = P.ph[g.phase];
  const unsigned G = gridDim.x, c = blockIdx.x;
  if (g.phase == P.n_phases - 1) {
    g.ai = 0;
    g.ai_hi = sm.n_act - 1;
  } else {
    const unsigned long long U = (unsigned long long)sm.n_act * ph.rows;
    const unsigned long long u0 = c * U / G, u1 = (c + 1) * U / G;
    if (u1 > u0) {
      g.ai = (int)(u0 / ph.rows);
      g.ai_hi = (int)((u1 - 1) / ph.rows);
    } else {
      g.ai = 0;
      g.ai_hi = -1;
    }
  }
  g.grp = 0;
  g.ra = g.rb = g.row = 0;
  g.ngrp = 1;
  if (g.ai <= g.ai_hi) {
    item_bounds(P, sm, g.phase, g.ai, g.ra, g.rb, g.ngrp);
    g.row = g.ra;
  }
}

__device__ __forceinline__ void gen_init(const StreamParams& P, const Smem& sm, Gen& g) {
  g.phase = 0;
  gen_setup_phase(P, sm, g);
  if (sm.n_act == 0) g.phase = P.n_phases;  // nothing to do
}

// Next entry.  One D_BARRIER between phases, D_END when everything has been handed out.
__device__ __forceinline__ void gen_next(const StreamParams& P, const Smem& sm, Gen& g, Desc& d) {
  for (;;) {
    if (g.phase >= P.n_phases) {
      d.kind = D_END;
      return;
    }
    if (g.ai > g.ai_hi) {
      g.phase++;
      if (g.phase < P.n_phases) {
        gen_setup_phase(P, sm, g);
        d.kind = D_BARRIER;
        d.phase = g.phase - 1;
        return;
      }
      continue;
    }
    if (g.row >= g.rb) {
      if (g.ra < g.rb && g.grp + 1 < g.ngrp) {  // same rows again for the next group of slots
        g.grp++;
        g.row = g.ra;
        continue;
      }
      g.ai++;
      g.grp = 0;
      if (g.ai <= g.ai_hi) {
        item_bounds(P, sm, g.phase, g.ai, g.ra, g.rb, g.ngrp);
        g.row = g.ra;
      }
      continue;
    }
    const Phase& ph = P.ph[g.phase];
    const int ne = sm.act_off[g.ai + 1] - sm.act_off[g.ai];
    d.kind = D_STAGE;
    d.phase = g.phase;
    d.ai = g.ai;
    d.s0 = g.grp * kMaxSlotsPerGroup;
    d.ns = min(kMaxSlotsPerGroup, ne - d.s0);
    d.row0 = g.row;
    d.nrows = min(ph.rows_per_stage, g.rb - g.row);
    d.first = (g.row == g.ra);
    g.row += d.nrows;
    return;
  }
}

// A pass keeps its input vectors in registers (one token, few chunks per lane) or in shared memory.
__device__ __forceinline__ bool reg_path(const Phase& ph, int ns) {
  const int chunks = ph.cols >> 3;
  return ns == 1 && (chunks + ph.segs - 1) / ph.segs <= 32 * kRegIters;
}

// 8 bf16 weights (packed) times 8 fp32 inputs, added into two independent accumulators.
__device__ __forceinline__ void dot8(const uint4& wv, const float4& a, const float4& b, float& t0, float& t1) {
  t0 = fmaf(__uint_as_float(wv.x << 16), a.x, t0);
  t1 = fmaf(__uint_as_float(wv.x & 0xffff0000u), a.y, t1);
  t0 = fmaf(__uint_as_float(wv.y << 16), a.z, t0);
  t1 = fmaf(__uint_as_float(wv.y & 0xffff0000u), a.w, t1);
  t0 = fmaf(__uint_as_float(wv.z << 16), b.x, t0);
  t1 = fmaf(__uint_as_float(wv.z & 0xffff0000u), b.y, t1);
  t0 = fmaf(__uint_as_float(wv.w << 16), b.z, t0);
  t1 = fmaf(__uint_as_float(wv.w & 0xffff0000u), b.w, t1);
}

// Shared-memory vectors: fp32, each 8-element chunk split over two planes of float4 so that
// consecutive lanes read consecutive 16-byte words.
template <int NSL>
__device__ __noinline__ void task_smem(const uint4* __restrict__ wrow, const float* __restrict__ vec0, int vstride,
                                       int cols, int c0, int c1, int lane, int ns, float* out) {
  float acc0[NSL], acc1[NSL];
#pragma unroll
  for (int s = 0; s < NSL; ++s) acc0[s] = 0.f, acc1[s] = 0.f;
  const int half = cols >> 1;
#pragma unroll 2
  for (int c = c0 + lane; c < c1; c += 32) {
    const uint4 wv = wrow[c];
#pragma unroll
    for (int s = 0; s < NSL; ++s) {
      const float* vb = vec0 + (size_t)(s < ns ? s : ns - 1) * vstride;
      const float4 a = *reinterpret_cast<const float4*>(vb + c * 4);
      const float4 b = *reinterpret_cast<const float4*>(vb + half + c * 4);
      dot8(wv, a, b, acc0[s], acc1[s]);
    }
  }
#pragma unroll
  for (int s = 0; s < NSL; ++s) {
    const float t = warp_sum(acc0[s] + acc1[s]);
    if (lane == 0 && s < ns) out[s] = t;
  }
}

__device__ __forceinline__ void set_abort(const StreamParams& P, Smem& sm, unsigned detail) {
  sm.abort = 1;
  flag_error(P.st, MOE_ERR_TIMEOUT, detail);
}

__global__ void __launch_bounds__(kThreads, 1) stream_ffn_kernel(const StreamParams P) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  unsigned char* ring = smem_raw + kSmemHeaderBytes;
  float* vec = reinterpret_cast<float*>(ring + (size_t)P.n_stages * P.stage_bytes);
  float* yacc = vec + P.vec_cap_floats;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = P.n_stages;

  // ---- routing products -> active experts and their slots (same numbering as moe_permute) ----
  if (tid == 0) {
    const int n = P.T * P.k;
    int na = 0, bad = 0;
    sm.act_off[0] = 0;
    if (P.mode == 0) {
      for (int e = 0; e < P.E; ++e) sm.cursor[e] = 0;
      for (int p = 0; p < n && !bad; ++p) {
        const int e = P.topk_idx[p];
        if (e < 0 || e >= P.E)
          bad = 1;
        else
          sm.cursor[e]++;
      }
      int off = 0;
      for (int e = 0; e < P.E && !bad; ++e) {
        const int cnt = sm.cursor[e];
        sm.cursor[e] = off;
        if (cnt) {
          sm.act_e[na] = e;
          sm.act_off[na] = off;
          ++na;
          off += cnt;
        }
      }
      sm.act_off[na] = off;
      for (int p = 0; p < n && !bad; ++p) {
        const int s = sm.cursor[P.topk_idx[p]]++;
        sm.slot_tok[s] = p / P.k;
        sm.slot_w[s] = P.topk_w[p];
      }
    } else {
      for (int e = 0; e < P.E; ++e) {
        const int lo = P.offsets[e], hi = P.offsets[e + 1];
        if (lo < 0 || hi < lo || hi > n) {
          bad = 1;
          break;
        }
        if (hi > lo) {
          if (lo != sm.act_off[na]) bad = 1;
          for (int s = lo; s < hi && !bad; ++s) {
            const int p = P.perm[s];
            if (p < 0 || p >= n) {
              bad = 1;
              break;
            }
            sm.slot_tok[s] = p / P.k;
            sm.slot_w[s] = 1.0f;
          }
          sm.act_e[na] = e;
          sm.act_off[na + 1] = hi;
          ++na;
        }
      }
      if (!bad && sm.act_off[na] != n) bad = 1;
    }
    for (int a = 0; a < na && !bad; ++a) {
      const int sl = P.expert_slot ? P.expert_slot[sm.act_e[a]] : sm.act_e[a];
      if (sl < 0) bad = 1;
      sm.act_slot[a] = sl < 0 ? 0 : sl;
    }
    if (bad) {
      flag_error(P.st, MOE_ERR_STATE, 0x200u);
      na = 0;  // every CTA takes the same decision from the same data: they all run zero stages
    }
    sm.n_act = na;
    sm.abort = 0;
    for (int i = 0; i < NS; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.done[i], kWarps);
      mbar_init(&sm.freeb[i], 1);
    }
    mbar_init(&sm.vec_ready, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  for (int i = tid; i < P.T * P.yacc_rows; i += kThreads) yacc[i] = 0.f;
  __syncthreads();
  // From here on the roles meet at mbarriers only; every wait is bounded.

  Gen gen;
  gen_init(P, sm, gen);
  Desc d;

  if (warp == kProducerWarp) {
    // ================================================================= producer
    if (lane != 0) return;
    int i = 0;
    bool ok = true;
    unsigned copy_mask = 0;  // bit (i % NS): ring slot holds a copy issued by this thread
    for (;; ++i) {
      gen_next(P, sm, gen, d);
      if (d.kind == D_END) break;
      const int slot = i % NS;
      if (i >= NS && !mbar_wait(&sm.freeb[slot], ((i / NS) - 1) & 1)) {
        set_abort(P, sm, 0x230u);
        ok = false;
        break;
      }
      if (sm.abort) {
        ok = false;
        break;
      }
      if (d.kind == D_STAGE) {
        const Phase& ph = P.ph[d.phase];
        const size_t row_elems = (size_t)ph.nsub * ph.cols;
        const uint16_t* src = ph.mat + (size_t)sm.act_slot[d.ai] * ph.slot_stride + (size_t)d.row0 * row_elems;
        const uint32_t bytes = (uint32_t)(d.nrows * row_elems * 2);
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&sm.full[slot], bytes);
        bulk_g2s(ring + (size_t)slot * P.stage_bytes, src, bytes, &sm.full[slot]);
        copy_mask |= 1u << slot;
      } else {
        copy_mask &= ~(1u << slot);
      }
    }
    if (!ok) {
      // copies already in flight must land before this CTA's shared memory goes away: entries
      // i-NS .. i-1 are the ones that can still be outstanding
      for (int j = max(0, i - NS); j < i; ++j)
        if ((copy_mask >> (j % NS)) & 1u) (void)mbar_wait(&sm.full[j % NS], (j / NS) & 1);
    }
    return;
  }

  if (warp == kEpilogueWarp) {
    // ================================================================= epilogue / barrier / vectors
    const int yrow0 = (int)((unsigned long long)blockIdx.x * P.d / gridDim.x);
    int vec_fills = 0;
    int i = 0;
    bool ok = true;
    for (;; ++i) {
      gen_next(P, sm, gen, d);
      if (d.kind == D_END) break;
      const int slot = i % NS;
      const unsigned par = (i / NS) & 1;
      if (d.kind == D_BARRIER) {
        // all earlier stages' outputs were stored by this warp: publish them and meet the other CTAs
        __syncwarp();
        int okb = 1;
        if (lane == 0) {
          const unsigned gen0 = ld_acquire(&P.st->bar_gen);
          __threadfence();
          const unsigned old = atom_add_acq_rel(&P.st->bar_count, 1u);
          if (old == gridDim.x - 1u) {
            P.st->bar_count = 0u;
            __threadfence();
            st_release(&P.st->bar_gen, gen0 + 1u);
          } else {
            const long long t0 = clock64();
            unsigned spins = 0;
            while (ld_acquire(&P.st->bar_gen) == gen0) {
              if ((++spins & 255u) == 0u && (clock64() - t0 > kWaitBudgetCycles || sm.abort)) {
                okb = 0;
                break;
              }
            }
          }
          __threadfence();
        }
        okb = __shfl_sync(0xffffffffu, okb, 0);
        if (!okb) {
          if (lane == 0) set_abort(P, sm, 0x220u);
          ok = false;
          break;
        }
        if (lane == 0) mbar_arrive(&sm.full[slot]);
      } else if (d.first && !reg_path(P.ph[d.phase], d.ns)) {
        // input vectors of this pass -> shared memory (every earlier entry is fully consumed: this warp
        // has waited for their `done` barriers in order)
        const Phase& ph = P.ph[d.phase];
        const int cols = ph.cols, quads = cols >> 2;
        const int nvec = ph.in_kind == IN_PAIR ? 2 * d.ns : d.ns;
        for (int idx = lane; idx < nvec * quads; idx += 32) {
          const int v = idx / quads, q = idx % quads;
          const int s_local = ph.in_kind == IN_PAIR ? (v >> 1) : v;
          const int gs = sm.act_off[d.ai] + d.s0 + s_local;
          float4 val;
          if (ph.in_kind == IN_X) {
            const int t = sm.slot_tok[gs];
            if (P.x_is_bf16) {
              const uint2 raw = *reinterpret_cast<const uint2*>((const uint16_t*)P.x + (size_t)t * cols + q * 4);
              val.x = __uint_as_float(raw.x << 16), val.y = __uint_as_float(raw.x & 0xffff0000u);
              val.z = __uint_as_float(raw.y << 16), val.w = __uint_as_float(raw.y & 0xffff0000u);
            } else {
              val = *reinterpret_cast<const float4*>((const float*)P.x + (size_t)t * cols + q * 4);
            }
          } else if (ph.in_kind == IN_PAIR) {
            val = __ldcg(reinterpret_cast<const float4*>(ph.in + ((size_t)gs * 2 + (v & 1)) * cols + q * 4));
          } else {
            val = __ldcg(reinterpret_cast<const float4*>(ph.in + (size_t)gs * cols + q * 4));
          }
          *reinterpret_cast<float4*>(vec + (size_t)v * cols + (q & 1) * (cols >> 1) + (q >> 1) * 4) = val;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.vec_ready);
        ++vec_fills;
      }
      if (!mbar_wait(&sm.done[slot], par)) {
        if (lane == 0) set_abort(P, sm, 0x240u);
        ok = false;
        break;
      }
      if (d.kind == D_STAGE) {
        const Phase& ph = P.ph[d.phase];
        const int S = ph.segs;
        const float* part = sm.part[slot];
        const int per_row = ph.epi_kind == EPI_PAIR_RAW ? 2 * d.ns : d.ns;
        for (int idx = lane; idx < d.nrows * per_row; idx += 32) {
          const int rl = idx / per_row, j = idx % per_row;
          const int s = ph.epi_kind == EPI_PAIR_RAW ? (j >> 1) : j;
          const int gs = sm.act_off[d.ai] + d.s0 + s;
          const int row = d.row0 + rl;
          auto total = [&](int sr) {
            float t = 0.f;
            for (int seg = 0; seg < S; ++seg) t += part[(sr * S + seg) * kMaxSlotsPerGroup + s];
            return t;
          };
          if (ph.epi_kind == EPI_SWIGLU) {
            const float g = total(2 * rl), u = total(2 * rl + 1);
            ph.out[(size_t)gs * ph.rows + row] = g / (1.0f + expf(-g)) * u;
          } else if (ph.epi_kind == EPI_PAIR_RAW) {
            ph.out[((size_t)gs * 2 + (j & 1)) * ph.rows + row] = total(2 * rl + (j & 1));
          } else if (ph.epi_kind == EPI_RAW) {
            ph.out[(size_t)gs * ph.rows + row] = total(rl);
          } else {
            const float v = total(rl);
            if (P.mode == 1)
              P.out_slots[(size_t)gs * P.d + row] = v;
            else
              yacc[sm.slot_tok[gs] * P.yacc_rows + (row - yrow0)] += sm.slot_w[gs] * v;
          }
        }
        __syncwarp();
      }
      if (lane == 0) mbar_arrive(&sm.freeb[slot]);
    }
    if (ok && P.mode == 0) {
      __syncwarp();
      const int yrow1 = (int)((unsigned long long)(blockIdx.x + 1) * P.d / gridDim.x);
      const int nr = yrow1 - yrow0;
      for (int idx = lane; idx < P.T * nr; idx += 32) {
        const int t = idx / nr, r = idx % nr;
        const float v = yacc[t * P.yacc_rows + r];
        if (P.x_is_bf16)
          ((__nv_bfloat16*)P.y)[(size_t)t * P.d + yrow0 + r] = __float2bfloat16_rn(v);
        else
          ((float*)P.y)[(size_t)t * P.d + yrow0 + r] = v;
      }
    }
    return;
  }

  // ===================================================================== consumers
  float4 xr[kRegIters][2];  // register-resident input vector chunks (one token)
  int vec_waits = 0;
  bool use_regs = false;
  for (int i = 0;; ++i) {
    gen_next(P, sm, gen, d);
    if (d.kind == D_END) break;
    const int slot = i % NS;
    int cols = 0, chunks = 0, S = 1, c0 = 0, c1 = 0, sub = 0;
    if (d.kind == D_STAGE) {
      const Phase& ph = P.ph[d.phase];
      cols = ph.cols, chunks = cols >> 3, S = ph.segs;
      const int seg = warp & (S - 1);
      c0 = (int)((long long)seg * chunks / S), c1 = (int)((long long)(seg + 1) * chunks / S);
      sub = ph.nsub == 2 ? ((warp / S) & 1) : 0;  // constant per warp: kWarps / S is even when nsub == 2
      if (d.first) {
        use_regs = reg_path(ph, d.ns);
        if (use_regs) {
          // this warp's chunks of the single token's input vector, straight from global memory
          const int gs = sm.act_off[d.ai] + d.s0;
#pragma unroll
          for (int it = 0; it < kRegIters; ++it) {
            const int c = c0 + lane + 32 * it;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
            if (c < c1) {
              if (ph.in_kind == IN_X) {
                const int t = sm.slot_tok[gs];
                if (P.x_is_bf16) {
                  const uint4 raw = *reinterpret_cast<const uint4*>((const uint16_t*)P.x + (size_t)t * cols + c * 8);
                  a.x = __uint_as_float(raw.x << 16), a.y = __uint_as_float(raw.x & 0xffff0000u);
                  a.z = __uint_as_float(raw.y << 16), a.w = __uint_as_float(raw.y & 0xffff0000u);
                  b.x = __uint_as_float(raw.z << 16), b.y = __uint_as_float(raw.z & 0xffff0000u);
                  b.z = __uint_as_float(raw.w << 16), b.w = __uint_as_float(raw.w & 0xffff0000u);
                } else {
                  const float* p = (const float*)P.x + (size_t)t * cols + c * 8;
                  a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
                }
              } else {
                const float* p = ph.in + (ph.in_kind == IN_PAIR ? ((size_t)gs * 2 + sub) : (size_t)gs) * cols + c * 8;
                a = __ldcg(reinterpret_cast<const float4*>(p)), b = __ldcg(reinterpret_cast<const float4*>(p + 4));
              }
            }
            xr[it][0] = a, xr[it][1] = b;
          }
        } else {
          if (!mbar_wait(&sm.vec_ready, vec_waits & 1)) {
            if (lane == 0) set_abort(P, sm, 0x250u);
            break;
          }
          ++vec_waits;
        }
      }
    }
    if (!mbar_wait(&sm.full[slot], (i / NS) & 1)) {
      if (lane == 0) set_abort(P, sm, 0x210u + (unsigned)d.kind);
      break;
    }
    if (d.kind == D_STAGE) {
      const Phase& ph = P.ph[d.phase];
      const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)slot * P.stage_bytes);
      float* part = sm.part[slot];
      const int tasks = d.nrows * ph.nsub * S;
      for (int task = warp; task < tasks; task += kWarps) {
        const int sr = task / S;  // sub-row inside the stage; task % S == seg
        const uint4* wrow = stage + (size_t)sr * chunks;
        float* out = part + task * kMaxSlotsPerGroup;
        if (use_regs) {
          // chunk indices past the segment are clamped (their register inputs are zero), so the loads
          // carry no branch and can all be in flight together
          const int cb = c0 + lane, cl = c1 - 1;
          float a0 = 0.f, a1 = 0.f;
          {
            uint4 wv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) wv[j] = wrow[min(cb + 32 * j, cl)];
#pragma unroll
            for (int j = 0; j < 4; ++j) dot8(wv[j], xr[j][0], xr[j][1], a0, a1);
          }
          if (c1 - c0 > 128) {
            uint4 wv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) wv[j] = wrow[min(cb + 32 * (j + 4), cl)];
#pragma unroll
            for (int j = 0; j < 4; ++j) dot8(wv[j], xr[j + 4][0], xr[j + 4][1], a0, a1);
          }
          const float t = warp_sum(a0 + a1);
          if (lane == 0) out[0] = t;
        } else {
          const int tsub = ph.nsub == 2 ? (sr & 1) : 0;
          const int vstride = (ph.in_kind == IN_PAIR ? 2 : 1) * cols;
          const float* vec0 = vec + (ph.in_kind == IN_PAIR ? (size_t)tsub * cols : 0);
          if (d.ns == 1)
            task_smem<1>(wrow, vec0, vstride, cols, c0, c1, lane, d.ns, out);
          else if (d.ns == 2)
            task_smem<2>(wrow, vec0, vstride, cols, c0, c1, lane, d.ns, out);
          else if (d.ns <= 4)
            task_smem<4>(wrow, vec0, vstride, cols, c0, c1, lane, d.ns, out);
          else
            task_smem<8>(wrow, vec0, vstride, cols, c0, c1, lane, d.ns, out);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.done[slot]);
  }
}

}  // namespace

int launch_stream_ffn(moe_ctx* ctx, int mode, const void* x, int T, const moe_weights* w, const int32_t* topk_idx,
                      const float* topk_w, const int32_t* offsets, const int32_t* perm, void* y, float* out_slots,
                      char* ws, const WsLayout& L, cudaStream_t s) {
  const moe_config& c = ctx->cfg;
  StreamParams P{};
  P.T = T, P.k = c.top_k, P.E = c.n_experts, P.d = c.d_model, P.mode = mode;
  P.x_is_bf16 = c.x_dtype == MOE_BF16;
  P.x = x, P.topk_idx = topk_idx, P.topk_w = topk_w, P.offsets = offsets, P.perm = perm;
  P.expert_slot = w->expert_slot;
  P.y = y, P.out_slots = out_slots, P.st = ctx->d_state;
  const int d = c.d_model, f = c.d_ff, r = c.wd_rank;
  float* vec_a = (float*)(ws + L.vec_a);
  float* vec_b = (float*)(ws + L.vec_b);
  float* vec_c = (float*)(ws + L.vec_c);
  auto set = [&](int i, const void* mat, int rows, int cols, int nsub, int in_kind, int epi, const float* in,
                 float* out) {
    Phase& ph = P.ph[i];
    ph.mat = (const uint16_t*)mat;
    ph.rows = rows, ph.cols = cols, ph.nsub = nsub;
    ph.slot_stride = (unsigned long long)rows * cols * nsub;
    ph.in_kind = in_kind, ph.epi_kind = epi, ph.in = in, ph.out = out;
  };
  if (r == 0) {
    P.n_phases = 2;
    set(0, w->gate_up, f, d, 2, IN_X, EPI_SWIGLU, nullptr, vec_b);
    set(1, w->down_t, d, f, 1, IN_SLOT, EPI_FINAL, vec_b, nullptr);
  } else {
    P.n_phases = 4;
    set(0, w->wd_a, r, d, 2, IN_X, EPI_PAIR_RAW, nullptr, vec_a);
    set(1, w->wd_b, f, r, 2, IN_PAIR, EPI_SWIGLU, vec_a, vec_b);
    set(2, w->wd_c, r, f, 1, IN_SLOT, EPI_RAW, vec_b, vec_c);
    set(3, w->wd_d, d, r, 1, IN_SLOT, EPI_FINAL, vec_c, nullptr);
  }
  // shared-memory plan
  int max_row_bytes = 0, max_vec_floats = 0;
  for (int i = 0; i < P.n_phases; ++i) {
    const Phase& ph = P.ph[i];
    max_row_bytes = max(max_row_bytes, ph.nsub * ph.cols * 2);
    const int per_slot = (ph.in_kind == IN_PAIR ? 2 : 1) * ph.cols;
    max_vec_floats = max(max_vec_floats, per_slot * min(T, kMaxSlotsPerGroup));
  }
  const int G = ctx->sm_count;
  P.stage_bytes = max(32768, (max_row_bytes + 127) / 128 * 128);
  P.vec_cap_floats = (max_vec_floats + 31) / 32 * 32;
  P.yacc_rows = (d + G - 1) / G + 1;
  const size_t fixed = (size_t)P.vec_cap_floats * 4 + (size_t)T * P.yacc_rows * 4 + kSmemHeaderBytes + 256;
  const long long avail = (long long)ctx->max_smem_optin - (long long)fixed;
  if (avail < 2ll * P.stage_bytes) return MOE_ERR_UNSUPPORTED;
  P.n_stages = (int)min((long long)kMaxStages, avail / P.stage_bytes);
  for (int i = 0; i < P.n_phases; ++i) {
    Phase& ph = P.ph[i];
    int rps = 1;  // power of two, so that a stage is a whole number of tasks per consumer warp
    while (rps * 2 <= kMaxRowsPerStage && rps * 2 * (ph.nsub * ph.cols * 2) <= P.stage_bytes) rps *= 2;
    ph.rows_per_stage = rps;
    int S = 1;
    while (S * 2 <= kWarps / (rps * ph.nsub) && (ph.cols >> 3) / (S * 2) >= 32) S *= 2;
    ph.segs = S;
  }
  const size_t smem = (size_t)P.n_stages * P.stage_bytes + fixed;
  MOE_CUDA_TRY(cudaFuncSetAttribute(stream_ffn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  void* args[] = {(void*)&P};
  MOE_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)stream_ffn_kernel, dim3(G), dim3(kThreads), args, smem, s));
  ctx->launches++;
  return MOE_OK;
}

}  // namespace cosmoe
