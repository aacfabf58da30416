// Streaming (decode) path of weight-decomposed experts (Eq. 1): T <= 16 tokens.
//
// The work is bandwidth: every selected expert's factors are read once.  All matrices are stored
// with one output neuron's weights contiguous ("rows"), so a phase is "for my rows: dot(row, input
// vector) for every token routed to that expert".  One cooperative kernel, one CTA per SM:
//
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
// Every role derives the same list of passes (phase, expert, token group, row range) and stages from the
// routing by itself, so no descriptors are passed; the per-stage loops carry almost no bookkeeping.
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
  int seg_shift;                   // log2(segs)
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
  int stage_bytes, n_stages, vec_cap_floats, yacc_rows, vstage_bytes;
  Phase ph[kMaxPhases];
};

struct Smem {
  uint64_t full[kMaxStages];   // stage data landed (producer / TMA), or grid barrier crossed (epilogue warp)
  uint64_t done[kMaxStages];   // all consumer warps finished with the slot
  uint64_t freeb[kMaxStages];  // epilogue finished: slot and its partials may be reused
  uint64_t vec_ready;          // shared-memory input vectors of the current pass are in place (multi-token passes)
  uint64_t vfull[2];           // single-token passes: the input vector landed in staging buffer 0 / 1
  Phase ph[kMaxPhases];        // copy of the launch parameters (indexed dynamically)
  int n_phases;
  int act_e[MOE_MAX_EXPERTS];
  int act_slot[MOE_MAX_EXPERTS];     // packed-array slot of the active expert
  int act_off[MOE_MAX_EXPERTS + 1];  // slot ranges, expert-ascending (same numbering as moe_permute)
  int slot_tok[kMaxSlots];
  float slot_w[kMaxSlots];
  int cursor[MOE_MAX_EXPERTS];
  int stage_e[kMaxSlots];  // routing as read from global memory, before grouping
  float stage_w[kMaxSlots];
  int n_act;
  volatile int abort;
  float part[kMaxStages][kMaxTasks * kMaxSlotsPerGroup];
};
constexpr int kSmemHeaderBytes = (sizeof(Smem) + 127) / 128 * 128;

// ---- the list of passes: a pure function of (routing, blockIdx), walked identically by every role ----
// A pass = rows [ra, rb) of one active expert's matrix in one phase, for one group of <= 8 tokens.
// Its stages are consecutive runs of rows_per_stage rows.  Between phases comes one K_BARRIER entry,
// which takes a ring slot like a stage does.
enum { K_PASS = 0, K_BARRIER = 1, K_END = 2 };
struct Pass {
  int phase, ai, s0, ns, ra, rb;
};
struct PassIt {
  int phase, ai, ai_hi, grp, ngrp, ra, rb;
};

__device__ __forceinline__ void item_bounds(const Smem& sm, PassIt& g) {
  const Phase& ph = sm.ph[g.phase];
  const unsigned G = gridDim.x, c = blockIdx.x;
  if (g.phase == sm.n_phases - 1) {
    g.ra = (int)((unsigned long long)c * ph.rows / G);
    g.rb = (int)((unsigned long long)(c + 1) * ph.rows / G);
  } else {
    const unsigned long long U = (unsigned long long)sm.n_act * ph.rows;
    const unsigned long long u0 = c * U / G, u1 = (c + 1) * U / G;
    const unsigned long long lo = (unsigned long long)g.ai * ph.rows, hi = lo + ph.rows;
    const unsigned long long a = u0 > lo ? u0 : lo, b = u1 < hi ? u1 : hi;
    g.ra = (int)(a - lo);
    g.rb = b > a ? (int)(b - lo) : g.ra;
  }
  const int ne = sm.act_off[g.ai + 1] - sm.act_off[g.ai];
  g.ngrp = (ne + kMaxSlotsPerGroup - 1) / kMaxSlotsPerGroup;
  g.grp = 0;
}

__device__ __forceinline__ void setup_phase(const Smem& sm, PassIt& g) {
  const Phase& ph = sm.ph[g.phase];
  const unsigned G = gridDim.x, c = blockIdx.x;
  if (g.phase == sm.n_phases - 1) {
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
  g.ra = g.rb = g.grp = 0;
  g.ngrp = 0;
  if (g.ai <= g.ai_hi) item_bounds(sm, g);
}

__device__ __forceinline__ void pass_init(const Smem& sm, PassIt& g) {
  g.phase = 0;
  setup_phase(sm, g);
  if (sm.n_act == 0) g.phase = sm.n_phases;  // nothing to do
}

__device__ __forceinline__ int next_pass(const Smem& sm, PassIt& g, Pass& ps) {
  for (;;) {
    if (g.phase >= sm.n_phases) return K_END;
    if (g.ai > g.ai_hi) {
      g.phase++;
      if (g.phase < sm.n_phases) {
        setup_phase(sm, g);
        return K_BARRIER;
      }
      continue;
    }
    if (g.ra >= g.rb || g.grp >= g.ngrp) {
      g.ai++;
      if (g.ai <= g.ai_hi) item_bounds(sm, g);
      continue;
    }
    const int ne = sm.act_off[g.ai + 1] - sm.act_off[g.ai];
    ps.phase = g.phase;
    ps.ai = g.ai;
    ps.s0 = g.grp * kMaxSlotsPerGroup;
    ps.ns = min(kMaxSlotsPerGroup, ne - ps.s0);
    ps.ra = g.ra;
    ps.rb = g.rb;
    g.grp++;
    return K_PASS;
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

__device__ __forceinline__ float4 bf16x4_lo(const uint4& r) {
  return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u), __uint_as_float(r.y << 16),
                     __uint_as_float(r.y & 0xffff0000u));
}
__device__ __forceinline__ float4 bf16x4_hi(const uint4& r) {
  return make_float4(__uint_as_float(r.z << 16), __uint_as_float(r.z & 0xffff0000u), __uint_as_float(r.w << 16),
                     __uint_as_float(r.w & 0xffff0000u));
}

__device__ __forceinline__ void set_abort(DeviceState* st, Smem& sm, unsigned detail) {
  sm.abort = 1;
  flag_error(st, MOE_ERR_TIMEOUT, detail);
}

// Position in the ring: slot index and the parity of its current use.
struct RingPos {
  int slot;
  unsigned par;
  int n;  // entries handed out so far
  __device__ __forceinline__ void advance(int NS) {
    ++n;
    if (++slot == NS) slot = 0, par ^= 1u;
  }
};

// ---- consumer: one pass with the (single) input vector in registers -------------------------------
// GROUPS = 1: at most 4 chunks per lane, GROUPS = 2: up to 8.  Chunk indices past the segment are clamped
// for the load (their register inputs are zero), so the loads carry no branch and are all in flight together.
template <int GROUPS>
__device__ __forceinline__ bool consume_pass_regs(DeviceState* st, int NS, int stage_bytes, Smem& sm, const Phase& ph,
                                                  const Pass& ps, const unsigned char* ring, RingPos& rp, int warp,
                                                  int lane, int c0, int c1, const float4 (&xr)[kRegIters][2]) {
  const int chunks = ph.cols >> 3, sshift = ph.seg_shift, rps = ph.rows_per_stage;
  const int cb = c0 + lane, cl = c1 - 1;
  for (int row = ps.ra; row < ps.rb; row += rps) {
    const int tasks = (min(rps, ps.rb - row) * ph.nsub) << sshift;
    if (!mbar_wait(&sm.full[rp.slot], rp.par)) {
      if (lane == 0) set_abort(st, sm, 0x210u);
      return false;
    }
    const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)rp.slot * stage_bytes);
    float* part = sm.part[rp.slot];
    for (int task = warp; task < tasks; task += kWarps) {
      const uint4* wrow = stage + (task >> sshift) * chunks;
      float a0 = 0.f, a1 = 0.f;
      uint4 wv[4 * GROUPS];
#pragma unroll
      for (int j = 0; j < 4 * GROUPS; ++j) wv[j] = wrow[min(cb + 32 * j, cl)];
#pragma unroll
      for (int j = 0; j < 4 * GROUPS; ++j) dot8(wv[j], xr[j][0], xr[j][1], a0, a1);
      const float t = warp_sum(a0 + a1);
      if (lane == 0) part[task * kMaxSlotsPerGroup] = t;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.done[rp.slot]);
    rp.advance(NS);
  }
  return true;
}

// ---- consumer: one pass with NSL input vectors in shared memory ----------------------------------------
// Vectors are fp32; each 8-element chunk is split over two planes of float4 so that consecutive lanes read
// consecutive 16-byte words.
template <int NSL>
__device__ __noinline__ bool consume_pass_smem(DeviceState* st, int NS, int stage_bytes, Smem& sm, const Phase& ph,
                                               const Pass& ps, const unsigned char* ring, const float* vec,
                                               RingPos& rp, int warp, int lane, int c0, int c1) {
  const int cols = ph.cols, chunks = cols >> 3, sshift = ph.seg_shift, rps = ph.rows_per_stage;
  const int half = cols >> 1, ns = ps.ns;
  const int vstride = (ph.in_kind == IN_PAIR ? 2 : 1) * cols;
  for (int row = ps.ra; row < ps.rb; row += rps) {
    const int tasks = (min(rps, ps.rb - row) * ph.nsub) << sshift;
    if (!mbar_wait(&sm.full[rp.slot], rp.par)) {
      if (lane == 0) set_abort(st, sm, 0x211u);
      return false;
    }
    const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)rp.slot * stage_bytes);
    float* part = sm.part[rp.slot];
    for (int task = warp; task < tasks; task += kWarps) {
      const int sr = task >> sshift;
      const uint4* wrow = stage + sr * chunks;
      const float* vec0 = vec + ((ph.in_kind == IN_PAIR && (sr & 1)) ? cols : 0);
      float acc0[NSL], acc1[NSL];
#pragma unroll
      for (int s = 0; s < NSL; ++s) acc0[s] = 0.f, acc1[s] = 0.f;
#pragma unroll 2
      for (int c = c0 + lane; c < c1; c += 32) {
        const uint4 wv = wrow[c];
#pragma unroll
        for (int s = 0; s < NSL; ++s) {
          const float* vb = vec0 + (s < ns ? s : ns - 1) * vstride;
          const float4 a = *reinterpret_cast<const float4*>(vb + c * 4);
          const float4 b = *reinterpret_cast<const float4*>(vb + half + c * 4);
          dot8(wv, a, b, acc0[s], acc1[s]);
        }
      }
#pragma unroll
      for (int s = 0; s < NSL; ++s) {
        const float t = warp_sum(acc0[s] + acc1[s]);
        if (lane == 0 && s < ns) part[task * kMaxSlotsPerGroup + s] = t;
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.done[rp.slot]);
    rp.advance(NS);
  }
  return true;
}

__global__ void __launch_bounds__(kThreads, 1) stream_ffn_kernel(const StreamParams P) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  unsigned char* ring = smem_raw + kSmemHeaderBytes;
  unsigned char* vstage = ring + (size_t)P.n_stages * P.stage_bytes;  // 2 staging buffers, single-token passes
  float* vec = reinterpret_cast<float*>(vstage + 2 * (size_t)P.vstage_bytes);
  float* yacc = vec + P.vec_cap_floats;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = P.n_stages;
  DeviceState* const st = P.st;

  // ---- routing products -> active experts and their slots (same numbering as moe_permute) ----
  if (P.mode == 0 && warp == 0) {
    for (int p = lane; p < P.T * P.k; p += 32) {  // the routing (at most 128 pairs) in one round trip
      sm.stage_e[p] = P.topk_idx[p];
      sm.stage_w[p] = P.topk_w[p];
    }
  }
  for (int i = tid; i < P.T * P.yacc_rows; i += kThreads) yacc[i] = 0.f;
  if (tid == 32) {
#pragma unroll
    for (int i = 0; i < kMaxPhases; ++i) sm.ph[i] = P.ph[i];
    sm.n_phases = P.n_phases;
  }
  __syncthreads();
  if (tid == 0) {
    const int n = P.T * P.k;
    int na = 0, bad = 0;
    sm.act_off[0] = 0;
    if (P.mode == 0) {
      for (int e = 0; e < P.E; ++e) sm.cursor[e] = 0;
      for (int p = 0; p < n && !bad; ++p) {
        const int e = sm.stage_e[p];
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
        const int s = sm.cursor[sm.stage_e[p]]++;
        sm.slot_tok[s] = p / P.k;
        sm.slot_w[s] = sm.stage_w[p];
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
    mbar_init(&sm.vfull[0], 1);
    mbar_init(&sm.vfull[1], 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  __syncthreads();
  // From here on the roles meet at mbarriers only; every wait is bounded.

  PassIt pit;
  pass_init(sm, pit);
  Pass ps;
  RingPos rp{0, 0u, 0};
  int kind, kind_n = K_END;

  if (warp == kProducerWarp) {
    // ================================================================= producer
    if (lane != 0) return;
    bool ok = true;
    unsigned copy_mask = 0;  // bit s: ring slot s holds a copy issued by this thread
    while (ok && (kind = next_pass(sm, pit, ps)) != K_END) {
      if (kind == K_BARRIER) {
        copy_mask &= ~(1u << rp.slot);
        rp.advance(NS);
        continue;
      }
      const Phase& ph = sm.ph[ps.phase];
      const uint32_t row_bytes = (uint32_t)(ph.nsub * ph.cols * 2);
      const unsigned char* src = reinterpret_cast<const unsigned char*>(ph.mat) +
                                 ((size_t)sm.act_slot[ps.ai] * ph.slot_stride) * 2 + (size_t)ps.ra * row_bytes;
      for (int row = ps.ra; row < ps.rb; row += ph.rows_per_stage) {
        const uint32_t bytes = (uint32_t)min(ph.rows_per_stage, ps.rb - row) * row_bytes;
        if (rp.n >= NS && !mbar_wait(&sm.freeb[rp.slot], rp.par ^ 1u)) {
          set_abort(st, sm, 0x230u);
          ok = false;
          break;
        }
        if (sm.abort) {
          ok = false;
          break;
        }
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&sm.full[rp.slot], bytes);
        bulk_g2s(ring + (size_t)rp.slot * P.stage_bytes, src, bytes, &sm.full[rp.slot]);
        copy_mask |= 1u << rp.slot;
        src += bytes;
        rp.advance(NS);
      }
    }
    if (!ok) {
      // copies already in flight must land before this CTA's shared memory goes away: the last NS
      // entries are the ones that can still be outstanding
      for (int back = 1; back <= NS && back <= rp.n; ++back) {
        const int j = rp.n - back;
        if ((copy_mask >> (j % NS)) & 1u) (void)mbar_wait(&sm.full[j % NS], (unsigned)(j / NS) & 1u);
      }
    }
    return;
  }

  if (warp == kEpilogueWarp) {
    // ================================================================= epilogue / barrier / vectors
    const int yrow0 = (int)((unsigned long long)blockIdx.x * P.d / gridDim.x);
    bool ok = true;
    // Single-token passes read their input vector from a staging buffer that this warp fills with one
    // bulk copy per pass, one pass ahead (two buffers).  Buffer (n & 1) serves the n-th such pass; it is free
    // again once this warp has seen the `done` barriers of the pass that used it before.
    int nreg = 0;
    auto issue_vec = [&](const Pass& q) {
      const Phase& qh = sm.ph[q.phase];
      const int gs = sm.act_off[q.ai] + q.s0;
      const unsigned char* src;
      uint32_t bytes;
      if (qh.in_kind == IN_X) {
        const uint32_t esz = P.x_is_bf16 ? 2u : 4u;
        bytes = (uint32_t)qh.cols * esz;
        src = (const unsigned char*)P.x + (size_t)sm.slot_tok[gs] * bytes;
      } else if (qh.in_kind == IN_PAIR) {
        bytes = (uint32_t)qh.cols * 8u;
        src = (const unsigned char*)(qh.in + (size_t)gs * 2 * qh.cols);
      } else {
        bytes = (uint32_t)qh.cols * 4u;
        src = (const unsigned char*)(qh.in + (size_t)gs * qh.cols);
      }
      const int b = nreg & 1;
      fence_proxy_async_all();
      mbar_arrive_expect_tx(&sm.vfull[b], bytes);
      bulk_g2s(vstage + (size_t)b * P.vstage_bytes, src, bytes, &sm.vfull[b]);
      ++nreg;
    };
    Pass ps_n;
    kind = next_pass(sm, pit, ps);
    if (lane == 0 && kind == K_PASS && reg_path(sm.ph[ps.phase], ps.ns)) issue_vec(ps);
    for (; ok && kind != K_END; ps = ps_n, kind = kind_n) {
      kind_n = next_pass(sm, pit, ps_n);
      const bool next_reg = kind_n == K_PASS && reg_path(sm.ph[ps_n.phase], ps_n.ns);
      if (kind == K_BARRIER) {
        // all earlier stages' outputs were stored by this warp: publish them and meet the other CTAs
        __syncwarp();
        int okb = 1;
        if (lane == 0) {
          // (release / acquire at GPU scope on the counter and the generation word order the stores: no fences)
          const unsigned gen0 = ld_acquire(&P.st->bar_gen);
          const unsigned old = atom_add_acq_rel(&P.st->bar_count, 1u);
          if (old == gridDim.x - 1u) {
            P.st->bar_count = 0u;
            st_release(&P.st->bar_gen, gen0 + 1u);
          } else {
            const long long t0 = clock64();
            unsigned spins = 0;
            while (ld_acquire(&P.st->bar_gen) == gen0) {
              __nanosleep(32);
              if ((++spins & 255u) == 0u && (clock64() - t0 > kWaitBudgetCycles || sm.abort)) {
                okb = 0;
                break;
              }
            }
          }
        }
        okb = __shfl_sync(0xffffffffu, okb, 0);
        if (!okb) {
          if (lane == 0) set_abort(st, sm, 0x220u);
          ok = false;
          break;
        }
        if (lane == 0) {
          if (next_reg) issue_vec(ps_n);  // the next phase's first input vector exists now
          mbar_arrive(&sm.full[rp.slot]);
        }
        if (!mbar_wait(&sm.done[rp.slot], rp.par)) {
          if (lane == 0) set_abort(st, sm, 0x241u);
          ok = false;
          break;
        }
        if (lane == 0) mbar_arrive(&sm.freeb[rp.slot]);
        rp.advance(NS);
        continue;
      }
      const Phase& ph = sm.ph[ps.phase];
      const int slot0 = sm.act_off[ps.ai] + ps.s0;  // first global slot of this pass
      if (lane == 0 && next_reg) issue_vec(ps_n);   // same phase: its input exists already
      if (!reg_path(ph, ps.ns)) {
        // input vectors of this pass -> shared memory (every earlier entry is fully consumed: this warp
        // has waited for their `done` barriers in order)
        const int cols = ph.cols, quads = cols >> 2;
        const int nvec = ph.in_kind == IN_PAIR ? 2 * ps.ns : ps.ns;
        for (int idx = lane; idx < nvec * quads; idx += 32) {
          const int v = idx / quads, q = idx - v * quads;
          const int gs = slot0 + (ph.in_kind == IN_PAIR ? (v >> 1) : v);
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
      }
      const int S = ph.segs, rps = ph.rows_per_stage;
      const int per_row = ph.epi_kind == EPI_PAIR_RAW ? 2 * ps.ns : ps.ns;
      for (int row0 = ps.ra; row0 < ps.rb; row0 += rps) {
        const int nrows = min(rps, ps.rb - row0);
        if (!mbar_wait(&sm.done[rp.slot], rp.par)) {
          if (lane == 0) set_abort(st, sm, 0x240u);
          ok = false;
          break;
        }
        const float* part = sm.part[rp.slot];
        for (int idx = lane; idx < nrows * per_row; idx += 32) {
          const int rl = idx / per_row, j = idx - rl * per_row;
          const int s = ph.epi_kind == EPI_PAIR_RAW ? (j >> 1) : j;
          const int gs = slot0 + s;
          const int row = row0 + rl;
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
        if (lane == 0) mbar_arrive(&sm.freeb[rp.slot]);
        rp.advance(NS);
      }
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
  unsigned vec_par = 0;
  int nreg = 0;  // single-token passes so far (same count as the epilogue warp keeps)
  bool ok = true;
  while (ok && (kind = next_pass(sm, pit, ps)) != K_END) {
    if (kind == K_BARRIER) {
      if (!mbar_wait(&sm.full[rp.slot], rp.par)) {
        if (lane == 0) set_abort(st, sm, 0x212u);
        break;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.done[rp.slot]);
      rp.advance(NS);
      continue;
    }
    const Phase& ph = sm.ph[ps.phase];
    const int cols = ph.cols, chunks = cols >> 3, S = ph.segs, sshift = ph.seg_shift;
    const int seg = warp & (S - 1);
    const int c0 = (seg * chunks) >> sshift, c1 = ((seg + 1) * chunks) >> sshift;
    if (reg_path(ph, ps.ns)) {
      // this warp's chunks of the single token's input vector, from the staging buffer
      const int sub = ph.nsub == 2 ? ((warp >> sshift) & 1) : 0;  // constant per warp: kWarps / S is even
      const int cl = c1 - 1;
      const int b = nreg & 1;
      if (!mbar_wait(&sm.vfull[b], (unsigned)(nreg >> 1) & 1u)) {
        if (lane == 0) set_abort(st, sm, 0x251u);
        break;
      }
      ++nreg;
      const unsigned char* vb = vstage + (size_t)b * P.vstage_bytes;
      if (ph.in_kind == IN_X && P.x_is_bf16) {
        const uint4* p = reinterpret_cast<const uint4*>(vb);
#pragma unroll
        for (int it = 0; it < kRegIters; ++it) {
          const uint4 raw = p[min(c0 + lane + 32 * it, cl)];
          xr[it][0] = bf16x4_lo(raw), xr[it][1] = bf16x4_hi(raw);
        }
      } else {
        const float* p = reinterpret_cast<const float*>(vb) + (ph.in_kind == IN_PAIR ? sub * cols : 0);
#pragma unroll
        for (int it = 0; it < kRegIters; ++it) {
          const float4* q = reinterpret_cast<const float4*>(p + min(c0 + lane + 32 * it, cl) * 8);
          xr[it][0] = q[0], xr[it][1] = q[1];
        }
      }
#pragma unroll
      for (int it = 0; it < kRegIters; ++it)
        if (c0 + lane + 32 * it > cl) xr[it][0] = xr[it][1] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c1 - c0 > 128)
        ok = consume_pass_regs<2>(st, NS, P.stage_bytes, sm, ph, ps, ring, rp, warp, lane, c0, c1, xr);
      else
        ok = consume_pass_regs<1>(st, NS, P.stage_bytes, sm, ph, ps, ring, rp, warp, lane, c0, c1, xr);
    } else {
      if (!mbar_wait(&sm.vec_ready, vec_par)) {
        if (lane == 0) set_abort(st, sm, 0x250u);
        break;
      }
      vec_par ^= 1u;
      if (ps.ns == 1)
        ok = consume_pass_smem<1>(st, NS, P.stage_bytes, sm, ph, ps, ring, vec, rp, warp, lane, c0, c1);
      else if (ps.ns == 2)
        ok = consume_pass_smem<2>(st, NS, P.stage_bytes, sm, ph, ps, ring, vec, rp, warp, lane, c0, c1);
      else if (ps.ns <= 4)
        ok = consume_pass_smem<4>(st, NS, P.stage_bytes, sm, ph, ps, ring, vec, rp, warp, lane, c0, c1);
      else
        ok = consume_pass_smem<8>(st, NS, P.stage_bytes, sm, ph, ps, ring, vec, rp, warp, lane, c0, c1);
    }
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
    return MOE_ERR_UNSUPPORTED;  // dense experts stream through launch_dense_stream
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
  P.vec_cap_floats = T > 1 ? (max_vec_floats + 31) / 32 * 32 : 0;  // multi-token passes only
  int vstage = 0;
  for (int i = 0; i < P.n_phases; ++i)
    vstage = max(vstage, P.ph[i].cols * (P.ph[i].in_kind == IN_PAIR ? 8 : 4));
  P.vstage_bytes = (vstage + 127) / 128 * 128;
  P.yacc_rows = (d + G - 1) / G + 1;
  const size_t fixed = 2 * (size_t)P.vstage_bytes + (size_t)P.vec_cap_floats * 4 + (size_t)T * P.yacc_rows * 4 +
                       kSmemHeaderBytes + 256;
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
    ph.seg_shift = 0;
    while ((1 << ph.seg_shift) < S) ph.seg_shift++;
  }
  const size_t smem = (size_t)P.n_stages * P.stage_bytes + fixed;
  MOE_CUDA_TRY(cudaFuncSetAttribute(stream_ffn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  void* args[] = {(void*)&P};
  MOE_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)stream_ffn_kernel, dim3(G), dim3(kThreads), args, smem, s));
  ctx->launches++;
  return MOE_OK;
}

}  // namespace cosmoe
