// Streaming (decode) path of dense experts: T <= 16 tokens, d_model <= 2048, ONE kernel per layer.
//
// The work is bandwidth: every selected expert's weights are read once.  In the packed layout
// gud[S][f][3][d] all a hidden unit c of an expert needs -- its gate column, its up column and its
// row of the down matrix -- is one contiguous run of 3*d values, so a CTA that owns a range of hidden
// units streams one contiguous run of bytes and finishes those units completely:
//
//     g_c = x . gate_c,  u_c = x . up_c,  h_c = silu(g_c) * u_c,      y += (gate weight) * h_c * down_c
//
// No second phase, no grid-wide barrier: the CTAs' partial y vectors are summed with 64-bit fixed-point
// atomics (integer addition is associative, so the sum does not depend on arrival order and repeated
// calls are bit-identical).  Who turns the sums into the output: with one token and the whole layer in the
// launch, the accumulator words count their own arrivals and every CTA finishes a slice of the output by
// polling its words (see kCntBits); otherwise the last CTAs to arrive at a counter do.  Either way the
// accumulators are left zero for the next call.
//
// (active expert x hidden unit) pairs are split evenly over the CTAs (one per SM).  Inside a CTA:
//   producer thread   brings stages of 4 hidden units (8 with several tokens at d <= 1024; <= 48 KB) into a ring
//                     with one bulk asynchronous copy each (TMA without a tensor map), and each pass's token rows of x;
//   8 consumer warps  per stage: (1) one dot product each (4 units x {gate, up}) against the token(s),
//                     (2) after an mbarrier, each lane owns 8 output columns and adds the 4 units'
//                     h_c * down_c into register accumulators; at the end of a pass the accumulators go
//                     out as atomics.
// With one token (T == 1, the batch-1 decode case) the router runs in the prologue of every CTA
// (logits, softmax, top-k, gate weights: Eq. 2, Eq. 3), so the layer is a single launch.
// Every wait is bounded; an expired wait sets the ctx's status word and the kernel winds down.
#include <mutex>

#include "common.cuh"

namespace cosmoe {

namespace {

constexpr int kWarps = 8;  // consumer warps
constexpr int kProducerWarp = kWarps;
constexpr int kThreads = (kWarps + 1) * 32;
constexpr int kConsumerThreads = kWarps * 32;
constexpr int kRows = 4;       // hidden units per stage: kWarps dot products
constexpr int kRowsWide = 8;   // several tokens at d <= 1024: 8 units per stage fill both the 16 rows and the 8 k-values of the MMAs
constexpr int kMaxN = 8;       // tokens of one expert handled per pass over its units
constexpr int kMaxStages = 8;
constexpr int kXIters = 8;     // 16-byte chunks of x per lane: d <= 2048
constexpr int kMaxSlots = MOE_STREAM_MAX_TOKENS * MOE_MAX_TOPK;
constexpr int kPreStages = 3;   // one token: stages whose copies go out before the general issue loop starts
constexpr int kFinalizers = 8;  // CTAs that share the conversion of the sums into the output
constexpr float kFixScale = 68719476736.0f;      // 2^36
constexpr double kFixInv = 1.0 / 68719476736.0;
// One token, one launch per layer: the accumulator words also count the CTAs that have added to them.  A CTA adds
// (sum * 2^32 rounded) * 2^8 + 1, so the low 8 bits of a word are the number of arrivals (at most 255 per word)
// and the rest is the sum in units of 2^-32 (|sum| < 2^23): whoever reads a word with the full count has the
// final sum in hand -- no arrival counter, no fence between the sums and the count, no second read.
constexpr float kFixScaleCnt = 4294967296.0f;  // 2^32
constexpr double kFixInvCnt = 1.0 / 4294967296.0;
constexpr int kCntBits = 8;

struct DenseParams {
  int T, k, E, d, f, mode, x_is_bf16, renorm, fused_route;
  const void* x;
  const uint16_t* w_router;
  const float* b_router;
  int32_t* topk_idx;  // mode 0: routing in (fused_route == 0) or out (fused_route == 1, may be null)
  float* topk_w;
  const int32_t* offsets;  // mode 1
  const int32_t* perm;
  const int32_t* expert_slot;
  const uint16_t* gud;
  void* y;
  float* out_slots;
  DeviceState* st;
  long long* acc;
  int stage_bytes, n_stages, xs_bytes;
  int stage_rows;              // hidden units per stage: kRows, or kRowsWide for several tokens at d <= 1024
  int unit_stride;             // bytes between the hidden units of a stage (3 rows, padded for the MMA passes)
  int use_mma;                 // more than one token: every pass goes through consume_pass_mma
  int wpart_ok;                // shared memory holds the [8][d] merge buffer of the unit-owner passes (d <= 1024)
  int acc_copies;              // the CTAs spread their atomics over this many accumulator copies
  long long acc_copy_stride;   // elements between copies
  long long fin_wait_budget;   // cycles a finalising CTA waits for the arrival counter to fill up
  int f_full;                  // hidden units per expert in memory (f may be a sub-range of them, starting at ex.unit_lo)
  int given1;                  // one token, routing taken from topk_idx / topk_w (possibly a subset of its entries)
  int dyn;                     // one token, d > 1024: stages are handed out from per-expert counters (see consume_pass_cols)
  int counted;                 // one token, whole layer in this launch: arrivals are counted in the accumulator words
  DenseExtra ex;
};

struct Smem {
  uint64_t full[kMaxStages];   // stage landed
  uint64_t hbar[kMaxStages];   // all dot products of the stage are in `gu`
  uint64_t freeb[kMaxStages];  // all consumer warps are done with the stage
  uint64_t xfull[2];           // token rows of a pass landed in xs[0/1]
  uint64_t cbar;               // barrier over the consumer warps
  int stage_n[kMaxStages];             // dynamic hand-out: hidden units in the stage (0 = no more stages)
  // `red` belongs to the passes with several tokens.  Before the passes, and in launches with one token, the same
  // bytes hold what only the prologue (or only a single-token pass) needs: with them in the header a launch with 8
  // tokens at d = 1024 would have room for 3 ring stages instead of 4.
  union {
    __align__(16) float red[4][2][kRowsWide * 8][kWarps];  // [stage index & 3][gate | up][unit * 8 + token][warp]
    struct {
      float scratch[kWarps * 16 * 16];     // several tokens: the router's partial logits [warp][token][expert]; h = x / rms: 8 sums
      float rlog[kWarps][MOE_MAX_EXPERTS]; // one token: the router's partial logits
      float gu[kMaxStages][kRows * 2];     // single-token passes at d > 1024: the stage's 8 dot products
      int cursor[MOE_MAX_EXPERTS];         // grouping of several tokens
      int stage_e[kMaxSlots];              // routing as selected, before the grouping
      float stage_w[kMaxSlots];
    };
  };
  __align__(16) uint32_t zero16[4];    // what ldmatrix reads for padding rows
  int act_e[MOE_MAX_EXPERTS];
  int act_slot[MOE_MAX_EXPERTS];
  int act_off[MOE_MAX_EXPERTS + 1];
  int slot_tok[kMaxSlots];
  float slot_w[kMaxSlots];
  int n_act;
  int last;
  volatile int abort;
};
constexpr int kSmemHeaderBytes = (sizeof(Smem) + 127) / 128 * 128;

struct Pass {
  int ai, s0, ns, ra, rb;
};
struct PassIt {
  int ai, ai_hi, grp, ngrp, ra, rb;
  unsigned u0, u1;
  int cta_j, cta_c;  // few active experts: this CTA is number cta_j of the cta_c that work for its expert (else cta_c = 0)
};

__device__ __forceinline__ void item_bounds(const Smem& sm, int f, PassIt& g) {
  const unsigned lo = (unsigned)g.ai * (unsigned)f, hi = lo + (unsigned)f;
  const unsigned a = g.u0 > lo ? g.u0 : lo, b = g.u1 < hi ? g.u1 : hi;
  g.ra = (int)(a - lo);
  g.rb = b > a ? (int)(b - lo) : g.ra;
  const int ne = sm.act_off[g.ai + 1] - sm.act_off[g.ai];
  g.ngrp = (ne + kMaxN - 1) / kMaxN;
  g.grp = 0;
}
// This CTA's share [u0, u1) of the na * f hidden units of the active experts: a function of the launch shape and
// of the NUMBER of active experts only (a single token always has k of them, so its share can be worked out
// before the routing is known -- the divisions below then leave the launch's serial path).
__device__ __forceinline__ void pass_split(unsigned na, int f, PassIt& g) {
  const unsigned G = gridDim.x, b = blockIdx.x;
  g.ra = g.rb = g.grp = g.ngrp = 0;
  g.cta_j = g.cta_c = 0;
  if (na > 0 && na <= 16u && G >= na) {
    // few active experts: every CTA works for ONE expert (a second pass costs its set-up and its output atomics
    // again); the first G % na experts get one CTA more than the others
    const unsigned base = G / na, extra = G % na;
    unsigned ai, j, c;
    if (b < extra * (base + 1u)) {
      ai = b / (base + 1u), j = b % (base + 1u), c = base + 1u;
    } else {
      const unsigned b2 = b - extra * (base + 1u);
      ai = extra + b2 / base, j = b2 % base, c = base;
    }
    g.cta_j = (int)j, g.cta_c = (int)c;
    g.u0 = ai * (unsigned)f + j * (unsigned)f / c;  // j * f < 2^23
    g.u1 = ai * (unsigned)f + (j + 1u) * (unsigned)f / c;
  } else {
    const unsigned U = na * (unsigned)f;  // <= 2^22, and G * U < 2^32 (checked at launch)
    g.u0 = b * U / G;
    g.u1 = (b + 1u) * U / G;
  }
  if (g.u1 > g.u0) {
    g.ai = (int)((unsigned)g.u0 / (unsigned)f);
    g.ai_hi = (int)((unsigned)(g.u1 - 1) / (unsigned)f);
  } else {
    g.ai = 0;
    g.ai_hi = -1;
  }
}
// `presplit`: pass_split(hint_na) has already filled g; it stands if the routing found that many active experts.
__device__ __forceinline__ void pass_init(const Smem& sm, int f, PassIt& g, bool presplit = false, unsigned hint_na = 0u) {
  const unsigned na = (unsigned)sm.n_act;
  if (!presplit || na != hint_na) pass_split(na, f, g);
  if (g.ai <= g.ai_hi) item_bounds(sm, f, g);
}
__device__ __forceinline__ bool next_pass(const Smem& sm, int f, PassIt& g, Pass& ps) {
  for (;;) {
    if (g.ai > g.ai_hi) return false;
    if (g.ra >= g.rb || g.grp >= g.ngrp) {
      g.ai++;
      if (g.ai <= g.ai_hi) item_bounds(sm, f, g);
      continue;
    }
    const int ne = sm.act_off[g.ai + 1] - sm.act_off[g.ai];
    ps.ai = g.ai;
    ps.s0 = g.grp * kMaxN;
    ps.ns = min(kMaxN, ne - ps.s0);
    ps.ra = g.ra;
    ps.rb = g.rb;
    g.grp++;
    return true;
  }
}

struct RingPos {
  int slot;
  unsigned par;
  int n;
  __device__ __forceinline__ void advance(int NS) {
    ++n;
    if (++slot == NS) slot = 0, par ^= 1u;
  }
};

__device__ __forceinline__ void set_abort(DeviceState* st, Smem& sm, unsigned detail) {
  sm.abort = 1;
  flag_error(st, MOE_ERR_TIMEOUT, detail);
}

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
// 8 consecutive elements of a token row of x held in shared memory (bf16 or fp32).
__device__ __forceinline__ void load_x_chunk(const unsigned char* row, int c, bool bf16, float4& a, float4& b) {
  if (bf16) {
    const uint4 r = reinterpret_cast<const uint4*>(row)[c];
    a = bf16x4_lo(r), b = bf16x4_hi(r);
  } else {
    const float4* q = reinterpret_cast<const float4*>(row) + 2 * c;
    a = q[0], b = q[1];
  }
}

// Barrier over the consumer warps with a bounded wait (an mbarrier, not bar.sync: a warp that gave up on an
// expired wait elsewhere must not leave the others parked for ever).  `par` is the caller's phase parity.
__device__ __forceinline__ bool consumer_sync(Smem& sm, unsigned& par, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(&sm.cbar);
  const bool ok = mbar_wait_spin(&sm.cbar, par);
  par ^= 1u;
  return ok;
}

// One pass with a single token and d <= 1024: warp (g, r) = (warp >> 2, warp & 3) owns hidden unit r of the
// stages whose ring index has parity g, and does all of that unit's work -- both dot products, h, and the
// update of a d-wide partial output it keeps in registers (lane owns chunks lane, lane + 32, ...) -- so
// warps never wait for each other inside the pass.  At the end the eight partial outputs are summed in a
// fixed order through shared memory and leave as fixed-point atomics.
constexpr int kT1Iters = 4;  // 16-byte chunks of a row per lane
__device__ __forceinline__ bool consume_pass_t1(const DenseParams& P, Smem& sm, const Pass& ps, const unsigned char* ring,
                                                const unsigned char* xs, float* wpart, RingPos& rp, unsigned& cpar,
                                                int warp, int lane) {
  DeviceState* st = P.st;
  const int NS = P.n_stages, d = P.d, chunks = d >> 3, cl = chunks - 1;
  const bool xbf = P.x_is_bf16 != 0;
  const int slot0 = sm.act_off[ps.ai] + ps.s0;
  const float wgt = sm.slot_w[slot0];
  const int grp = warp >> 2, r = warp & 3;
  float4 xr[kT1Iters][2];
  float acc[kT1Iters][8];
  int cidx[kT1Iters];
#pragma unroll
  for (int it = 0; it < kT1Iters; ++it) {
    const int c = lane + 32 * it;
    cidx[it] = min(c, cl);
    load_x_chunk(xs, cidx[it], xbf, xr[it][0], xr[it][1]);
    if (c > cl) xr[it][0] = xr[it][1] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[it][j] = 0.f;
  }
  for (int row0 = ps.ra; row0 < ps.rb; row0 += kRows) {
    const int nrows = min(kRows, ps.rb - row0);
    if (!mbar_wait(&sm.full[rp.slot], rp.par)) {
      if (lane == 0) set_abort(st, sm, 0x313u);
      return false;
    }
    if ((rp.n & 1) == grp && r < nrows) {
      const uint4* base = reinterpret_cast<const uint4*>(ring + (size_t)rp.slot * P.stage_bytes + (size_t)r * P.unit_stride);
      uint4 wg[kT1Iters], wu[kT1Iters], wd[kT1Iters];
#pragma unroll
      for (int it = 0; it < kT1Iters; ++it) wg[it] = base[cidx[it]];
#pragma unroll
      for (int it = 0; it < kT1Iters; ++it) wu[it] = base[chunks + cidx[it]];
#pragma unroll
      for (int it = 0; it < kT1Iters; ++it) wd[it] = base[2 * chunks + cidx[it]];
      float g0 = 0.f, g1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
      for (int it = 0; it < kT1Iters; ++it) {
        dot8(wg[it], xr[it][0], xr[it][1], g0, g1);
        dot8(wu[it], xr[it][0], xr[it][1], u0, u1);
      }
      float g = g0 + g1, u = u0 + u1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        g += __shfl_xor_sync(0xffffffffu, g, o);
        u += __shfl_xor_sync(0xffffffffu, u, o);
      }
      const float h = g / (1.0f + expf(-g)) * u * wgt;
#pragma unroll
      for (int it = 0; it < kT1Iters; ++it) {
        float w[8];
        unpack8(wd[it], w);
        const float hh = (lane + 32 * it <= cl) ? h : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[it][j] = fmaf(hh, w[j], acc[it][j]);
      }
    }
    __syncwarp();
    if (lane == 0) {
      mbar_arrive(&sm.hbar[rp.slot]);  // keeps this barrier's phase in step with the slot's uses
      mbar_arrive(&sm.freeb[rp.slot]);
    }
    rp.advance(NS);
  }
  // ---- sum the eight warps' partial outputs in a fixed order, send the CTA's sum to the global accumulators
  float* mine = wpart + (size_t)warp * d;
#pragma unroll
  for (int it = 0; it < kT1Iters; ++it) {
    if (lane + 32 * it <= cl) {
      float4* q = reinterpret_cast<float4*>(mine + (lane + 32 * it) * 8);
      q[0] = make_float4(acc[it][0], acc[it][1], acc[it][2], acc[it][3]);
      q[1] = make_float4(acc[it][4], acc[it][5], acc[it][6], acc[it][7]);
    }
  }
  if (!consumer_sync(sm, cpar, lane)) return false;
  {
    const int rowi = P.mode == 0 ? sm.slot_tok[slot0] : slot0;
    unsigned long long* dst = reinterpret_cast<unsigned long long*>(P.acc) +
                              (size_t)(blockIdx.x % P.acc_copies) * P.acc_copy_stride + (size_t)rowi * d;
    for (int i = warp * 32 + lane; i < d; i += kConsumerThreads) {
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) v += wpart[(size_t)w * d + i];
      atomicAdd(dst + i, P.counted ? ((unsigned long long)__float2ll_rn(v * kFixScaleCnt) << kCntBits) + 1ull
                                   : (unsigned long long)__float2ll_rn(v * kFixScale));
    }
  }
  return consumer_sync(sm, cpar, lane);  // wpart may be rewritten by the next pass
}

// ---------------------------------------------------------------------------------------------------
// Passes with several tokens: the same streamed bytes, but the per-token arithmetic goes to the tensor cores
// (mma.sync m16n8k16, bf16 inputs, fp32 accumulation) so that the instruction count does not grow with the
// number of tokens and the path stays bound by the weight stream.  Up to 8 tokens per pass (the MMA's N).
//
// Per stage of 4 hidden units:
//  (1) gate/up logits: D[8 weight rows][8 tokens] = W[8][d] . X^T[d][8].  The k range is split over the
//      8 warps; warp w keeps its slice of X as B fragments in registers for the whole pass.  A thread
//      (row g = lane >> 2, q = lane & 3) loads ONE 16-byte chunk of weight row g per 32 k-values and feeds
//      its four bf16 pairs to two MMAs; the token rows are chunked the same way, so the k order inside an
//      MMA is a permutation applied to both operands, which a dot product does not see.  fp32 token rows
//      are split into a bf16 head and a bf16 remainder (two MMAs).
//  (2) after an mbarrier over the warps, every warp sums the 8 partial D tiles, forms
//      h = silu(g) * u for the 4 x 8 (unit, token) pairs (one per lane), and
//  (3) adds h . down rows into the 16-column output blocks it owns: D[16 cols][8 tokens] += A . B with
//      A = the 4 down rows read transposed by ldmatrix (k = unit, zero-padded to 8), B = h rounded to bf16
//      (m16n8k8).  The token's gate weight multiplies the pass's sum at the end.  The accumulators stay in registers for the pass and leave as fixed-point atomics.
// Units of a stage sit `unit_stride` = 3*d*2 + 16 bytes apart, so the 4 down rows fall into different banks.
// Template sizes: GROUPS = 32-value k groups per warp, BLOCKS = 16-column output blocks per warp
// (4 and 8 for d <= 1024, 8 and 16 for d <= 2048).

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_1688(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr)
               : "memory");
}
// (a, b) -> bf16 pair `head` (a in the low half) and the pair of what rounding left over
__device__ __forceinline__ void split_bf16x2(float a, float b, uint32_t& head, uint32_t& rest) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  const __nv_bfloat162 l = __floats2bfloat162_rn(a - __low2float(h), b - __high2float(h));
  head = *reinterpret_cast<const uint32_t*>(&h);
  rest = *reinterpret_cast<const uint32_t*>(&l);
}

// ROWS = hidden units per stage.  4: the 8 gate / up rows of a stage fill rows 0-7 of the first product's MMAs (rows
// 8-15 are zeros) and the 4 units half of the second product's k range.  8: a thread also feeds rows gid + 8 (units
// 4-7) and handles two (unit, token) pairs; both products run at full MMA width, and there are half as many
// stages, barriers and ldmatrix loads per byte.
template <bool XBF, int GROUPS, int BLOCKS, int ROWS>  // XBF: token rows are bf16 (else fp32: head + remainder)
__device__ __forceinline__ bool consume_pass_mma(const DenseParams& P, Smem& sm, const Pass& ps, const unsigned char* ring,
                                                 const unsigned char* xs, RingPos& rp, int warp, int lane) {
  constexpr bool WIDE = ROWS == 8;
  static_assert(ROWS == 4 || ROWS == 8, "4 or 8 hidden units per stage");
  DeviceState* st = P.st;
  const int NS = P.n_stages, d = P.d, chunks = d >> 3, cl = chunks - 1;
  const int n = ps.ns;
  const int xrow_bytes = d * (XBF ? 2 : 4);
  const int slot0 = sm.act_off[ps.ai] + ps.s0;
  const int gid = lane >> 2, q = lane & 3;
  // (1) k groups of 32 values owned by this warp: byte offset of this thread's chunk in a row, and its slice of
  // the token rows as B fragments (zero where the group or the chunk does not exist: the product vanishes
  // whatever weight bytes are read there)
  const int G = (chunks + 3) >> 2;
  const int g_lo = warp * G / kWarps, g_n = (warp + 1) * G / kWarps - g_lo;
  uint32_t coff[GROUPS];
  uint32_t bh[GROUPS][4], bl[XBF ? 1 : GROUPS][4];
  {
    // xs holds every token row of the call; tokens past n: a copy, never used
    const unsigned char* xr = xs + (size_t)sm.slot_tok[slot0 + min(gid, n - 1)] * xrow_bytes;
#pragma unroll
    for (int gi = 0; gi < GROUPS; ++gi) {
      const int c = 4 * (g_lo + gi) + q, cc = min(c, cl);
      const bool live = gi < g_n && c <= cl;
      coff[gi] = (uint32_t)cc * 16u;
      if (XBF) {
        const uint4 v = reinterpret_cast<const uint4*>(xr)[cc];
        bh[gi][0] = live ? v.x : 0u, bh[gi][1] = live ? v.y : 0u, bh[gi][2] = live ? v.z : 0u, bh[gi][3] = live ? v.w : 0u;
      } else {
        float4 a = reinterpret_cast<const float4*>(xr)[2 * cc], b = reinterpret_cast<const float4*>(xr)[2 * cc + 1];
        if (!live) a = b = make_float4(0.f, 0.f, 0.f, 0.f);
        constexpr int li = XBF ? 0 : 1;
        split_bf16x2(a.x, a.y, bh[gi][0], bl[gi * li][0]);
        split_bf16x2(a.z, a.w, bh[gi][1], bl[gi * li][1]);
        split_bf16x2(b.x, b.y, bh[gi][2], bl[gi * li][2]);
        split_bf16x2(b.z, b.w, bh[gi][3], bl[gi * li][3]);
      }
    }
  }
  // weight row r of a stage (unit r >> 1, gate | up): this thread feeds rows gid and, WIDE, gid + 8
  const uint32_t row_lo = (uint32_t)(gid >> 1) * (uint32_t)P.unit_stride + (uint32_t)(gid & 1) * (uint32_t)(2 * d);
  const uint32_t row_hi = row_lo + 4u * (uint32_t)P.unit_stride;
  // (3) output blocks of 16 columns owned by this warp.  ldmatrix: lane i gives the address of row (i & 7) =
  // hidden unit, for columns 8 * (i >> 3) of a pair of blocks; rows and columns that do not exist read zeros.
  const int NB = (d + 15) >> 4;
  const int b_lo = warp * NB / kWarps, b_n = (warp + 1) * NB / kWarps - b_lo;
  float acc[BLOCKS][4];
  uint32_t lmoff[BLOCKS / 2];
  unsigned lmok = 0;
  const int lm_unit = lane & 7;
#pragma unroll
  for (int b = 0; b < BLOCKS; ++b) acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.f;
#pragma unroll
  for (int bp = 0; bp < BLOCKS; bp += 2) {
    const int col = 16 * (b_lo + bp) + 8 * (lane >> 3);
    lmoff[bp / 2] = (uint32_t)lm_unit * (uint32_t)P.unit_stride + (uint32_t)(4 * d) + (uint32_t)col * 2u;
    if (col < d && (bp + (lane >> 4)) < b_n && lm_unit < ROWS) lmok |= 1u << (bp / 2);
  }
  const uint32_t zero_addr = (uint32_t)__cvta_generic_to_shared(sm.zero16);
  const uint32_t ring_addr = (uint32_t)__cvta_generic_to_shared(ring);
  constexpr int kPairs = kRowsWide * 8;  // (unit, token) entries of one gate | up plane of `red`
  float* const red_st = &sm.red[0][gid & 1][(gid >> 1) * 8 + 2 * q][warp];  // + buf * (elements of one buffer)
  const float* const red_ld = &sm.red[0][0][q * 8 + gid][0];
  constexpr int kRedBuf = 2 * kPairs * kWarps;

  // gate/up partial logits of one stage -> red[stage index & 3]
  auto phase1 = [&](const RingPos& r1, int nrows) {
    const unsigned char* stage = ring + (size_t)r1.slot * P.stage_bytes;
    // (a ragged last stage: rows of units that do not exist are read from the last unit that does, and never used)
    const uint32_t off_lo = nrows == ROWS ? row_lo
                                          : (uint32_t)min(gid >> 1, nrows - 1) * (uint32_t)P.unit_stride +
                                                (uint32_t)(gid & 1) * (uint32_t)(2 * d);
    const uint32_t off_hi = nrows == ROWS ? row_hi
                                          : (uint32_t)min(4 + (gid >> 1), nrows - 1) * (uint32_t)P.unit_stride +
                                                (uint32_t)(gid & 1) * (uint32_t)(2 * d);
    const unsigned char* arow = stage + off_lo;
    const unsigned char* brow = stage + off_hi;
    uint4 w[GROUPS], w2[WIDE ? GROUPS : 1];
#pragma unroll
    for (int gi = 0; gi < GROUPS; ++gi) {
      w[gi] = *reinterpret_cast<const uint4*>(arow + coff[gi]);
      if (WIDE) w2[WIDE ? gi : 0] = *reinterpret_cast<const uint4*>(brow + coff[gi]);
    }
    float c[4][4];  // four independent accumulation chains
#pragma unroll
    for (int j = 0; j < 4; ++j) c[j][0] = c[j][1] = c[j][2] = c[j][3] = 0.f;
#pragma unroll
    for (int gi = 0; gi < GROUPS; ++gi) {
      const uint4 v2 = WIDE ? w2[WIDE ? gi : 0] : make_uint4(0u, 0u, 0u, 0u);
      mma_16816(c[(2 * gi) & 3], w[gi].x, v2.x, w[gi].y, v2.y, bh[gi][0], bh[gi][1]);
      mma_16816(c[(2 * gi + 1) & 3], w[gi].z, v2.z, w[gi].w, v2.w, bh[gi][2], bh[gi][3]);
      if (!XBF) {
        mma_16816(c[(2 * gi + 2) & 3], w[gi].x, v2.x, w[gi].y, v2.y, bl[XBF ? 0 : gi][0], bl[XBF ? 0 : gi][1]);
        mma_16816(c[(2 * gi + 3) & 3], w[gi].z, v2.z, w[gi].w, v2.w, bl[XBF ? 0 : gi][2], bl[XBF ? 0 : gi][3]);
      }
    }
    // D[row gid (and gid + 8)][tokens 2q, 2q+1] -> red[buf][gate | up][unit * 8 + token][warp]
    float* dst = red_st + (r1.n & 3) * kRedBuf;
    dst[0] = (c[0][0] + c[1][0]) + (c[2][0] + c[3][0]);
    dst[kWarps] = (c[0][1] + c[1][1]) + (c[2][1] + c[3][1]);
    if (WIDE) {  // rows gid + 8: units 4 + (gid >> 1)
      dst[4 * 8 * kWarps] = (c[0][2] + c[1][2]) + (c[2][2] + c[3][2]);
      dst[4 * 8 * kWarps + kWarps] = (c[0][3] + c[1][3]) + (c[2][3] + c[3][3]);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.hbar[r1.slot]);
  };

  // The logits of stage i + 1 are issued before the barrier of stage i is waited for, so the barrier's round
  // trip and the other warps' skew hide behind tensor-core work.  A warp can be at most two stages behind
  // another one that is writing `red`, hence its four buffers.
  RingPos r1 = rp;  // the stage whose logits are computed next
  if (ps.ra < ps.rb) {
    if (!mbar_wait(&sm.full[r1.slot], r1.par)) {
      if (lane == 0) set_abort(st, sm, 0x315u);
      return false;
    }
    phase1(r1, min(ROWS, ps.rb - ps.ra));
    r1.advance(NS);
  }
  for (int row0 = ps.ra; row0 < ps.rb; row0 += ROWS) {
    const int nrows = min(ROWS, ps.rb - row0);
    if (row0 + ROWS < ps.rb) {
      if (!mbar_wait(&sm.full[r1.slot], r1.par)) {
        if (lane == 0) set_abort(st, sm, 0x315u);
        return false;
      }
      phase1(r1, min(ROWS, ps.rb - row0 - ROWS));
      r1.advance(NS);
    }
    if (!mbar_wait_spin(&sm.hbar[rp.slot], rp.par)) {
      if (lane == 0) set_abort(st, sm, 0x316u);
      return false;
    }
    // ---- (2) lane (token gid, unit q -- and, WIDE, unit q + 4): h
    float h, h2 = 0.f;
    {
      const float4* rg = reinterpret_cast<const float4*>(red_ld + (rp.n & 3) * kRedBuf);
      const float4* ru = rg + kPairs * kWarps / 4;
      const float4 g0 = rg[0], g1 = rg[1], u0 = ru[0], u1 = ru[1];
      const float g = ((g0.x + g0.y) + (g0.z + g0.w)) + ((g1.x + g1.y) + (g1.z + g1.w));
      const float u = ((u0.x + u0.y) + (u0.z + u0.w)) + ((u1.x + u1.y) + (u1.z + u1.w));
      h = (q < nrows && gid < n) ? g / (1.0f + __expf(-g)) * u : 0.f;  // the gate weight multiplies the pass's sum
      if (WIDE) {
        const float4* rg2 = rg + 4 * 8 * kWarps / 4;
        const float4* ru2 = ru + 4 * 8 * kWarps / 4;
        const float4 p0 = rg2[0], p1 = rg2[1], v0 = ru2[0], v1 = ru2[1];
        const float gg = ((p0.x + p0.y) + (p0.z + p0.w)) + ((p1.x + p1.y) + (p1.z + p1.w));
        const float uu = ((v0.x + v0.y) + (v0.z + v0.w)) + ((v1.x + v1.y) + (v1.z + v1.w));
        h2 = (q + 4 < nrows && gid < n) ? gg / (1.0f + __expf(-gg)) * uu : 0.f;
      }
    }
    // B fragment (k = units 2q, 2q+1 of 8; n = token gid): h rounded to bf16, as the hidden activations of the
    // tensor-core prefill path are.  Unit u's value sits in lane (gid, u & 3): as h for u < 4, as h2 above.
    uint32_t hb;
    {
      const int s0 = (lane & ~3) | ((2 * q) & 3), s1 = (lane & ~3) | ((2 * q + 1) & 3);
      float ha = __shfl_sync(0xffffffffu, h, s0), hc = __shfl_sync(0xffffffffu, h, s1);
      if (WIDE) {
        const float ha2 = __shfl_sync(0xffffffffu, h2, s0), hc2 = __shfl_sync(0xffffffffu, h2, s1);
        if (q >= 2) ha = ha2, hc = hc2;
      } else if (q >= 2) {
        ha = hc = 0.f;  // units 4.. are padding
      }
      const __nv_bfloat162 hp = __floats2bfloat162_rn(ha, hc);
      hb = *reinterpret_cast<const uint32_t*>(&hp);
    }
    // ---- (3) this warp's output blocks, two per ldmatrix
    const uint32_t stage_addr = ring_addr + (uint32_t)rp.slot * (uint32_t)P.stage_bytes;
    const unsigned ok = lm_unit < nrows ? lmok : 0u;
#pragma unroll
    for (int bp = 0; bp < BLOCKS; bp += 2) {
      if (bp < b_n) {
        uint32_t a[4];
        ldmatrix_x4_trans(a, ((ok >> (bp / 2)) & 1u) ? stage_addr + lmoff[bp / 2] : zero_addr);
        mma_1688(acc[bp], a[0], a[1], hb);
        mma_1688(acc[bp + 1], a[2], a[3], hb);  // zeros if the block does not exist
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.freeb[rp.slot]);
    rp.advance(NS);
  }
  // ---- the pass's partial outputs -> fixed-point accumulators: acc[b] = (cols 16b + gid, + 8; tokens 2q, 2q+1)
  {
    unsigned long long* const acc0 =
        reinterpret_cast<unsigned long long*>(P.acc) + (size_t)(blockIdx.x % P.acc_copies) * P.acc_copy_stride;
#pragma unroll
    for (int tt = 0; tt < 2; ++tt) {
      const int tk = 2 * q + tt;
      if (tk < n) {
        const int gs = slot0 + tk;
        const float wf = sm.slot_w[gs] * kFixScale;  // gate weight of the token (1 for unweighted per-slot output)
        unsigned long long* dst = acc0 + (size_t)(P.mode == 0 ? sm.slot_tok[gs] : gs) * d;
#pragma unroll
        for (int b = 0; b < BLOCKS; ++b) {
          if (b < b_n) {
            const int col = 16 * (b_lo + b) + gid;
            if (col < d) atomicAdd(dst + col, (unsigned long long)__float2ll_rn(acc[b][tt] * wf));
            if (col + 8 < d) atomicAdd(dst + col + 8, (unsigned long long)__float2ll_rn(acc[b][2 + tt] * wf));
          }
        }
      }
    }
  }
  return true;
}

// One pass with a single token and d > 1024 (the token row, 8 chunks per lane, does not leave room in the
// registers for a d-wide partial output per warp): per stage (1) warp w takes one of the 8 dot products
// (unit w >> 1, gate or up), (2) after an mbarrier each lane owns one 8-column chunk of the output and adds
// the 4 units' h_c * down_c to it.
__device__ __forceinline__ bool consume_pass_cols(const DenseParams& P, Smem& sm, const Pass& ps, const unsigned char* ring,
                                                  const unsigned char* xs, RingPos& rp, int warp, int lane) {
  DeviceState* st = P.st;
  const int NS = P.n_stages, d = P.d, chunks = d >> 3, cl = chunks - 1;
  const bool xbf = P.x_is_bf16 != 0;
  const int slot0 = sm.act_off[ps.ai] + ps.s0;
  const int cw0 = (warp * chunks) / kWarps, cw1 = ((warp + 1) * chunks) / kWarps;
  const int mychunk = cw0 + lane;
  const bool owner = mychunk < cw1;
  const int cclamp = owner ? mychunk : cw0;
  const float fix = P.counted ? kFixScaleCnt : kFixScale;
  float acc[8];
  long long iacc[8];  // dynamic hand-out: fixed-point sums, so that the result does not depend on which CTA took which stage
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f, iacc[j] = 0;
  float4 xr[kXIters][2];
#pragma unroll
  for (int it = 0; it < kXIters; ++it) {
    load_x_chunk(xs, min(lane + 32 * it, cl), xbf, xr[it][0], xr[it][1]);
    if (lane + 32 * it > cl) xr[it][0] = xr[it][1] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float wgt = sm.slot_w[slot0];

  for (int row0 = ps.ra; P.dyn || row0 < ps.rb; row0 += kRows) {
    if (!mbar_wait(&sm.full[rp.slot], rp.par)) {
      if (lane == 0) set_abort(st, sm, 0x310u);
      return false;
    }
    const int nrows = P.dyn ? sm.stage_n[rp.slot] : min(kRows, ps.rb - row0);
    if (nrows == 0) break;  // dynamic hand-out: the producer found no stage left
    const unsigned char* stage = ring + (size_t)rp.slot * P.stage_bytes;
    const int r = warp >> 1;
    if (r < nrows) {
      const uint4* wrow = reinterpret_cast<const uint4*>(stage + (size_t)r * P.unit_stride) + (size_t)(warp & 1) * chunks;
      float a0 = 0.f, a1 = 0.f;
      {
        uint4 wv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) wv[j] = wrow[min(lane + 32 * j, cl)];
#pragma unroll
        for (int j = 0; j < 4; ++j) dot8(wv[j], xr[j][0], xr[j][1], a0, a1);
      }
      if (chunks > 128) {
        uint4 wv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) wv[j] = wrow[min(lane + 32 * (j + 4), cl)];
#pragma unroll
        for (int j = 0; j < 4; ++j) dot8(wv[j], xr[j + 4][0], xr[j + 4][1], a0, a1);
      }
      const float t = warp_sum(a0 + a1);
      if (lane == 0) sm.gu[rp.slot][warp] = t;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.hbar[rp.slot]);
    if (!mbar_wait_spin(&sm.hbar[rp.slot], rp.par)) {
      if (lane == 0) set_abort(st, sm, 0x311u);
      return false;
    }
    uint4 dw[kRows];
#pragma unroll
    for (int rr = 0; rr < kRows; ++rr)
      dw[rr] = (reinterpret_cast<const uint4*>(stage + (size_t)min(rr, nrows - 1) * P.unit_stride) + 2 * (size_t)chunks)[cclamp];
    float hv = 0.f;
    if (lane < nrows) {
      const float g = sm.gu[rp.slot][2 * lane], u = sm.gu[rp.slot][2 * lane + 1];
      hv = g / (1.0f + expf(-g)) * u * wgt;
    }
#pragma unroll
    for (int rr = 0; rr < kRows; ++rr) {
      float w[8];
      unpack8(dw[rr], w);
      const float h = __shfl_sync(0xffffffffu, hv, rr);  // 0 for units past nrows
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = fmaf(h, w[j], acc[j]);
    }
    if (P.dyn) {  // a stage's sum depends on the stage alone; integer addition across stages is associative
#pragma unroll
      for (int j = 0; j < 8; ++j) iacc[j] += __float2ll_rn(acc[j] * fix), acc[j] = 0.f;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.freeb[rp.slot]);
    rp.advance(NS);
  }
  if (owner) {
    const int rowi = P.mode == 0 ? sm.slot_tok[slot0] : slot0;
    unsigned long long* dst = reinterpret_cast<unsigned long long*>(P.acc) +
                              (size_t)(blockIdx.x % P.acc_copies) * P.acc_copy_stride + (size_t)rowi * d + mychunk * 8;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long v = P.dyn ? iacc[j] : __float2ll_rn(acc[j] * fix);
      atomicAdd(dst + j, P.counted ? ((unsigned long long)v << kCntBits) + 1ull : (unsigned long long)v);
    }
  }
  return true;
}

// One instantiation per kind of pass, so that each gets its own register allocation and a short instruction
// stream: V_T1 and V_COLS single token (d <= 1024 / larger), V_MMA_* several tokens.
enum Variant { V_T1 = 0, V_COLS, V_MMA_BF16_S, V_MMA_F32_S, V_MMA_BF16_L, V_MMA_F32_L };

template <int V>
__global__ void __launch_bounds__(kThreads, 1) dense_stream_kernel(const DenseParams P) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  unsigned char* ring = smem_raw + kSmemHeaderBytes;
  unsigned char* xs = ring + (size_t)P.n_stages * P.stage_bytes;  // 2 buffers of xs_bytes
  float* wpart = reinterpret_cast<float*>(xs + 2 * (size_t)P.xs_bytes);  // [8 warps][d], single-token passes at d <= 1024
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = P.n_stages;
  DeviceState* const st = P.st;
  const int n_pairs = P.T * P.k;
  // The variant fixes whether the launch has one token (V_T1, V_COLS) or several (the others): each variant is
  // compiled without the other case's prologue.
  constexpr bool kAllX = V >= V_MMA_BF16_S;                 // several tokens: every token row is staged once
  const bool fused1 = !kAllX && P.fused_route && P.T == 1;  // one token: the router is spread over the whole CTA
  const bool given1 = !kAllX && P.given1;

  // ------------------------------------------------------------------ prologue
  // Programmatic dependent launch: the next kernel in the stream may be scheduled as soon as this one's CTAs
  // leave their SMs (its set-up then overlaps this kernel's last CTAs); this kernel in turn reads nothing a
  // predecessor may have written (x, routing, accumulators) before griddepcontrol.wait below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint64_t stream_policy = 0;     // the producer thread's cache hint for the streamed weights
  if (tid == kConsumerThreads) {  // the producer thread sets up the barriers
    for (int i = 0; i < NS; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.hbar[i], kWarps);
      mbar_init(&sm.freeb[i], kWarps);
    }
    mbar_init(&sm.xfull[0], 1);
    mbar_init(&sm.xfull[1], 1);
    mbar_init(&sm.cbar, kWarps);
    fence_mbar_init();
    fence_proxy_async_smem();
    sm.abort = 0;
    sm.last = 0;
    sm.zero16[0] = sm.zero16[1] = sm.zero16[2] = sm.zero16[3] = 0u;
    stream_policy = l2_policy_evict_first();
    if (fused1) {  // one token: k active experts with one slot each, whatever the router will select
      for (int i = 0; i <= P.k; ++i) sm.act_off[i] = i;
      for (int i = 0; i < P.k; ++i) sm.slot_tok[i] = 0;
      sm.n_act = P.k;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (fused1 && !P.ex.h_in) {
      // one token: every pass reads token row 0, so the first pass's copy of x can start before the routing
      const uint32_t xrow_bytes = (uint32_t)P.d * (P.x_is_bf16 ? 2u : 4u);
      mbar_arrive_expect_tx(&sm.xfull[0], xrow_bytes);
      bulk_g2s(xs, P.x, xrow_bytes, &sm.xfull[0]);
    } else if (kAllX) {
      // several tokens: all token rows stay in shared memory for the whole kernel (router and every pass)
      const uint32_t bytes = (uint32_t)P.T * (uint32_t)P.d * (P.x_is_bf16 ? 2u : 4u);
      mbar_arrive_expect_tx(&sm.xfull[0], bytes);
      bulk_g2s(xs, P.x, bytes, &sm.xfull[0]);
    }
  }
  PassIt pit;
  Pass ps;
  bool pass_known = false;
  // producer thread, one token: its first pass is fetched (pre_stage 1) and the barriers of that pass's first pre_n
  // stages already expect their bytes before the routing is known; pre_off: where those stages start inside an expert
  int pre_stage = 0, pre_n = 0;
  size_t pre_off = 0;
  if (fused1) pass_split((unsigned)P.k, P.f, pit);  // a single token has k active experts: known before the routing
  // the host may know the slot of routing entry `lane`'s expert (offload cache); read before anything waits
  const int given_slot = lane < MOE_MAX_TOPK ? P.ex.slot_of_entry[lane] : -1;
  // the router's weights do not depend on any earlier kernel: the first group of eight experts is fetched
  // before the dependency wait, so its DRAM latency overlaps the predecessor's tail
  // (input features per thread in the router: 4 cover d <= 1024, the shapes of these variants)
  constexpr int kRJ = (V == V_T1 || V == V_MMA_BF16_S || V == V_MMA_F32_S) ? 4 : kXIters;
  uint4 wr0[kRJ];
  const bool prefetched = P.fused_route && warp < kWarps && (P.E & 7) == 0;
  if (prefetched) {
#pragma unroll
    for (int j = 0; j < kRJ; ++j)
      wr0[j] = __ldg(reinterpret_cast<const uint4*>(P.w_router + (size_t)min(tid + j * kConsumerThreads, P.d - 1) * P.E));
  }
  if (tid != kConsumerThreads) asm volatile("griddepcontrol.wait;" ::: "memory");
  // Stacked decode: the layer input is u = h / rms(h) (fp32 h, no learned scale), formed here by every CTA, rounded
  // to the type of x, kept in shared memory as token row 0 and used for the router below.
  const bool from_h = fused1 && P.ex.h_in != nullptr;
  if (from_h) {
    float* rsum = sm.scratch;
    float hv[kRJ];
    float ss = 0.f;
    if (warp < kWarps) {
#pragma unroll
      for (int j = 0; j < kRJ; ++j) {
        const int i = tid + j * kConsumerThreads;
        hv[j] = i < P.d ? P.ex.h_in[i] : 0.f;
        ss = fmaf(hv[j], hv[j], ss);
      }
      ss = warp_sum(ss);
      if (lane == 0) rsum[warp] = ss;
    }
    __syncthreads();
    if (warp < kWarps) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) tot += rsum[w];
      const float inv = rsqrtf(tot / (float)P.d);
#pragma unroll
      for (int j = 0; j < kRJ; ++j) {
        const int i = tid + j * kConsumerThreads;
        if (i < P.d) {
          if (P.x_is_bf16)
            reinterpret_cast<__nv_bfloat16*>(xs)[i] = __float2bfloat16_rn(hv[j] * inv);
          else
            reinterpret_cast<float*>(xs)[i] = hv[j] * inv;
        }
      }
    }
  }
  // (each thread reads back only the elements it wrote itself: no barrier needed before the router)
  const void* const xsrc = from_h ? (const void*)xs : P.x;
  if (fused1) {
    // router logits of the single token: every consumer thread takes rows of W_r (row i = the E weights
    // of input feature i), 8 experts at a time
    if (warp < kWarps) {
      const int d = P.d, E = P.E;
      if ((E & 7) == 0) {
        // this thread's input features (d <= 2048: at most 8), fetched in one round trip
        float xv[kRJ];
#pragma unroll
        for (int j = 0; j < kRJ; ++j) {
          const int i = min(tid + j * kConsumerThreads, d - 1);
          xv[j] = P.x_is_bf16 ? bf16_to_float(((const uint16_t*)xsrc)[i]) : ((const float*)xsrc)[i];
          if (tid + j * kConsumerThreads >= d) xv[j] = 0.f;
        }
        for (int e8 = 0; e8 < E; e8 += 8) {
          uint4 wr[kRJ];
#pragma unroll
          for (int j = 0; j < kRJ; ++j)
            wr[j] = e8 == 0 ? wr0[j]
                            : __ldg(reinterpret_cast<const uint4*>(P.w_router +
                                                                   (size_t)min(tid + j * kConsumerThreads, d - 1) * E + e8));
          float a[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) a[j] = 0.f;
#pragma unroll
          for (int j = 0; j < kRJ; ++j) {
            float w[8];
            unpack8(wr[j], w);
#pragma unroll
            for (int q = 0; q < 8; ++q) a[q] = fmaf(xv[j], w[q], a[q]);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float t = warp_sum(a[j]);
            if (lane == 0) sm.rlog[warp][e8 + j] = t;
          }
        }
      } else {
        for (int e = 0; e < E; ++e) {
          float a = 0.f;
          for (int i = tid; i < d; i += kConsumerThreads) {
            const float xv = P.x_is_bf16 ? bf16_to_float(((const uint16_t*)xsrc)[i]) : ((const float*)xsrc)[i];
            a = fmaf(xv, bf16_to_float(__ldg(P.w_router + (size_t)i * E + e)), a);
          }
          a = warp_sum(a);
          if (lane == 0) sm.rlog[warp][e] = a;
        }
      }
    }
    float bias0 = 0.f, bias1 = 0.f;
    if (warp == 0 && P.b_router) {  // fetched while the logits are being reduced
      if (lane < P.E) bias0 = P.b_router[lane];
      if (lane + 32 < P.E) bias1 = P.b_router[lane + 32];
    }
    __syncthreads();
    // token row 0 was written by the consumer threads (input formed from h): it counts as landed
    if (from_h && tid == kConsumerThreads) mbar_arrive(&sm.xfull[0]);
    if (warp == 0) {
      // This warp alone stands between the logits and the first weight copy: everything below stays in registers.
      // The eight warps' partial logits are fetched together and summed in a fixed tree.
      float l0 = bias0, l1 = bias1;
      if (lane < P.E) {
        float v[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) v[w] = sm.rlog[w][lane];
        l0 += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
      }
      if (lane + 32 < P.E) {
        float v[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) v[w] = sm.rlog[w][lane + 32];
        l1 += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
      }
      int e = 0;
      float wv = 0.f;
      unsigned long long selmask = 0ull;
      if (P.ex.use_forced) {
        warp_route_forced(l0, l1, P.E, P.k, P.renorm, lane, P.ex.forced, sm.stage_e, sm.stage_w);
        __syncwarp();
        if (lane < P.k) e = sm.stage_e[lane], wv = sm.stage_w[lane];
        const unsigned lo = __reduce_or_sync(0xffffffffu, (lane < P.k && e < 32) ? 1u << e : 0u);
        const unsigned hi = __reduce_or_sync(0xffffffffu, (lane < P.k && e >= 32) ? 1u << (e - 32) : 0u);
        selmask = (unsigned long long)lo | ((unsigned long long)hi << 32);
      } else {
        warp_route_top(l0, l1, P.E, P.k, P.renorm, lane, nullptr, e, wv, selmask);
      }
      // the k selected experts in ascending order are the active experts, one slot (token 0) each; act_off,
      // slot_tok and n_act do not depend on the selection and were written in the prologue
      if (lane < P.k) {
        const int rank = __popcll(selmask & ((1ull << e) - 1ull));
        const int sl = given_slot >= 0 ? given_slot : (P.expert_slot ? P.expert_slot[e] : e);
        if (sl < 0) flag_error(st, MOE_ERR_STATE, 0x301u);
        sm.act_e[rank] = e;
        sm.act_slot[rank] = sl < 0 ? 0 : sl;
        sm.slot_w[rank] = wv;
        if (blockIdx.x == 0) {
          if (P.topk_idx) P.topk_idx[lane] = e;
          if (P.topk_w) P.topk_w[lane] = wv;
        }
      }
    } else {
      // meanwhile the other warps work out this CTA's share: it depends on the number of active experts only
      pass_init(sm, P.f, pit, true, (unsigned)P.k);
      pass_known = true;
      // The producer thread readies its first stages now: which hidden units they cover depends on the launch shape
      // only, so their barriers are armed here and, once the expert is known, the copies go out from a loop of a
      // few instructions -- the general issue loop below is cold code at that point (its instructions come from L2,
      // a few hundred cycles per line), and warms up while these copies are on their way.
      // (a CTA that works for one expert; with dynamic hand-out the first stages come from its static share)
      if (!kAllX && tid == kConsumerThreads && pit.cta_c > 0 && next_pass(sm, P.f, pit, ps)) {
        const int n_st = (P.f + kRows - 1) / kRows;
        const int dyn_s0 = P.dyn ? n_st / (2 * pit.cta_c) : 0;
        const int first = P.dyn ? pit.cta_j * dyn_s0 * kRows : ps.ra;  // first hidden unit this CTA streams
        const int whole = P.dyn ? min(dyn_s0, (P.f - first) / kRows) : (ps.rb - ps.ra) / kRows;  // stages of kRows units
        pre_n = min(min(kPreStages, NS), whole);
        for (int i = 0; i < pre_n; ++i) {
          if (P.dyn) sm.stage_n[i] = kRows;
          mbar_arrive_expect_tx(&sm.full[i], (uint32_t)kRows * (uint32_t)(3 * P.d * 2));
        }
        pre_off = (size_t)(P.ex.unit_lo + first) * (size_t)(3 * P.d * 2);
        pre_stage = 1;
      }
    }
  } else if (kAllX && P.fused_route) {
    // several tokens, E a multiple of 8 (Eq. 2, Eq. 3); every CTA routes all tokens.  A thread owns the input
    // features tid, tid + 256, ...: their router rows are fetched once and serve every token; the tokens go
    // four at a time so that all their loads are in flight together.
    float* part = sm.scratch;  // [warp][16 tokens][16 experts]
    constexpr int XJ = (V == V_MMA_BF16_S || V == V_MMA_F32_S) ? 4 : kXIters;  // features per thread
    constexpr int TC = 32 / XJ;                                                // tokens per round trip
    __syncthreads();  // the barriers the producer thread initialised are waited on below
    if (warp < kWarps) {
      const int d = P.d, E = P.E;
      if (!mbar_wait(&sm.xfull[0], 0u) && lane == 0) set_abort(st, sm, 0x317u);
      for (int e8 = 0; e8 < E; e8 += 8) {
        uint4 wr[XJ];
#pragma unroll
        for (int j = 0; j < XJ; ++j)
          wr[j] = e8 == 0 ? wr0[j]
                          : __ldg(reinterpret_cast<const uint4*>(P.w_router +
                                                                 (size_t)min(tid + j * kConsumerThreads, d - 1) * E + e8));
        for (int t0 = 0; t0 < P.T; t0 += TC) {
          float xv[TC][XJ];
#pragma unroll
          for (int tt = 0; tt < TC; ++tt) {
            const size_t rowo = (size_t)min(t0 + tt, P.T - 1) * d;
#pragma unroll
            for (int j = 0; j < XJ; ++j) {
              const int i = tid + j * kConsumerThreads;
              if (i < d)
                xv[tt][j] = P.x_is_bf16 ? bf16_to_float(((const uint16_t*)xs)[rowo + i]) : ((const float*)xs)[rowo + i];
              else
                xv[tt][j] = 0.f;
            }
          }
#pragma unroll
          for (int tt = 0; tt < TC; ++tt) {
            float a[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) a[q] = 0.f;
#pragma unroll
            for (int j = 0; j < XJ; ++j) {
              float w[8];
              unpack8(wr[j], w);
#pragma unroll
              for (int q = 0; q < 8; ++q) a[q] = fmaf(xv[tt][j], w[q], a[q]);
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float v = warp_sum(a[q]);
              if (lane == 0 && t0 + tt < P.T) part[(warp * 16 + t0 + tt) * 16 + e8 + q] = v;
            }
          }
        }
      }
    }
    const float bias = (P.b_router && lane < P.E) ? P.b_router[lane] : 0.f;
    __syncthreads();
    if (warp < kWarps) {
      for (int t = warp; t < P.T; t += kWarps) {
        float l0 = 0.f, l1 = 0.f;
        if (lane < P.E) {
          for (int w = 0; w < kWarps; ++w) l0 += part[(w * 16 + t) * 16 + lane];
          l0 += bias;
        }
        warp_route_finish(l0, l1, P.E, P.k, P.renorm, lane, sm.stage_e + t * P.k, sm.stage_w + t * P.k, nullptr);
        __syncwarp();
        if (blockIdx.x == 0 && lane < P.k) {
          if (P.topk_idx) P.topk_idx[t * P.k + lane] = sm.stage_e[t * P.k + lane];
          if (P.topk_w) P.topk_w[t * P.k + lane] = sm.stage_w[t * P.k + lane];
        }
      }
    }
  } else if (given1) {
    // one token, routing given: the entries of topk_idx / topk_w this launch was asked for, ascending by expert
    if (warp == 0) {
      const bool mine = lane < P.k && ((P.ex.sel_mask >> lane) & 1u);
      int e = mine ? P.topk_idx[lane] : -1;
      const float wv = mine ? P.topk_w[lane] : 0.f;
      int bad = mine && (e < 0 || e >= P.E);
      if (bad) e = -1;
      int rank = 0;
      for (int i = 0; i < P.k; ++i) {
        const int ei = __shfl_sync(0xffffffffu, e, i);
        rank += (ei >= 0 && ei < e);
      }
      const int na = __popc(__ballot_sync(0xffffffffu, e >= 0));
      if (e >= 0) {
        const int given = P.ex.slot_of_entry[lane];
        const int sl = given >= 0 ? given : (P.expert_slot ? P.expert_slot[e] : e);
        bad |= sl < 0;
        sm.act_e[rank] = e;
        sm.act_slot[rank] = sl < 0 ? 0 : sl;
        sm.act_off[rank] = rank;
        sm.slot_tok[rank] = 0;
        sm.slot_w[rank] = wv;
      }
      bad = __any_sync(0xffffffffu, bad);
      if (lane == 0) {
        sm.act_off[bad ? 0 : na] = bad ? 0 : na;
        sm.n_act = bad ? 0 : na;
        if (bad) flag_error(st, MOE_ERR_STATE, 0x302u);
      }
    }
  } else if (kAllX && P.mode == 0 && warp == 0) {
    for (int p = lane; p < n_pairs; p += 32) {
      sm.stage_e[p] = P.topk_idx[p];
      sm.stage_w[p] = P.topk_w[p];
    }
  }
  if (!fused1) __syncthreads();  // (one token with the router fused: nothing happens between this barrier and the next)
  if (kAllX && warp == 0 && !fused1 && !given1 && P.mode == 0) {
    // routing products -> active experts and their slots (same numbering as moe_permute): lane e works for
    // experts e and e + 32
    const int n = n_pairs, E = P.E;
    const unsigned below = (1u << lane) - 1u;
    int bad = 0;
    sm.cursor[lane] = 0, sm.cursor[lane + 32] = 0;
    __syncwarp();
    // counts: the pairs 32 at a time, one per lane; the first lane of each group of equal experts adds the group
    for (int p0 = 0; p0 < n; p0 += 32) {
      const int p = p0 + lane;
      int e = p < n ? sm.stage_e[p] : -1;
      if (p < n && (e < 0 || e >= E)) bad = 1, e = -1;
      const unsigned peers = __match_any_sync(0xffffffffu, e);
      if (e >= 0 && (peers & below) == 0u) sm.cursor[e] += __popc(peers);
      __syncwarp();
    }
    const int c0 = sm.cursor[lane], c1 = sm.cursor[lane + 32];
    int s0 = c0, s1 = c1;  // inclusive scans over the lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v0 = __shfl_up_sync(0xffffffffu, s0, o), v1 = __shfl_up_sync(0xffffffffu, s1, o);
      if (lane >= o) s0 += v0, s1 += v1;
    }
    const int tot0 = __shfl_sync(0xffffffffu, s0, 31);
    const int off0 = s0 - c0, off1 = tot0 + s1 - c1;
    const unsigned m0 = __ballot_sync(0xffffffffu, c0 > 0), m1 = __ballot_sync(0xffffffffu, c1 > 0);
    const int na = __popc(m0) + __popc(m1);
    int sl0 = lane, sl1 = lane + 32;
    if (P.expert_slot) {
      if (c0 > 0) sl0 = P.expert_slot[lane];
      if (c1 > 0) sl1 = P.expert_slot[lane + 32];
    }
    bad |= (c0 > 0 && sl0 < 0) || (c1 > 0 && sl1 < 0);
    bad = __any_sync(0xffffffffu, bad);
    if (c0 > 0) {
      const int a = __popc(m0 & below);
      sm.act_e[a] = lane, sm.act_off[a] = off0, sm.act_slot[a] = sl0 < 0 ? 0 : sl0;
    }
    if (c1 > 0) {
      const int a = __popc(m0) + __popc(m1 & below);
      sm.act_e[a] = lane + 32, sm.act_off[a] = off1, sm.act_slot[a] = sl1 < 0 ? 0 : sl1;
    }
    __syncwarp();
    sm.cursor[lane] = off0, sm.cursor[lane + 32] = off1;  // next free slot of every expert
    __syncwarp();
    if (!bad) {
      for (int p0 = 0; p0 < n; p0 += 32) {
        const int p = p0 + lane;
        const int e = p < n ? sm.stage_e[p] : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        const int base = e >= 0 ? sm.cursor[e] : 0;
        __syncwarp();
        if (e >= 0) {
          const int sl = base + __popc(peers & below);  // pairs of one expert keep their order
          sm.slot_tok[sl] = p / P.k;
          sm.slot_w[sl] = sm.stage_w[p];
          if ((peers & below) == 0u) sm.cursor[e] = base + __popc(peers);
        }
        __syncwarp();
      }
    }
    if (lane == 0) {
      sm.act_off[bad ? 0 : na] = bad ? 0 : n;
      sm.n_act = bad ? 0 : na;  // every CTA takes the same decision from the same data: no CTA streams anything
      if (bad) flag_error(st, MOE_ERR_STATE, 0x300u);
    }
  }
  if (tid == 0 && !fused1 && P.mode != 0) {
    // the caller's grouping (moe_permute's products) -> active experts and their slots
    const int n = n_pairs;
    int na = 0, bad = 0;
    sm.act_off[0] = 0;
    {
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
      flag_error(st, MOE_ERR_STATE, 0x300u);
      na = 0;  // every CTA takes the same decision from the same data: no CTA streams anything
    }
    sm.n_act = na;
  }
  __syncthreads();

  if (!pass_known) pass_init(sm, P.f, pit, fused1, (unsigned)P.k);
  RingPos rp{0, 0u, 0};

  if (warp == kProducerWarp) {
    // ================================================================= producer
    if (lane != 0) return;
    const uint32_t row_bytes = (uint32_t)(3 * P.d * 2);
    const uint32_t xrow_bytes = (uint32_t)P.d * (P.x_is_bf16 ? 2u : 4u);
    bool ok = true;
    int pn = 0, pn_issued = 0;
    int last_idx0 = -1, last_idx1 = -1;  // ring index of the last stage of the pass that used xs[0 / 1] before
    int known_free = -1;         // every ring index <= known_free has been released by the consumers
    unsigned copy_mask = 0;
    if (pre_n > 0) {  // the stages armed before the routing was known: only the expert was missing
      const unsigned char* src0 = reinterpret_cast<const unsigned char*>(P.gud) +
                                  (size_t)sm.act_slot[ps.ai] * P.f_full * row_bytes + pre_off;
      for (int i = 0; i < pre_n; ++i, src0 += kRows * row_bytes)
        bulk_g2s_hint(ring + (size_t)i * P.stage_bytes, src0, kRows * row_bytes, &sm.full[i], stream_policy);
    }
    while (ok && (pre_stage == 1 || next_pass(sm, P.f, pit, ps))) {
      const int skip = pre_stage == 1 ? pre_n : 0;  // stages of this pass that are already on their way
      pre_stage = 2;
      const int b = pn & 1;
      if (!kAllX && (b ? last_idx1 : last_idx0) > known_free) {
        const int L = b ? last_idx1 : last_idx0;
        if (!mbar_wait(&sm.freeb[L % NS], (unsigned)(L / NS) & 1u)) {
          set_abort(st, sm, 0x331u);
          ok = false;
          break;
        }
        known_free = L;
      }
      // the pass's token rows (pass 0 of a single-token launch: already on its way since the prologue)
      const int slot0 = sm.act_off[ps.ai] + ps.s0;
      ++pn_issued;
      if (!kAllX && !(fused1 && pn == 0)) {
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&sm.xfull[b], (uint32_t)ps.ns * xrow_bytes);
        for (int s = 0; s < ps.ns; ++s)
          bulk_g2s(xs + (size_t)b * P.xs_bytes + (size_t)s * xrow_bytes,
                   (const unsigned char*)P.x + (size_t)sm.slot_tok[slot0 + s] * xrow_bytes, xrow_bytes, &sm.xfull[b]);
      }
      const unsigned char* src = reinterpret_cast<const unsigned char*>(P.gud) +
                                 ((size_t)sm.act_slot[ps.ai] * P.f_full + P.ex.unit_lo + ps.ra + skip * kRows) * row_bytes;
      // Dynamic hand-out (one token, one pass per CTA): the CTAs of an expert do not stream at the same rate -- equal
      // shares end up to 4 us apart at the phone shape -- so a CTA takes half of its equal share of the
      // expert's stages (4 hidden units each) statically and then draws single stages from the expert's counter until
      // none is left.  A stage with zero units tells the consumers that the pass is over.
      const int n_st = (P.f + kRows - 1) / kRows;
      const int dyn_s0 = P.dyn ? n_st / (2 * pit.cta_c) : 0;
      int dyn_next = pit.cta_j * dyn_s0 + skip;
      const int dyn_stat_end = pit.cta_j * dyn_s0 + dyn_s0, dyn_base = pit.cta_c * dyn_s0;
      for (int i = 0; i < skip; ++i) {
        copy_mask |= 1u << rp.slot;
        rp.advance(NS);
      }
      const int SR = kAllX ? P.stage_rows : kRows;  // hidden units per stage
      for (int row = ps.ra + skip * kRows; P.dyn || row < ps.rb; row += SR) {
        int cur = 0;
        if (P.dyn) {
          cur = dyn_next < dyn_stat_end ? dyn_next++ : dyn_base + (int)atomicAdd(&st->stage_ctr[ps.ai], 1u);
          if (cur >= n_st) cur = -1;
        }
        const int nrows = P.dyn ? (cur < 0 ? 0 : min(kRows, P.f - cur * kRows)) : min(SR, ps.rb - row);
        const uint32_t bytes = (uint32_t)nrows * row_bytes;
        if (rp.n >= NS) {
          if (!mbar_wait(&sm.freeb[rp.slot], rp.par ^ 1u)) {
            set_abort(st, sm, 0x330u);
            ok = false;
            break;
          }
          known_free = max(known_free, rp.n - NS);
        }
        if (sm.abort) {
          ok = false;
          break;
        }
        if (P.dyn) {
          sm.stage_n[rp.slot] = nrows;
          if (nrows == 0) {  // no stage left: the consumers leave on this one
            mbar_arrive(&sm.full[rp.slot]);
            rp.advance(NS);
            break;
          }
          src = reinterpret_cast<const unsigned char*>(P.gud) +
                ((size_t)sm.act_slot[ps.ai] * P.f_full + P.ex.unit_lo + (size_t)cur * kRows) * row_bytes;
        }
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&sm.full[rp.slot], bytes);
        if (P.use_mma) {  // one copy per hidden unit: the units are padded apart in shared memory
          for (uint32_t o = 0, u = 0; o < bytes; o += row_bytes, ++u)
            bulk_g2s_hint(ring + (size_t)rp.slot * P.stage_bytes + (size_t)u * P.unit_stride, src + o, row_bytes,
                          &sm.full[rp.slot], stream_policy);
        } else {
          bulk_g2s_hint(ring + (size_t)rp.slot * P.stage_bytes, src, bytes, &sm.full[rp.slot], stream_policy);
        }
        copy_mask |= 1u << rp.slot;
        src += bytes;
        rp.advance(NS);
      }
      if (b)
        last_idx1 = rp.n - 1;
      else
        last_idx0 = rp.n - 1;
      ++pn;
    }
    if ((fused1 || kAllX) && pn_issued == 0) (void)mbar_wait(&sm.xfull[0], 0u);  // the early copy of x must land
    if (!ok) {
      // copies already in flight must land before this CTA's shared memory goes away
      for (int back = 1; back <= NS && back <= rp.n; ++back) {
        const int j = rp.n - back;
        if ((copy_mask >> (j % NS)) & 1u) (void)mbar_wait(&sm.full[j % NS], (unsigned)(j / NS) & 1u);
      }
      if (kAllX)
        (void)mbar_wait(&sm.xfull[0], 0u);
      else
        for (int q = max(0, pn_issued - 2); q < pn_issued; ++q) (void)mbar_wait(&sm.xfull[q & 1], (unsigned)(q >> 1) & 1u);
    }
    return;
  }

  // ===================================================================== consumers
  unsigned cpar = 0;
  int passes_done = 0;
  {
    bool ok = true;
    int pn = 0;
    while (ok && next_pass(sm, P.f, pit, ps)) {
      const int b = kAllX ? 0 : (pn & 1);
      if (!mbar_wait(&sm.xfull[b], kAllX ? 0u : ((unsigned)(pn >> 1) & 1u))) {
        if (lane == 0) set_abort(st, sm, 0x312u);
        ok = false;
        break;
      }
      const unsigned char* xsb = xs + (size_t)b * P.xs_bytes;
      if (V == V_T1)
        ok = consume_pass_t1(P, sm, ps, ring, xsb, wpart, rp, cpar, warp, lane);
      else if (V == V_COLS)
        ok = consume_pass_cols(P, sm, ps, ring, xsb, rp, warp, lane);
      else if (V == V_MMA_BF16_S)
        ok = consume_pass_mma<true, 4, 8, kRowsWide>(P, sm, ps, ring, xsb, rp, warp, lane);
      else if (V == V_MMA_F32_S)
        ok = consume_pass_mma<false, 4, 8, kRowsWide>(P, sm, ps, ring, xsb, rp, warp, lane);
      else if (V == V_MMA_BF16_L)
        ok = consume_pass_mma<true, 8, 16, kRows>(P, sm, ps, ring, xsb, rp, warp, lane);
      else
        ok = consume_pass_mma<false, 8, 16, kRows>(P, sm, ps, ring, xsb, rp, warp, lane);
      ++pn;
    }
    passes_done = ok ? pn : -1;
  }
  // ------------------------------------------------------------------ all partial sums are out
  // (after an expired wait the warps may be out of step with this barrier: then it can expire too; the
  // status word is already set and nobody finalises)
  if (!kAllX && P.counted) {
    // ---------------------------------------------------------------- one token: the words count their arrivals
    // Every CTA adds to every output element exactly once (a CTA without a share adds zeros), into the copy
    // blockIdx % copies; CTA b finishes the elements [b d / G, (b + 1) d / G): thread (element, copy) polls its
    // word until the count is full, the copies of an element are summed over neighbouring lanes, the sum is
    // converted and stored and the words are left zero.  The wait is bounded like every other.
    const int G = (int)gridDim.x, b = (int)blockIdx.x, d = P.d, copies = P.acc_copies;  // copies: a power of two <= 32
    if (passes_done < 0) return;  // an expired wait: the status word is set, the pollers elsewhere give up on it
    if (passes_done == 0) {
      unsigned long long* dst = reinterpret_cast<unsigned long long*>(P.acc) + (size_t)(b % copies) * P.acc_copy_stride;
      for (int i = tid; i < d; i += kConsumerThreads) atomicAdd(dst + i, 1ull);
    }
    const int lo = (int)((long long)b * d / G), hi = (int)((long long)(b + 1) * d / G);
    const int per_round = kConsumerThreads / copies;  // elements handled at a time
    const unsigned bias = ld_relaxed(&st->tail_bias);  // 0 (the diagnostics hook: 1, a count the launch never reaches)
    for (int e0 = lo; e0 < hi; e0 += per_round) {
      const int el = e0 + tid / copies, c = tid % copies;
      const bool mine = el < hi;
      if (__ballot_sync(0xffffffffu, mine) == 0u) continue;  // (whole warps leave together: the shuffles below are warp-wide)
      const unsigned expect = (unsigned)((G - c + copies - 1) / copies) + bias;
      unsigned long long* word = reinterpret_cast<unsigned long long*>(P.acc) + (size_t)c * P.acc_copy_stride + (mine ? el : lo);
      unsigned long long v = 0ull;
      bool ok = true;
      const long long t0 = clock64();
      for (unsigned spins = 0;; ++spins) {
        v = ld_relaxed64(word);
        const bool full = !mine || (unsigned)(v & ((1ull << kCntBits) - 1ull)) == expect;
        if (__all_sync(0xffffffffu, full)) break;
        const bool give_up = (spins & 7u) == 7u && (clock64() - t0 > P.fin_wait_budget || ld_relaxed(&st->status) != 0u);
        if (__any_sync(0xffffffffu, give_up)) {
          ok = false;
          break;
        }
      }
      if (!ok) {
        if (lane == 0) flag_error(st, MOE_ERR_TIMEOUT, 0x341u);  // (keeps an earlier error code if one is set)
        break;
      }
      long long sum = (long long)v >> kCntBits;  // arithmetic shift: the count falls off, the sum keeps its sign
      if (!mine) sum = 0;
      for (int o = 1; o < copies; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (mine) {
        *word = 0ull;
        if (c == 0) {
          const float fv = (float)((double)sum * kFixInvCnt);
          if (P.ex.resid)
            P.ex.resid[el] += fv;  // h += y
          else if (P.x_is_bf16)
            ((__nv_bfloat16*)P.y)[el] = __float2bfloat16_rn(fv);
          else
            ((float*)P.y)[el] = fv;
        }
      }
      // CTA 0's first element is complete: every CTA has streamed its last stage, nobody draws stages any more
      if (b == 0 && e0 == lo && tid < MOE_MAX_TOPK) st->stage_ctr[tid] = 0u;
    }
    return;
  }
  bool fin = consumer_sync(sm, cpar, lane);
  if (!P.ex.finalize) return;  // a later launch of the group adds its share and finalises
  // The last kFinalizers CTAs to arrive turn the fixed-point sums into the output, one slice each, and leave
  // zeros behind.  All but the very last of them first wait (bounded) for the arrival counter to fill up: the
  // CTAs they wait for are running or can start on the SMs the finished ones have left.
  const unsigned G = gridDim.x, K = G < (unsigned)kFinalizers ? G : (unsigned)kFinalizers;
  if (tid == 0) {
    // (the barrier above orders every warp's accumulator atomics before this thread; the arrival below is a
    // release at GPU scope, so they are performed before the count moves -- no separate fence)
    const unsigned long long old_total = atom_add_acq_rel64(&st->done_total, 1ull);
    const unsigned old = (unsigned)(old_total % G);  // this CTA's arrival number within the launch
    const unsigned long long target = old_total - old + G;
    int slice = (int)old - (int)(G - K);
    if (slice >= 0 && old != G - 1u) {
      const long long t0 = clock64();
      for (;;) {
        // both words in one round trip: the status load is not ordered against the counter's, it only ends a wait
        // that an error elsewhere has made pointless
        const unsigned err = ld_relaxed(&st->status);
        if (ld_acquire64(&st->done_total) >= target) break;
        if (clock64() - t0 > P.fin_wait_budget || sm.abort || err != 0u) {
          flag_error(st, MOE_ERR_TIMEOUT, 0x340u);  // (keeps an earlier error code if one is set)
          slice = -1;
          break;
        }
      }
    }
    sm.last = slice;  // (published to the CTA by the barrier below; the counter was read with acquire loads)
  }
  fin = consumer_sync(sm, cpar, lane) && fin;
  const int slice = sm.last;
  if (fin && slice >= 0) {
    if (slice == 0 && tid < MOE_MAX_TOPK) st->stage_ctr[tid] = 0u;  // every CTA has arrived: nobody draws stages any more
    const int rows = P.mode == 0 ? P.T : n_pairs;
    const long long total = (long long)rows * P.d;
    const long long per = (total + K - 1) / K;
    const long long lo = per * slice, hi = lo + per < total ? lo + per : total;
    // (ordered after the full arrival count by the barrier above; an acquire here would hold the loads below back)
    const unsigned err_seen = ld_relaxed(&st->status);
    // four outputs per thread at a time: all their copies are fetched in one round trip, then summed,
    // converted, stored, and the copies zeroed
    for (long long i0 = lo + tid; i0 < hi; i0 += 4 * kConsumerThreads) {
      long long part[4][8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const long long i = i0 + (long long)j * kConsumerThreads;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          part[j][c] = (i < hi && c < P.acc_copies) ? __ldcg(P.acc + (size_t)c * P.acc_copy_stride + i) : 0ll;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const long long i = i0 + (long long)j * kConsumerThreads;
        if (i >= hi) continue;
        long long v = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          v += part[j][c];
          if (c < P.acc_copies) P.acc[(size_t)c * P.acc_copy_stride + i] = 0;
        }
        if (err_seen != 0u) continue;
        const float fv = (float)((double)v * kFixInv);
        if (P.mode == 1)
          P.out_slots[i] = fv;
        else if (P.ex.resid)
          P.ex.resid[i] += fv;  // h += y (one token; exactly one thread of one CTA owns element i)
        else if (P.x_is_bf16)
          ((__nv_bfloat16*)P.y)[i] = __float2bfloat16_rn(fv);
        else
          ((float*)P.y)[i] = fv;
      }
    }
  }
}

template <int V>
int launch_variant(const DenseParams& P, int grid, size_t smem, cudaStream_t s) {
  MOE_CUDA_TRY(cudaFuncSetAttribute(dense_stream_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(grid), lc.blockDim = dim3(kThreads), lc.dynamicSmemBytes = smem, lc.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr, lc.numAttrs = 1;
  MOE_CUDA_TRY(cudaLaunchKernelEx(&lc, dense_stream_kernel<V>, P));
  return MOE_OK;
}

}  // namespace

static_assert(MOE_STREAM_MAX_TOKENS <= 16, "the fused router's staging area holds 16 tokens");
bool dense_stream_fuses_route(const moe_config& c, int T) {
  return T == 1 || ((c.n_experts & 7) == 0 && c.n_experts <= 16);  // several tokens: 8 or 16 experts
}

int launch_dense_stream(moe_ctx* ctx, int mode, const void* x, int T, const moe_weights* w, int32_t* topk_idx,
                        float* topk_w, const int32_t* offsets, const int32_t* perm, void* y, float* out_slots,
                        cudaStream_t s, const DenseExtra* ex) {
  const moe_config& c = ctx->cfg;
  if (c.d_model > 32 * 8 * kXIters || !ctx->acc) return MOE_ERR_UNSUPPORTED;
  const bool routing_given = (mode == 2);  // mode 2: the whole layer, but with the caller's routing even at T == 1
  if (routing_given) mode = 0;
  DenseParams P{};
  P.T = T, P.k = c.top_k, P.E = c.n_experts, P.d = c.d_model, P.f = c.d_ff, P.mode = mode;
  P.x_is_bf16 = c.x_dtype == MOE_BF16, P.renorm = c.renorm;
  P.fused_route = (mode == 0 && !routing_given && dense_stream_fuses_route(c, T)) ? 1 : 0;
  P.x = x, P.w_router = (const uint16_t*)w->w_router, P.b_router = w->b_router;
  P.topk_idx = topk_idx, P.topk_w = topk_w, P.offsets = offsets, P.perm = perm;
  P.expert_slot = w->expert_slot, P.gud = (const uint16_t*)w->gud;
  P.y = y, P.out_slots = out_slots, P.st = ctx->d_state, P.acc = ctx->acc;
  P.f_full = c.d_ff;
  for (int j = 0; j < MOE_MAX_TOPK; ++j) P.ex.slot_of_entry[j] = -1;
  P.ex.sel_mask = 0xffffffffu, P.ex.finalize = 1;
  if (ex) {
    if (T != 1 || mode == 1) return MOE_ERR_INVALID_ARG;
    if ((ex->h_in || ex->use_forced) && !P.fused_route) return MOE_ERR_INVALID_ARG;
    P.ex = *ex;
    if (P.ex.sel_mask == 0u) P.ex.sel_mask = 0xffffffffu;
    if (P.ex.unit_cnt > 0) {
      if (P.ex.unit_lo < 0 || P.ex.unit_lo + P.ex.unit_cnt > c.d_ff) return MOE_ERR_INVALID_ARG;
      P.f = P.ex.unit_cnt;
    } else {
      P.ex.unit_lo = 0;
    }
  }
  P.given1 = (mode == 0 && T == 1 && !P.fused_route) ? 1 : 0;
  {
    // contended atomics on few lines are slow: with room in the accumulator buffer, CTAs use up to 8 copies
    const long long rows = (mode == 0) ? T : (long long)T * c.top_k;
    P.acc_copy_stride = rows * c.d_model;
    const long long fit = (long long)ctx->acc_elems / P.acc_copy_stride;
    if (fit < 1) return MOE_ERR_UNSUPPORTED;
    const long long want = rows >= 16 ? 1 : (16 / rows < 8 ? 16 / rows : 8);  // rows x copies of about 16 spread the atomics enough
    P.acc_copies = (int)(fit < want ? fit : want);
  }
  P.fin_wait_budget = ctx->fin_wait_budget > 0 ? ctx->fin_wait_budget : kWaitBudgetCycles;
  const int xrow = c.d_model * (P.x_is_bf16 ? 2 : 4);
  P.xs_bytes = T > 1 ? ((T * xrow + 1) / 2 + 127) / 128 * 128   // several tokens: the two buffers together hold all rows
                     : (xrow + 127) / 128 * 128;
  P.use_mma = T > 1 ? 1 : 0;
  P.unit_stride = 3 * c.d_model * 2 + (P.use_mma ? 16 : 0);  // multiple of 16; the ring base is 128-byte aligned
  P.stage_rows = (P.use_mma && c.d_model <= 1024) ? kRowsWide : kRows;
  P.stage_bytes = (P.stage_rows * P.unit_stride + 127) / 128 * 128;
  P.wpart_ok = (!P.use_mma && c.d_model <= 32 * 8 * kT1Iters) ? 1 : 0;
  const size_t fixed = 2 * (size_t)P.xs_bytes + (P.wpart_ok ? (size_t)kWarps * c.d_model * 4 : 0) + kSmemHeaderBytes + 256;
  const long long avail = (long long)ctx->max_smem_optin - (long long)fixed;
  if (avail < 2ll * P.stage_bytes) return MOE_ERR_UNSUPPORTED;
  P.n_stages = (int)min((long long)kMaxStages, avail / P.stage_bytes);
  const size_t smem = (size_t)P.n_stages * P.stage_bytes + fixed;
  const int G = ctx->sm_count;
  const int v = !P.use_mma ? (P.wpart_ok ? V_T1 : V_COLS)
                           : (c.d_model <= 1024 ? (P.x_is_bf16 ? V_MMA_BF16_S : V_MMA_F32_S)
                                                : (P.x_is_bf16 ? V_MMA_BF16_L : V_MMA_F32_L));
  P.dyn = (v == V_COLS && mode == 0 && T == 1 && P.ex.finalize && P.ex.unit_cnt == 0 &&
           (P.ex.sel_mask & ((1u << c.top_k) - 1u)) == (1u << c.top_k) - 1u &&
           G >= c.top_k && c.d_ff >= 8 * G)
              ? 1
              : 0;
  // one token and the whole layer in this launch: arrivals are counted in the accumulator words themselves
  P.counted = (mode == 0 && T == 1 && P.ex.finalize && P.ex.unit_cnt == 0 &&
               (P.ex.sel_mask & ((1u << c.top_k) - 1u)) == (1u << c.top_k) - 1u && G >= c.top_k && c.top_k <= 16 &&
               P.acc_copies >= 1 && P.acc_copies <= 32 && (P.acc_copies & (P.acc_copies - 1)) == 0 &&
               (G + P.acc_copies - 1) / P.acc_copies + 1 < (1 << kCntBits))
                  ? 1
                  : 0;
  int rc;
  switch (v) {
    case V_T1: rc = launch_variant<V_T1>(P, G, smem, s); break;
    case V_COLS: rc = launch_variant<V_COLS>(P, G, smem, s); break;
    case V_MMA_BF16_S: rc = launch_variant<V_MMA_BF16_S>(P, G, smem, s); break;
    case V_MMA_F32_S: rc = launch_variant<V_MMA_F32_S>(P, G, smem, s); break;
    case V_MMA_BF16_L: rc = launch_variant<V_MMA_BF16_L>(P, G, smem, s); break;
    default: rc = launch_variant<V_MMA_F32_L>(P, G, smem, s); break;
  }
  if (rc != MOE_OK) return rc;
  ctx->launches++;
  return MOE_OK;
}

}  // namespace cosmoe

// =====================================================================================================
// moe_layer_forward_static: the same layer for callers that must not allocate.
//
// The streaming kernel above needs scratch in global memory: the 64-bit fixed-point accumulators the CTAs
// add their partial outputs into, and a few words of state (status, arrival counter).  moe_create gets
// them from cudaMalloc.  Here they live in a file-scope __device__ array instead, so nothing is allocated,
// at the price of a fixed maximum problem size and of every call on a GPU sharing the one array.
// =====================================================================================================
namespace cosmoe {
namespace {

constexpr int kStaticMaxTokens = MOE_STREAM_MAX_TOKENS;  // 16
constexpr int kStaticMaxD = 32 * 8 * kXIters;            // 2048
constexpr size_t kStaticStateBytes = (sizeof(DeviceState) + 255) / 256 * 256;
constexpr size_t kStaticAccBytes = (size_t)kStaticMaxTokens * kStaticMaxD * sizeof(long long);  // 256 KiB
constexpr size_t kStaticBytes = kStaticStateBytes + kStaticAccBytes;

// Held by every GPU that loads the library, until the process exits.  In host code this name is only a
// handle for cudaGetSymbolAddress; it is not a device address and is never passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct StaticDevice {
  std::once_flag once;
  int rc;               // outcome of the one-off set-up
  unsigned char* base;  // device address of g_static_scratch on this GPU
  int sm_count, max_smem_optin;
};
StaticDevice g_static_dev[kMaxDevices];

int static_setup_once(int dev, StaticDevice& sd) {
  int major = 0;
  void* p = nullptr;
  MOE_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return MOE_ERR_NO_DEVICE;  // kernels are built for sm_100a only
  MOE_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
  MOE_CUDA_TRY(cudaDeviceGetAttribute(&sd.sm_count, cudaDevAttrMultiProcessorCount, dev));
  MOE_CUDA_TRY(cudaDeviceGetAttribute(&sd.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  sd.base = (unsigned char*)p;
  return MOE_OK;
}

// Once per device, with that device current: resolve the array's device address.  Safe to reach from several
// threads at once (std::call_once orders the set-up before every caller's use of its results).
int static_setup(int dev, StaticDevice** out) {
  if (dev < 0 || dev >= kMaxDevices) return MOE_ERR_UNSUPPORTED;
  StaticDevice& sd = g_static_dev[dev];
  std::call_once(sd.once, [&] { sd.rc = static_setup_once(dev, sd); });
  if (sd.rc != MOE_OK) return sd.rc;
  *out = &sd;
  return MOE_OK;
}

}  // namespace
}  // namespace cosmoe

extern "C" int moe_layer_forward_static(const moe_config* cfg, const void* x, int32_t T, const moe_weights* w, void* y,
                                        int32_t* topk_idx, float* topk_w, void* stream) {
  using namespace cosmoe;
  int rc = validate_config(cfg);
  if (rc != MOE_OK) return rc;
  if (T < 0) return MOE_ERR_INVALID_ARG;
  if (cfg->wd_rank != 0 || cfg->d_model > kStaticMaxD || T > kStaticMaxTokens) return MOE_ERR_UNSUPPORTED;
  int dev = 0;
  MOE_CUDA_TRY(cudaGetDevice(&dev));
  StaticDevice* sd = nullptr;
  rc = static_setup(dev, &sd);
  if (rc != MOE_OK) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  DeviceState* st = reinterpret_cast<DeviceState*>(sd->base);
  long long* acc = reinterpret_cast<long long*>(sd->base + kStaticStateBytes);
  if (T == 0) {
    // status query: what the kernels of earlier calls on this GPU reported
    DeviceState host{};
    MOE_CUDA_TRY(cudaMemcpyAsync(&host, st, sizeof(DeviceState), cudaMemcpyDeviceToHost, s));
    MOE_CUDA_TRY(cudaStreamSynchronize(s));
    if (host.status == 0) return MOE_OK;
    MOE_CUDA_TRY(cudaMemsetAsync(st, 0, sizeof(DeviceState), s));
    MOE_CUDA_TRY(cudaStreamSynchronize(s));
    return host.status == MOE_ERR_TIMEOUT ? MOE_ERR_TIMEOUT : MOE_ERR_STATE;
  }
  if (!x || !y || !w || !w->w_router || !w->gud) return MOE_ERR_INVALID_ARG;
  if (((uintptr_t)x | (uintptr_t)y | (uintptr_t)w->w_router | (uintptr_t)w->gud) & 15u) return MOE_ERR_INVALID_ARG;
  if (T > 1 && (!topk_idx || !topk_w)) return MOE_ERR_INVALID_ARG;
  // The array keeps what the last call left.  A call that ran to its end leaves the accumulators and the
  // arrival counter at zero, one that was cut short does not: clear the part this call uses, keep the status.
  MOE_CUDA_TRY(cudaMemsetAsync(&st->done_total, 0, offsetof(DeviceState, pad3) - offsetof(DeviceState, done_total), s));  // arrival and stage counters
  MOE_CUDA_TRY(cudaMemsetAsync(acc, 0, kStaticAccBytes, s));
  moe_ctx tmp{};  // a view, not a context: nothing here owns memory
  tmp.cfg = *cfg;
  tmp.cfg.path = MOE_PATH_STREAM;
  tmp.device = dev;
  tmp.sm_count = sd->sm_count;
  tmp.max_smem_optin = sd->max_smem_optin;
  tmp.d_state = st;
  tmp.h_state = nullptr;
  tmp.acc = acc;
  tmp.acc_elems = kStaticAccBytes / sizeof(long long);
  if (!dense_stream_fuses_route(tmp.cfg, T)) {
    rc = launch_route(&tmp, x, T, w, topk_idx, topk_w, nullptr, s);
    if (rc != MOE_OK) return rc;
  }
  return launch_dense_stream(&tmp, 0, x, T, w, topk_idx, topk_w, nullptr, nullptr, y, nullptr, s);
}
