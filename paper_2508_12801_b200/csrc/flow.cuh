// Token -> expert assignment: the min-cost max-flow of Eq. 7-8 on the network of Table 1, solved
// exactly on the GPU.
//
// Structure used.  The dual of the flow problem has one price p_e >= 0 per expert; given prices every
// token independently holds its k largest values of key(i, e) - p_e.  The solver therefore works on
// the E prices, never on the T x E arcs:
//
//   scan      (one warp per token) reads the score matrix once and keeps, per token, its 16 best experts
//             (score and index) with a rigorous bound on everything else: the token's candidate cache.
//   sweeps    (one persistent cooperative kernel, one thread per token) every token re-picks its top-k
//             under the current prices from its cache; per expert a load count, two histograms of margins
//             (how much a price rise makes a holder leave / how much a price cut makes an outsider join)
//             and the exact smallest margin are collected.  After a grid-wide barrier one warp per expert
//             moves the price of an over- or under-loaded expert to the histogram quantile that balances
//             it, plus a step eps that is halved as the sweeps go on; small imbalances move one exact
//             margin at a time.  This is an epsilon-scaled simultaneous price adjustment (auction-style);
//             it ends a few dozen token moves away from the optimum and stops early once a small imbalance
//             has stopped shrinking.  A token whose cache can no longer vouch for its top-(k+2) (the bound
//             on the uncached experts has come too close) is rescanned by a warp.  Whether prices may
//             fall below zero on the way (anchored afterwards) or keep their floor at zero, and whether a few
//             units of spare room are hidden at first, is decided from the loads of the first sweep (see
//             SweepArgs::slack and the comments at that decision).  The kernel ends by
//             writing every token's top-k under the final prices and listing the tokens whose k-th and
//             (k+1)-th values differ by at most theta as candidates.
//   records   per candidate, the experts it could give up or take within the arc window (whole GPU).
//   exact     one CTA runs successive shortest augmenting paths on the expert-level residual graph
//             (E experts + one node Z for the sink side); node potentials keep reduced costs
//             non-negative, so each search is a Bellman-Ford over E+1 nodes whose arcs are read off the
//             candidate records.  It ends with every expert within capacity and complementary slackness
//             satisfied for the candidates.
//   check     a data-parallel pass checks complementary slackness for EVERY token under the final prices
//             (from the cache where its bound allows, from the full row otherwise).  If a token is
//             violated it re-picks, theta grows and records/exact run again.  Passing this check is a
//             proof of optimality (LP duality of Eq. 7-8); the same pass gathers the statistics.
//
// All arithmetic is on int64 keys: key = rne(A * 2^40) (+ a 12-bit position hash) for float
// affinities, or the quantised logit with a hashed tie-break.
#pragma once
#include <cstddef>
#include <type_traits>
#include "common.cuh"

namespace msr {

constexpr int kNB = 256;                  // histogram bins per expert: 4 per octave of the margin
constexpr long long kInf = 1LL << 62;
constexpr long long kPriceLimit = 1LL << 56; // sweeps keep |price| below this
constexpr int kCapLogMax = 60;
constexpr int kStallSweeps = 3, kStallImbalance = 256;
constexpr int kExactNeed = 8;              // imbalances up to this are closed one exact margin at a time
constexpr int kEPLf = kMaxE / 32;          // experts per lane when a warp spans one token row

struct KeyGen {
  int mode;            // 0: float affinities, 1: quantised logits
  int quant_shift;
  uint32_t seed_mul;   // tiebreak_seed * 0x9E3779B9
  int S;               // shift of the quantised part
  float fshift, fS;    // 2^quant_shift and 2^S as floats (approximate keys)
};

__device__ __forceinline__ uint32_t fmix32(uint32_t h) {   // 32-bit finaliser of MurmurHash3
  h ^= h >> 16; h *= 0x85ebca6bu; h ^= h >> 13; h *= 0xc2b2ae35u; h ^= h >> 16;
  return h;
}

__device__ __forceinline__ long long make_key(const KeyGen& g, float x, uint32_t flat_idx) {
  if (!isfinite(x)) x = 0.f;   // reported separately by the scan
  // x * 2^40 is exact in fp32; the low 12 bits carry a multiplicative hash of the entry's position so
  // that identical rows do not tie exactly (it moves the optimum by less than 4e-9 per chosen pair)
  if (g.mode == 0) return __float2ll_rn(x * 1099511627776.0f) + (long long)((flat_idx * 2654435761u) >> 20);
  float sc = rintf(ldexpf(x, g.quant_shift));
  sc = fminf(fmaxf(sc, -32768.f), 32767.f);
  long long q = (long long)sc;
  uint32_t r = fmix32(flat_idx + g.seed_mul) >> 12;
  return q * (1LL << g.S) + (long long)r;
}

// Key in fp32 (24 significant bits): good enough to FIND the largest few entries of a row cheaply.
// key - approx_key lies in [-0.5, 4096.5) for float affinities and in [0, 2^20) for quantised logits.
__device__ __forceinline__ float approx_key(const KeyGen& g, float x) {
  if (!isfinite(x)) x = 0.f;
  if (g.mode == 0) return x * 1099511627776.0f;
  return fminf(fmaxf(rintf(x * g.fshift), -32768.f), 32767.f) * g.fS;
}


struct FlowState {
  long long p[kMaxE];        // expert prices
  long long theta;           // candidate threshold of the next listing
  long long theta_used;      // threshold the current candidate list was collected with
  long long cumdrop;         // bound on how much any expert's price has dropped since the caches were built
  double total_score;
  int load[kMaxE];           // accumulated by the running pass, consumed by its price step / last CTA
  int load_cur[kMaxE];       // loads of the assignment currently written in expert_idx
  int load0[kMaxE];          // loads of the first sweep (every price zero): how popular each expert is
  alignas(16) unsigned hist_up[2][kMaxE * kNB];   // [sweep parity]; read and cleared with 16-byte accesses
  alignas(16) unsigned hist_dn[2][kMaxE * kNB];
  long long min_up[kMaxE], min_dn[kMaxE];   // smallest margin recorded by the running sweep (reset by the price step)
  int cap_up[kMaxE], cap_dn[kMaxE];   // log2 of the largest margin worth recording
  int flag_dn[kMaxE];                 // expert whose join-histogram came out short: scan it in full next sweep
  int imb_e[kMaxE];                   // |load - C| of the experts that moved their price in the last price step
  long long drop_e[kMaxE];            // by how much the last price step lowered each price
  unsigned bar_count, bar_abort;      // grid-wide barrier of the sweeps kernel
  unsigned ticket;
  int sweep, balanced;
  int round, converged, done, ncand, violations, naug, rerouted;
  unsigned status;
  int ncand_last;
  int nrec, rec_overflow;             // entries of the exact phase's candidate records in use; set when they ran out
};

static_assert(offsetof(FlowState, hist_up) % 16 == 0 && offsetof(FlowState, hist_dn) % 16 == 0 && (kMaxE * kNB * 4) % 16 == 0,
              "histograms are accessed as uint4");

// ---------------------------------------------------------------------------------------------
__global__ void flow_init_kernel(FlowState* st, int cap0, long long theta0, int balanced, int E) {
  {   // both histogram buffers, by all CTAs of the launch
    uint4* zu = reinterpret_cast<uint4*>(st->hist_up[0]); uint4* zd = reinterpret_cast<uint4*>(st->hist_dn[0]);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 2 * kMaxE * kNB / 4; i += gridDim.x * blockDim.x) {
      zu[i] = make_uint4(0, 0, 0, 0); zd[i] = make_uint4(0, 0, 0, 0);
    }
  }
  if (blockIdx.x != 0) return;
  for (int e = threadIdx.x; e < kMaxE; e += blockDim.x) {
    st->p[e] = 0; st->load[e] = 0; st->load_cur[e] = 0; st->min_up[e] = kInf; st->min_dn[e] = kInf;
    st->cap_up[e] = cap0; st->cap_dn[e] = cap0; st->flag_dn[e] = 0; st->imb_e[e] = 0; st->drop_e[e] = 0;
  }
  if (threadIdx.x == 0) {
    st->theta = theta0; st->theta_used = theta0; st->total_score = 0.0; st->cumdrop = 0;
    st->bar_count = 0; st->bar_abort = 0;
    st->ticket = 0; st->sweep = 0; st->balanced = balanced;
    st->round = 0; st->converged = 0; st->done = 0; st->ncand = 0; st->violations = 0; st->naug = 0;
    st->rerouted = 0; st->status = 0; st->ncand_last = 0; st->nrec = 0; st->rec_overflow = 0;
  }
}

__device__ __forceinline__ bool last_block_arrives(unsigned* ticket) {
  __shared__ bool is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned t = atomicAdd(ticket, 1u);
    is_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (is_last) __threadfence();
  return is_last;
}

// Margin histograms are logarithmic with four bins per octave (a 2-bit mantissa): margins 0..3 have
// their own bins, a margin m >= 4 with top bit o falls in bin 4*(o-1) + (next two bits).  Every scale
// is resolved to 25 % at once, which matters when the scores are quantised (margins then cluster at
// multiples of the quantum, separated by gaps that a linear window would have to zoom across).
__device__ __forceinline__ int log_bin(long long m) {
  if (m < 4) return (int)m;
  const int o = 63 - __clzll(m);
  return 4 * (o - 1) + (int)((m >> (o - 2)) & 3);
}
__device__ __forceinline__ long long bin_lower_edge(int b) {
  if (b < 4) return b;
  const int o = b / 4 + 1, sub = b & 3;
  return (long long)(4 + sub) << (o - 2);
}

// Price step that moves `need` tokens across the threshold of one expert.  If the bin holding the
// need-th smallest margin also holds many more tokens, the step stops at that bin's lower edge:
// fewer tokens move, and the rest of the group then sits near zero margin, where the bins are fine.
// Otherwise the step goes to the bin's upper edge plus eps (capped by the bin width).  `cut` is the
// log2 of the largest margin the tokens were asked to record; if fewer than `need` lie below it the
// step goes to 2^cut and the cut-off is lifted for the next sweep.
// Computed by a whole warp: lane l holds bins 8l .. 8l+7 of the expert's histogram.
__device__ __forceinline__ long long price_step_warp(const uint4& ha, const uint4& hb, int need, long long eps, int& cut,
                                                     bool& window_short, int cut_max, long long m1) {
  const int lane = threadIdx.x & 31;
  const unsigned hv[8] = {ha.x, ha.y, ha.z, ha.w, hb.x, hb.y, hb.z, hb.w};
  unsigned mine = 0; int top = -1;
#pragma unroll
  for (int q = 0; q < 8; ++q) { mine += hv[q]; if (hv[q]) top = 8 * lane + q; }
  unsigned incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  const unsigned reach = __ballot_sync(0xffffffffu, incl >= (unsigned)need);
  window_short = false;
  if (!reach) {
    const int last = __reduce_max_sync(0xffffffffu, top);
    const long long step = cut < cut_max ? (1LL << cut) : (last >= 0 ? bin_lower_edge(last + 1) : 0);
    cut = cut_max;
    window_short = true;
    return step;
  }
  const int src = __ffs(reach) - 1;
  int pos = 0; unsigned cum = incl - mine, before = 0;
  if (lane == src) {
    unsigned c = incl - mine; bool found = false;
#pragma unroll
    for (int q = 0; q < 8; ++q) {                        // first bin of this lane at which the count is reached
      if (!found && c + hv[q] >= (unsigned)need) { pos = 8 * lane + q; before = c; cum = c + hv[q]; found = true; }
      c += hv[q];
    }
  }
  pos = __shfl_sync(0xffffffffu, pos, src);
  cum = __shfl_sync(0xffffffffu, cum, src);
  before = __shfl_sync(0xffffffffu, before, src);
  const long long lo = pos == 0 ? 0 : bin_lower_edge(pos), hi = bin_lower_edge(pos + 1);
  cut = min(cut_max, max(12, (pos >> 2) + 5));
  // end game: when a handful of tokens have to move and the bin would move more than that, move fewer
  // but exactly: everything below the bin, or else the single token with the smallest margin
  if (need <= kExactNeed && cum > (unsigned)need) {
    if (before > 0 && lo > 0) return lo;
    if (m1 < kInf) return m1 + 1;
  }
  if (cum <= 2u * (unsigned)need || lo == 0) {
    const long long w = hi - lo;
    return hi + (eps < w ? eps : w);
  }
  return lo;
}

// fp32 <-> unsigned integers that order the same way (for the integer warp reductions)
__device__ __forceinline__ unsigned flip_f32(float f) {
  const unsigned b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float unflip_f32(unsigned u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// Exact selection over one row held by a warp (lane l: entries l, l+32, ...).  Picks the `count`
// largest values (larger value first, lower expert index first on equal values), sets sel[] for the first
// `nsel` of them, and returns the values picked as number nsel (v_a) and nsel+1 (v_b), where reached.
// A 64-bit maximum is taken as three 32-bit warp reductions: high word, low word among the lanes that
// match the high word, lowest index among the entries that match both.
__device__ __forceinline__ void warp_select(const long long (&val)[kEPLf], int E, int count, bool (&sel)[kEPLf],
                                            long long& v_a, long long& v_b, int nsel) {
  const int lane = threadIdx.x & 31;
  unsigned hi[kEPLf], lo[kEPLf]; bool gone[kEPLf];
#pragma unroll
  for (int q = 0; q < kEPLf; ++q) {
    const unsigned long long u = (unsigned long long)val[q] ^ 0x8000000000000000ULL;   // order-preserving
    hi[q] = (unsigned)(u >> 32); lo[q] = (unsigned)u;
    gone[q] = lane + 32 * q >= E;
    sel[q] = false;
  }
  for (int r = 0; r < count && r < E; ++r) {
    unsigned mh = 0;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) if (!gone[q]) mh = max(mh, hi[q]);
    const unsigned bh = __reduce_max_sync(0xffffffffu, mh);
    unsigned ml = 0;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) if (!gone[q] && hi[q] == bh) ml = max(ml, lo[q]);
    const unsigned bl = __reduce_max_sync(0xffffffffu, ml);
    unsigned me = 0xffffffffu;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) if (!gone[q] && hi[q] == bh && lo[q] == bl) me = min(me, (unsigned)(lane + 32 * q));
    const unsigned be = __reduce_min_sync(0xffffffffu, me);
    const long long v = (long long)((((unsigned long long)bh << 32) | bl) ^ 0x8000000000000000ULL);
    if (r == nsel - 1) v_a = v;
    if (r == nsel) v_b = v;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q)
      if ((unsigned)(lane + 32 * q) == be) { gone[q] = true; if (r < nsel) sel[q] = true; }
  }
}

// ---------------------------------------------------------------------------------------------
// Per-token candidate cache.  A full scan of a token's row keeps its kCacheN best experts (score and
// index) and `bound` = an upper bound on key - price of every other expert at scan time, minus the
// total price drop up to then.  Later, every uncached expert is worth at most bound + (total price
// drop now), so while the (k+2)-th cached value stays at or above that, the cached entries still
// contain the token's k+2 best experts and the row need not be read again.
constexpr int kCacheN = 16;
struct SweepCache {
  float* x;              // [kCacheN][T] scores of the cached experts
  unsigned char* id;     // [T][kCacheN] their indices (255 = none)
  long long* bound;      // [T]
  unsigned char* raw;    // [T] 1 = scanned at zero prices: the cache also holds the token's best raw keys
};

// One warp rebuilds the cache of one token from its row under the prices sp (spf = the same as floats).
// Lane l looks at experts l, l+32, l+64, l+96: fp32 approximations of key - price, the expert index in
// the low 7 mantissa bits, mapped to unsigned integers that order the same way (0 = absent); kCacheN
// rounds of one warp reduction each pick the winners.  |approximation - exact| <= hash_bound +
// 2^-15 (|key| + |price|) (float conversion of the price, one rounding of the difference, the 7 index
// bits), which turns the last winner's approximate value into a rigorous bound on every loser.
__device__ __forceinline__ void rescan_row(const float* __restrict__ row, uint32_t flat, int tok, int T, int E,
                                           const KeyGen& g, const long long* sp, const float* spf, long long cumdrop,
                                           bool raw, const SweepCache& cache, bool& bad) {
  const int lane = threadIdx.x & 31;
  unsigned u[kEPLf]; float mag = 0.f;
#pragma unroll
  for (int q = 0; q < kEPLf; ++q) {
    const int e = lane + 32 * q;
    u[q] = 0;
    if (e < E) {
      const float x = __ldg(row + e);
      bad |= !isfinite(x);
      const float kf = approx_key(g, x), pf = spf[e];
      const float vf = kf - pf;
      mag = fmaxf(mag, fabsf(kf) + fabsf(pf));
      const unsigned bits = (__float_as_uint(vf) & ~127u) | (unsigned)e;
      u[q] = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
    }
  }
  unsigned mine = 0;
  for (int r = 0; r < kCacheN; ++r) {
    unsigned m = u[0];
#pragma unroll
    for (int q = 1; q < kEPLf; ++q) m = max(m, u[q]);
    const unsigned w = __reduce_max_sync(0xffffffffu, m);
    if (lane == r) mine = w;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) u[q] = (u[q] == w) ? 0u : u[q];
  }
  // lanes 0..kCacheN-1 now hold the winners in descending approximate order
  int ee = 255; float xv = 0.f;
  if (lane < kCacheN && mine != 0) {
    const unsigned bits = (mine & 0x80000000u) ? (mine & 0x7fffffffu) : ~mine;
    ee = (int)(bits & 127u);
    xv = __ldg(row + ee);
  }
  if (lane < kCacheN) {
    cache.x[(size_t)lane * T + tok] = xv;
    cache.id[(size_t)tok * kCacheN + lane] = (unsigned char)ee;
  }
  mag = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mag)));
  const unsigned wlast = __shfl_sync(0xffffffffu, mine, kCacheN - 1);
  if (lane == 0) {
    long long b = -kInf;                                // fewer than kCacheN experts: nothing is left out
    if (wlast != 0) {
      const float a = __uint_as_float((wlast & 0x80000000u) ? (wlast & 0x7fffffffu) : ~wlast);
      const double ub = (double)a + (double)(g.mode == 0 ? 4097.f : 1048577.f) + (double)mag * (1.0 / 32768.0) + 1.0;
      b = ub >= 4.0e18 ? kInf : (ub <= -4.0e18 ? -kInf : (long long)ceil(ub));
      if (b < kInf && b > -kInf) b -= cumdrop;
    }
    cache.bound[tok] = b;
    cache.raw[tok] = raw ? 1 : 0;
  }
}

// First pass over the score matrix: the cache of every token at zero prices, one warp per token.
__global__ void __launch_bounds__(256)
flow_scan_kernel(const float* __restrict__ M, FlowState* st, SweepCache cache, int T, int E, KeyGen g) {
  __shared__ long long sp[kMaxE];
  __shared__ float spf[kMaxE];
  for (int e = threadIdx.x; e < kMaxE; e += blockDim.x) { sp[e] = 0; spf[e] = 0.f; }
  __syncthreads();
  const int wid = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), nwarp = gridDim.x * (blockDim.x >> 5);
  bool bad = false;
  for (int tok = wid; tok < T; tok += nwarp)
    rescan_row(M + (size_t)tok * E, (uint32_t)tok * (uint32_t)E, tok, T, E, g, sp, spf, 0, true, cache, bad);
  if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(&st->status, 2u);
}

// ---------------------------------------------------------------------------------------------
// Grid-wide barrier of the cooperative sweeps kernel: a monotone arrival counter in global memory.
// Every wait is bounded: a CTA that gives up raises the abort flag, which releases all the others,
// and the kernel then returns with the internal-error status set.
constexpr unsigned kBarrierSpinLimit = 1u << 22;
__device__ __forceinline__ bool grid_barrier(FlowState* st, unsigned& epoch) {
  __syncthreads();
  __shared__ int s_bar_ok;
  if (threadIdx.x == 0) {
    epoch += gridDim.x;
    __threadfence();
    atomicAdd(&st->bar_count, 1u);
    bool ok = true;
    for (unsigned spins = 0;; ++spins) {
      unsigned c;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(c) : "l"(&st->bar_count) : "memory");
      if ((int)(c - epoch) >= 0) break;
      if (spins > kBarrierSpinLimit || *(volatile unsigned*)&st->bar_abort) {
        atomicExch(&st->bar_abort, 1u); atomicOr(&st->status, 4u); ok = false; break;
      }
      if (spins > 64) __nanosleep(20);
    }
    s_bar_ok = ok ? 1 : 0;
  }
  __syncthreads();
  return s_bar_ok != 0;
}

// Bin of a non-negative margin held as a float: the same bins as log_bin (exponent and two mantissa bits).
__device__ __forceinline__ int float_bin(float m) {
  if (m < 4.f) return (int)m;
  const unsigned b = __float_as_uint(m);
  return 4 * ((int)(b >> 23) - 128) + (int)((b >> 21) & 3u);
}

// A margin goes into the expert's global histogram (fire-and-forget) and, for the steps that move one token
// exactly, into the CTA's running minimum in shared memory (merged into global memory after the pass;
// non-negative floats order like their bit patterns).
__device__ __forceinline__ void emit_margin(unsigned* hist, unsigned* smin, const float* capf, int e, float m) {
  if (m >= 0.f && m < capf[e]) {
    atomicAdd(&hist[e * kNB + float_bin(m)], 1u);
    const unsigned mb = __float_as_uint(m);
    if (mb < smin[e]) atomicMin(&smin[e], mb);
  }
}

// The experts of a 128-bit mask in ascending order, as a token's row of expert_idx.
__device__ __forceinline__ void write_sorted_experts(int32_t* __restrict__ out, const unsigned (&hm)[4], int k) {
  int n = 0;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    unsigned m = hm[w];
    while (m && n < k) { const int b = __ffs(m) - 1; m &= m - 1; out[n++] = 32 * w + b; }
  }
}

constexpr int kSwThreads = 512;

struct SweepShared {
  long long sp[kMaxE];
  float spf[kMaxE];
  unsigned smin_up[kMaxE], smin_dn[kMaxE];   // smallest margins of the pass, as float bit patterns
  float capu[kMaxE], capd[kMaxE];            // margins at or above these are not recorded
  int sload[kMaxE], sflag[kMaxE], sdeaf[kMaxE];   // sdeaf: flagged experts that heard from no token at all
  int nflag, ndeaf, nslow, s_imb;
  long long s_drop, s_pmin;
  int slow[kSwThreads];
  int trim[kMaxE];                           // room the sweeps leave unused on purpose (see SweepArgs::slack)
  int l0[kMaxE], srt[kMaxE], s_nb, s_level, s_rem;
};

struct SweepArgs {
  int T, E, k, C, n_sweeps, balanced;
  long long eps0, eps_min, theta0;
  // E*C - T*k when that is positive but small (else 0).  Prices that may not fall below zero make the sweeps crawl
  // when almost every expert ends up full: the few experts that keep room pin the price floor and everyone else has
  // to climb away from it one sweep at a time.  So the sweeps then solve the problem with the spare room taken away
  // from the least popular experts (as much from each as brings them level), where prices are free to move both ways
  // as when nothing is spare; the pick anchors the lowest price at zero and the exact phase repairs what the guess
  // of who keeps the room got wrong.
  int slack;
};

struct TokCache {          // one token's cache entries in registers
  unsigned idws[4]; float x[kCacheN]; long long bound;
};
__device__ __forceinline__ void load_tok_cache(TokCache& c, const SweepCache& cache, int tok, int T) {
  const uint4 idv = __ldcg(reinterpret_cast<const uint4*>(cache.id + (size_t)tok * kCacheN));
  c.idws[0] = idv.x; c.idws[1] = idv.y; c.idws[2] = idv.z; c.idws[3] = idv.w;
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) c.x[j] = __ldcg(cache.x + (size_t)j * T + tok);
  c.bound = __ldcg(cache.bound + tok);
}

// One token of a sweep, from its cache, in fp32: the sweeps only steer the prices, so approximate values
// do (what they leave undone the exact phase repairs, and the first pick and the check pass are exact).
// Returns false when the cache cannot vouch for the token's k+2 best experts any more (the caller then has
// the row rescanned and calls again).
__device__ __forceinline__ bool sweep_token(const float* __restrict__ M, int tok, const TokCache& c, SweepShared& sh, const SweepArgs& a,
                                            const KeyGen& g, float cumdropf, unsigned* hup, unsigned* hdn) {
  const int E = a.E, k = a.k;
  const int need = min(k + 2, E);                       // sorted values a token has to know
  float v[kCacheN]; int rank[kCacheN];
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) {
    const int e = (int)((c.idws[j >> 2] >> (8 * (j & 3))) & 255u);
    v[j] = e < E ? approx_key(g, c.x[j]) - sh.spf[e] : -INFINITY;
    rank[j] = 0;
  }
#pragma unroll
  for (int j = 1; j < kCacheN; ++j)
#pragma unroll
    for (int i = 0; i < j; ++i) {
      const bool first = v[i] >= v[j];                  // the earlier entry wins a tie
      rank[j] += first ? 1 : 0; rank[i] += first ? 0 : 1;
    }
  float vk = -INFINITY, vk1 = -INFINITY, vneed = -INFINITY;
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) {
    if (rank[j] == k - 1) vk = v[j];
    if (rank[j] == k) vk1 = v[j];
    if (rank[j] == need - 1) vneed = v[j];
  }
  if (!(c.bound <= -kInf || vneed >= (float)c.bound + cumdropf)) return false;
  const bool has_alt = E > k;
  const int nflag = sh.nflag;
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) {
    const int e = (int)((c.idws[j >> 2] >> (8 * (j & 3))) & 255u);
    if (rank[j] < k) {
      atomicAdd(&sh.sload[e], 1);
      if (has_alt) emit_margin(hup, sh.smin_up, sh.capu, e, v[j] - vk1);        // price rise at which the token leaves e
    } else if (e < E) {
      bool rec = rank[j] <= k + 1;                                             // price cut at which the token joins e
      // experts whose join-histogram was short last time: count this token even if the expert is not among
      // its best alternatives
      for (int q = 0; q < nflag; ++q) rec |= sh.sflag[q] == e;
      if (rec) emit_margin(hdn, sh.smin_dn, sh.capd, e, vk - v[j]);
    }
  }
  // An expert that heard from no token at all (with a lopsided router the unpopular experts are in nobody's cache)
  // could never find the price at which anyone joins it: for those, one score per token is read from the matrix.
  const int ndeaf = sh.ndeaf;
  if (ndeaf) {
    unsigned cached[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < kCacheN; ++j) {
      const int e = (int)((c.idws[j >> 2] >> (8 * (j & 3))) & 255u);
#pragma unroll
      for (int w = 0; w < 4; ++w) if ((e >> 5) == w) cached[w] |= 1u << (e & 31);
    }
    for (int q = 0; q < ndeaf; ++q) {
      const int e = sh.sdeaf[q];
      const unsigned word = (e & 64) ? ((e & 32) ? cached[3] : cached[2]) : ((e & 32) ? cached[1] : cached[0]);
      if ((word >> (e & 31)) & 1u) continue;
      emit_margin(hdn, sh.smin_dn, sh.capd, e, vk - (approx_key(g, __ldg(M + (size_t)tok * E + e)) - sh.spf[e]));
    }
  }
  return true;
}

// One token of the first pick, from its cache, exact: the token's k best experts under the final prices go
// to expert_idx in ascending order, and the token is listed as a candidate when its k-th and (k+1)-th values
// are within theta.  Returns false when the cache cannot vouch for the token's k+1 best experts.
__device__ __forceinline__ bool pick_token(int tok, const TokCache& c, FlowState* st, SweepShared& sh, const SweepArgs& a,
                                           const KeyGen& g, long long cumdrop, int32_t* __restrict__ expert_idx,
                                           int32_t* __restrict__ cand) {
  const int E = a.E, k = a.k;
  const uint32_t flat = (uint32_t)tok * (uint32_t)E;
  const int need = min(k + 1, E);
  long long v[kCacheN]; int rank[kCacheN];
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) {
    const int e = (int)((c.idws[j >> 2] >> (8 * (j & 3))) & 255u);
    v[j] = e < E ? make_key(g, c.x[j], flat + e) - sh.sp[e] : -kInf;
    rank[j] = 0;
  }
#pragma unroll
  for (int j = 1; j < kCacheN; ++j)
#pragma unroll
    for (int i = 0; i < j; ++i) {
      const bool first = v[i] >= v[j];                  // the earlier entry wins a tie
      rank[j] += first ? 1 : 0; rank[i] += first ? 0 : 1;
    }
  long long vk = -kInf, vk1 = -kInf, vneed = -kInf;
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) {
    if (rank[j] == k - 1) vk = v[j];
    if (rank[j] == k) vk1 = v[j];
    if (rank[j] == need - 1) vneed = v[j];
  }
  if (!(c.bound <= -kInf || vneed >= c.bound + cumdrop)) return false;
  unsigned hm[4] = {0, 0, 0, 0};
#pragma unroll
  for (int j = 0; j < kCacheN; ++j) {
    const int e = (int)((c.idws[j >> 2] >> (8 * (j & 3))) & 255u);
    if (rank[j] < k && e < E) { hm[e >> 5] |= 1u << (e & 31); atomicAdd(&sh.sload[e], 1); }
  }
  write_sorted_experts(expert_idx + (size_t)tok * k, hm, k);
  if (E > k && vk - vk1 <= a.theta0) cand[atomicAdd(&st->ncand, 1)] = tok;     // the list has room for every token
  return true;
}

// All price sweeps and the first pick in one cooperative launch (every CTA resident, one thread per token
// and pass; the price step of expert e is taken by one warp of CTA e mod grid).  When the grid has a
// thread for every token, a token's cache entries stay in its thread's registers from sweep to sweep.
__global__ void __launch_bounds__(kSwThreads, 1)
flow_sweeps_kernel(const float* __restrict__ M, FlowState* st, SweepCache cache, int32_t* __restrict__ expert_idx,
                   int32_t* __restrict__ cand, SweepArgs a, KeyGen g) {
  __shared__ SweepShared sh;
  const int T = a.T, E = a.E, C = a.C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gtid = blockIdx.x * blockDim.x + tid, gsize = gridDim.x * blockDim.x;
  const bool resident = T <= gsize;
  bool hiding = false;                                     // spare room is hidden from the sweeps (see SweepArgs::slack)
  bool free_prices = a.balanced != 0;                      // prices may go below zero until they are anchored
  bool pending = false; long long pend_anchor = 0;         // an anchoring that the next price step still has to apply
  for (int e = tid; e < kMaxE; e += blockDim.x) sh.trim[e] = 0;
  unsigned epoch = 0;
  long long cumdrop = 0, eps = a.eps0;
  int best_imb = 0x7fffffff, stall = 0, sweep = 0;
  bool done = a.n_sweeps <= 0;
  TokCache mine;
  if (resident && gtid < T) load_tok_cache(mine, cache, gtid, T);

  // a pass over this CTA's tokens: one thread per token from the caches, then one warp per token whose
  // cache had to be rebuilt
  auto token_pass = [&](auto pick_tag, unsigned* hup, unsigned* hdn) {
    constexpr bool kPick = decltype(pick_tag)::value;
    for (int base = blockIdx.x * blockDim.x; base < T; base += gsize) {
      if (tid == 0) sh.nslow = 0;
      __syncthreads();
      const int tok = base + tid;
      bool was_slow = false;
      if (tok < T) {
        if (!resident) load_tok_cache(mine, cache, tok, T);
        const bool ok = kPick ? pick_token(tok, mine, st, sh, a, g, cumdrop, expert_idx, cand)
                              : sweep_token(M, tok, mine, sh, a, g, (float)cumdrop, hup, hdn);
        if (!ok) { sh.slow[atomicAdd(&sh.nslow, 1)] = tok; was_slow = true; }
      }
      __syncthreads();
      const int nslow = sh.nslow;
      if (nslow) {
        for (int s = warp; s < nslow; s += kSwThreads / 32) {
          const int t2 = sh.slow[s];
          bool bad = false;
          rescan_row(M + (size_t)t2 * E, (uint32_t)t2 * (uint32_t)E, t2, T, E, g, sh.sp, sh.spf, cumdrop, false, cache, bad);
          __syncwarp();
          if (lane == 0) {
            TokCache fresh;
            load_tok_cache(fresh, cache, t2, T);
            if (kPick) pick_token(t2, fresh, st, sh, a, g, cumdrop, expert_idx, cand);
            else sweep_token(M, t2, fresh, sh, a, g, (float)cumdrop, hup, hdn);
          }
        }
        __syncthreads();
        if (resident && was_slow) load_tok_cache(mine, cache, tok, T);
      }
    }
  };
  // prices, caps and flags for the next pass; on the way, what the last price step left behind
  auto load_state = [&]() {
    if (tid == 0) { sh.nflag = 0; sh.ndeaf = 0; sh.s_imb = 0; sh.s_drop = 0; }
    __syncthreads();
    for (int e = tid; e < E; e += blockDim.x) {
      const long long pe = __ldcg(&st->p[e]);
      const int cu = __ldcg(&st->cap_up[e]), cd = __ldcg(&st->cap_dn[e]), fl = __ldcg(&st->flag_dn[e]);
      const int im = __ldcg(&st->imb_e[e]); const long long dr = __ldcg(&st->drop_e[e]);
      sh.sp[e] = pe; sh.spf[e] = (float)pe; sh.sload[e] = 0; sh.capu[e] = ldexpf(1.f, cu); sh.capd[e] = ldexpf(1.f, cd);
      sh.smin_up[e] = 0x7f800000u; sh.smin_dn[e] = 0x7f800000u;
      if (fl) sh.sflag[atomicAdd(&sh.nflag, 1)] = e;
      if (fl == 2) sh.sdeaf[atomicAdd(&sh.ndeaf, 1)] = e;
      if (im) atomicAdd(&sh.s_imb, im);
      if (dr > 0) atomicMax(&sh.s_drop, dr);
    }
    __syncthreads();
  };

  // Anchoring (every CTA does the same to its copy of the prices).
  auto anchor_prices = [&]() -> long long {
      // Prices are only defined up to a shift when every expert must be full: anchor the minimum at 0.  A uniform shift
      // moves every value of a token alike, the bound on its uncached experts included.
      // With spare room hidden, the experts that gave up room are the ones that will keep it, so they belong at price
      // zero: the anchor is the highest price among them, and whoever is cheaper still is lifted to zero as well (these
      // fell less than the anchor, which therefore still bounds every expert's fall).
      __syncthreads();
      if (tid == 0) {
        long long m = kInf;
        if (a.slack > 0) {
          m = -kInf;
          for (int e = 0; e < E; ++e) if (sh.trim[e] > 0 && sh.sp[e] > m) m = sh.sp[e];
        }
        if (m >= kInf || m <= -kInf) { m = sh.sp[0]; for (int e = 1; e < E; ++e) m = sh.sp[e] < m ? sh.sp[e] : m; }
        sh.s_pmin = m;
      }
      __syncthreads();
      const long long pmin = sh.s_pmin;
      for (int e = tid; e < E; e += blockDim.x) {
        const long long pe = sh.sp[e] - pmin;
        sh.sp[e] = pe < 0 ? 0 : pe; sh.spf[e] = (float)sh.sp[e];
      }
      cumdrop += pmin;
      __syncthreads();
    return pmin;
  };

  load_state();
  while (!done) {
    const int par = sweep & 1;
    unsigned* hup = st->hist_up[par]; unsigned* hdn = st->hist_dn[par];
    {   // every CTA clears a slice of the other pair of histograms for the next sweep (its last reader,
        // the previous price step, finished before the barrier that let this sweep start)
      uint4* zu = reinterpret_cast<uint4*>(st->hist_up[par ^ 1]); uint4* zd = reinterpret_cast<uint4*>(st->hist_dn[par ^ 1]);
      for (int i = gtid; i < kMaxE * kNB / 4; i += gsize) { zu[i] = make_uint4(0, 0, 0, 0); zd[i] = make_uint4(0, 0, 0, 0); }
    }
    token_pass(std::false_type{}, hup, hdn);
    for (int e = tid; e < E; e += blockDim.x) {
      if (sh.sload[e]) atomicAdd(&st->load[e], sh.sload[e]);
      if (sh.smin_up[e] < 0x7f800000u) atomicMin(&st->min_up[e], (long long)__uint_as_float(sh.smin_up[e]));
      if (sh.smin_dn[e] < 0x7f800000u) atomicMin(&st->min_dn[e], (long long)__uint_as_float(sh.smin_dn[e]));
    }
    if (!grid_barrier(st, epoch)) return;

    // ---- price step: one warp per expert, every input fetched in one round trip -------------------------
    for (int e = blockIdx.x + warp * gridDim.x; e < E; e += gridDim.x * (kSwThreads / 32)) {
      const int load_e = __ldcg(&st->load[e]);
      const int xs = load_e - (C - sh.trim[e]);
      long long ps = __ldcg(&st->p[e]);
      if (pending) { ps -= pend_anchor; if (ps < 0) ps = 0; }
      const int cup = __ldcg(&st->cap_up[e]), cdn = __ldcg(&st->cap_dn[e]);
      const long long mu = __ldcg(&st->min_up[e]), md = __ldcg(&st->min_dn[e]);
      const uint4* hu = reinterpret_cast<const uint4*>(hup + e * kNB) + 2 * lane;
      const uint4* hd = reinterpret_cast<const uint4*>(hdn + e * kNB) + 2 * lane;
      const uint4 hau = __ldcg(hu), hbu = __ldcg(hu + 1), had = __ldcg(hd), hbd = __ldcg(hd + 1);
      const bool up = xs > 0, dn = xs < 0 && (free_prices || ps > 0);
      long long p = ps; int flag = 0, imb = 0;
      if (up) {
        int cl = cup; bool shortw;
        p += price_step_warp(hau, hbu, xs, eps, cl, shortw, kCapLogMax, mu);
        if (lane == 0) st->cap_up[e] = cl;
        imb = xs;
      } else if (dn) {
        int cl = cdn; bool shortw;
        const long long cutby = price_step_warp(had, hbd, -xs, eps, cl, shortw, kCapLogMax, md);
        p -= cutby;
        if (!free_prices && p < 0) p = 0;
        if (lane == 0) st->cap_dn[e] = cl;
        // 2: nothing recorded at all and the price could not move.  When every expert has to end up full such an
        // expert must be heard sooner or later; when there is room to spare it may simply be one that stays short.
        flag = shortw ? ((cutby == 0 && a.balanced) ? 2 : 1) : 0;
        imb = -xs;
      }
      p = p > kPriceLimit ? kPriceLimit : (p < -kPriceLimit ? -kPriceLimit : p);
      // when nothing was out of balance the prices stay put and the pick reproduces this state
      if (xs == 0) p = ps;
      if (lane == 0) {
        st->flag_dn[e] = flag; st->load[e] = 0; st->min_up[e] = kInf; st->min_dn[e] = kInf;
        st->imb_e[e] = imb; st->drop_e[e] = ps - p > 0 ? ps - p : 0;
        st->p[e] = p;
        if (sweep == 0) st->load0[e] = load_e;
      }
    }
    pending = false;
    if (!grid_barrier(st, epoch)) return;

    // ---- every CTA draws the same conclusions from the same numbers ----------------------------------
    load_state();
    if (sweep == 0 && (a.slack > 0 || a.balanced)) {
      // The first sweep (every price zero) tells how lopsided the router is.  Free prices pay off when the loads are
      // roughly even: experts short of tokens then hear from enough tokens that rank them next to cut their price by
      // the right amount.  With most pairs on a few experts they hear from hardly anyone, cut blindly and overshoot,
      // and the prices swing ever wider; there the prices keep their floor at zero and only the crowded experts move.
      for (int e = tid; e < E; e += blockDim.x) sh.l0[e] = __ldcg(&st->load0[e]);
      if (tid == 0) sh.s_nb = 0;
      __syncthreads();
      for (int e = tid; e < E; e += blockDim.x) if (sh.l0[e] > C) atomicAdd(&sh.s_nb, sh.l0[e] - C);
      __syncthreads();
      const bool even = (long long)sh.s_nb * 8 <= (long long)T * a.k;
      __syncthreads();
      if (a.slack > 0 && even) {
        // who gives up room: raise a water level under the first sweep's loads until the room below it is the spare room
        for (int e = tid; e < E; e += blockDim.x) {
          int rank = 0;
          for (int x = 0; x < E; ++x) rank += (sh.l0[x] < sh.l0[e] || (sh.l0[x] == sh.l0[e] && x < e)) ? 1 : 0;
          sh.srt[rank] = sh.l0[e]; sh.trim[e] = rank;
        }
        __syncthreads();
        if (tid == 0) {
          long long rem = a.slack; int j = 1;               // the j least popular experts are below the level srt[j - 1]
          while (j < E) {
            const long long need = (long long)j * (sh.srt[j] - sh.srt[j - 1]);
            if (need > rem) break;
            rem -= need; ++j;
          }
          sh.s_nb = j; sh.s_level = sh.srt[j - 1] + (int)(rem / j); sh.s_rem = (int)(rem % j);
        }
        __syncthreads();
        for (int e = tid; e < E; e += blockDim.x) {
          const int rank = sh.trim[e];
          const int t = rank < sh.s_nb ? sh.s_level - sh.l0[e] + (rank < sh.s_rem ? 1 : 0) : 0;
          sh.trim[e] = t < C ? t : C;
        }
        hiding = true; free_prices = true;
        __syncthreads();
      } else if (a.balanced && !even) {
        pend_anchor = anchor_prices(); pending = true;      // lowest price to zero, and from here on none below it
        free_prices = false;
      }
    }
    ++sweep;
    // a small imbalance that has stopped shrinking is a price war between a few experts: the exact phase
    // ends it faster than more sweeps would
    // (progress = the imbalance fell below 7/8 of the best one seen so far: slower than that, an augmentation of the
    // exact phase costs about as much as the sweep and removes more)
    const bool progress = (long long)sh.s_imb * 8 < (long long)best_imb * 7 || best_imb == 0x7fffffff;
    stall = progress ? 0 : stall + 1;
    if (sh.s_imb < best_imb) best_imb = sh.s_imb;
    done = (sh.s_imb == 0) || sweep >= a.n_sweeps || (stall >= kStallSweeps && sh.s_imb <= kStallImbalance);
    if (done && hiding && sweep < a.n_sweeps) {
      // the problem without the spare room is as good as solved: put the experts that gave up room at price zero, hand
      // the room back and let the sweeps go on under the real rules (no price below zero, room allowed at price zero)
      pend_anchor = anchor_prices(); pending = true;
      for (int e = tid; e < kMaxE; e += blockDim.x) sh.trim[e] = 0;
      hiding = false; free_prices = a.balanced != 0;
      best_imb = 0x7fffffff; stall = 0; done = false;
      __syncthreads();
    }
    cumdrop += sh.s_drop;
#ifdef MAXSCORE_TRACE
    if (gtid == 0) printf("sweep %d imbalance %d stall %d eps %lld drop %lld\n", sweep, sh.s_imb, stall, eps, sh.s_drop);
#endif
    { const long long ne = eps >> 1; eps = ne < a.eps_min ? a.eps_min : ne; }
  }

  // ---- first pick: every token's top-k under the final prices, candidates listed ----------------------
  if (free_prices) anchor_prices();
  token_pass(std::true_type{}, nullptr, nullptr);
  for (int e = tid; e < E; e += blockDim.x)
    if (sh.sload[e]) atomicAdd(&st->load[e], sh.sload[e]);
  if (!grid_barrier(st, epoch)) return;
  if (blockIdx.x != 0) return;
  // ---- CTA 0: is the state already a certificate? -------------------------------------------------------
  __shared__ int s_badload;
  if (tid == 0) s_badload = 0;
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) {
    const int load = __ldcg(&st->load[e]);
    st->load_cur[e] = load; st->load[e] = 0;
    st->p[e] = sh.sp[e];
    // primal feasibility and complementary slackness on the expert -> sink arcs
    if (load > C || (sh.sp[e] > 0 && load < C)) atomicAdd(&s_badload, 1);
  }
  __syncthreads();
  if (tid == 0) {
    st->sweep = sweep; st->cumdrop = cumdrop;
    st->round = 1; st->theta_used = a.theta0; st->theta = a.theta0 * 4;
    st->converged = s_badload == 0 ? 1 : 0;
  }
}

// ---------------------------------------------------------------------------------------------
// Check pass.  Every token's experts must still be a top-k under the current prices (ties included).
// A token that fails re-picks (unless this is the last pass); tokens within theta of a tie are listed
// as the next round's candidates; loads, violations and the statistics are gathered on the way.  The last
// CTA decides: no violation and every expert within capacity with complementary slackness = optimal.
//   fast path  one thread per token, from the cache, when the cache's bound settles every question;
//   slow path  one warp per token over the full row, exact int64 throughout.
struct CheckShared {
  long long sp[kMaxE];
  int sload[kMaxE];
  int nslow, viol, rer;
  unsigned flags;
  double score;
  int slow[256];
};

__global__ void __launch_bounds__(256)
flow_check_kernel(const float* __restrict__ M, FlowState* st, SweepCache cache, int32_t* __restrict__ expert_idx,
                  int32_t* __restrict__ cand, int T, int E, int k, int C, KeyGen g, int final_pass, int unbounded,
                  int32_t* __restrict__ expert_load_out, void* stats_out, const unsigned* __restrict__ error_flag) {
  if (*(volatile int*)&st->done) return;
  __shared__ CheckShared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < E; e += blockDim.x) { sh.sp[e] = st->p[e]; sh.sload[e] = 0; }
  if (tid == 0) { sh.viol = 0; sh.rer = 0; sh.flags = 0; sh.score = 0.0; }
  __syncthreads();
  const long long cumdrop = st->cumdrop;
  const long long theta = final_pass ? -1 : (unbounded ? kInf : st->theta);      // the last pass lists nothing, the one before every token
  const int gsize = gridDim.x * blockDim.x;
  int t_viol = 0, t_rer = 0; double t_score = 0.0;
  for (int base = blockIdx.x * blockDim.x; base < T; base += gsize) {
    if (tid == 0) sh.nslow = 0;
    __syncthreads();
    const int tok = base + tid;
    if (tok < T) {
      bool slow = false;
      const uint4 idv = *reinterpret_cast<const uint4*>(cache.id + (size_t)tok * kCacheN);
      const unsigned idws[4] = {idv.x, idv.y, idv.z, idv.w};
      float x[kCacheN];
#pragma unroll
      for (int j = 0; j < kCacheN; ++j) x[j] = cache.x[(size_t)j * T + tok];
      const long long bound = cache.bound[tok];
      const bool raw = cache.raw[tok] != 0;
      const uint32_t flat = (uint32_t)tok * (uint32_t)E;
      unsigned hm[4] = {0, 0, 0, 0}; bool sorted = true; int prev = -1;
      for (int j = 0; j < k; ++j) {
        const int h = expert_idx[(size_t)tok * k + j];
        if ((unsigned)h >= (unsigned)E) { slow = true; break; }
        if (hm[h >> 5] & (1u << (h & 31))) { slow = true; break; }
        hm[h >> 5] |= 1u << (h & 31);
        sorted &= h > prev; prev = h;
      }
      long long key[kCacheN], v[kCacheN]; unsigned heldbits = 0;
      long long min_held = kInf, max_non = -kInf;
      if (!slow) {
#pragma unroll
        for (int j = 0; j < kCacheN; ++j) {
          const int e = (int)((idws[j >> 2] >> (8 * (j & 3))) & 255u);
          const bool ok = e < E;
          key[j] = ok ? make_key(g, x[j], flat + e) : -kInf;
          v[j] = ok ? key[j] - sh.sp[e] : -kInf;
          const bool held = ok && ((hm[e >> 5] >> (e & 31)) & 1u);
          if (held) { heldbits |= 1u << j; min_held = v[j] < min_held ? v[j] : min_held; }
          else if (ok) max_non = v[j] > max_non ? v[j] : max_non;
        }
        if (__popc(heldbits) != k) slow = true;           // an expert the token holds is not in its cache
      }
      const long long ob = bound <= -kInf ? -kInf : (bound >= kInf ? kInf : bound + cumdrop);   // uncached experts
      bool list = false;
      if (!slow) {
        if (min_held >= max_non && min_held >= ob) {
          const long long other = max_non > ob ? max_non : ob;
          list = E > k && other > -kInf && min_held - other <= theta;
        } else if (max_non > min_held) {
          // a cached expert beats a held one: a violation for certain.  Re-pick from the cache if it still
          // holds the token's k+1 best experts for certain.
          int rank[kCacheN];
#pragma unroll
          for (int j = 0; j < kCacheN; ++j) rank[j] = 0;
#pragma unroll
          for (int j = 1; j < kCacheN; ++j)
#pragma unroll
            for (int i = 0; i < j; ++i) {
              const bool first = v[i] >= v[j];
              rank[j] += first ? 1 : 0; rank[i] += first ? 0 : 1;
            }
          long long vk = -kInf, vk1 = -kInf;
#pragma unroll
          for (int j = 0; j < kCacheN; ++j) { if (rank[j] == k - 1) vk = v[j]; if (rank[j] == k) vk1 = v[j]; }
          if (final_pass) {
            ++t_viol;                                     // reported, not repaired
          } else if (vk1 >= ob && vk1 > -kInf) {
            ++t_viol;
            heldbits = 0; hm[0] = hm[1] = hm[2] = hm[3] = 0;
#pragma unroll
            for (int j = 0; j < kCacheN; ++j) {
              const int e = (int)((idws[j >> 2] >> (8 * (j & 3))) & 255u);
              if (rank[j] < k && e < E) { heldbits |= 1u << j; hm[e >> 5] |= 1u << (e & 31); }
            }
            sorted = false;
            list = vk - vk1 <= theta;
          } else {
            slow = true;
          }
        } else {
          slow = true;                                    // only the bound on the uncached experts is in the way
        }
      }
      // statistics: the score of the held pairs and how many of them are not among the token's k best raw keys.
      // A cache built at zero prices lists its entries by descending raw value, so its first k entries are the
      // raw top-k as soon as each of them beats every later entry and the bound on the uncached ones exactly;
      // otherwise (a near-tie, or a cache rebuilt at other prices) the held entries are counted one by one.
      if (!slow) {
        int rer = 0; double sc = 0.0;
        long long lo_first = kInf, hi_rest = -kInf;
#pragma unroll
        for (int j = 0; j < kCacheN; ++j) {
          if (j < k) lo_first = key[j] < lo_first ? key[j] : lo_first;
          else hi_rest = key[j] > hi_rest ? key[j] : hi_rest;
        }
        if (raw && lo_first > hi_rest && (bound <= -kInf || lo_first > bound)) {
          rer = __popc(heldbits >> k);                    // held entries listed after the raw top-k
        } else {
#pragma unroll
          for (int j = 0; j < kCacheN; ++j) {
            if (!((heldbits >> j) & 1u)) continue;
            int above = 0;
#pragma unroll
            for (int i = 0; i < kCacheN; ++i) above += key[i] > key[j] ? 1 : 0;
            if (above >= k) ++rer;
            else if (bound > -kInf && (!raw || key[j] <= bound)) slow = true;   // an uncached raw key might be larger
          }
        }
#pragma unroll
        for (int j = 0; j < kCacheN; ++j)
          if ((heldbits >> j) & 1u) sc += g.mode == 0 ? (double)x[j] : (double)key[j];
        if (!slow) { t_rer += rer; t_score += sc; }
      }
      if (!slow) {
        if (!sorted) write_sorted_experts(expert_idx + (size_t)tok * k, hm, k);
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          unsigned m = hm[w];
          while (m) { const int b = __ffs(m) - 1; m &= m - 1; atomicAdd(&sh.sload[32 * w + b], 1); }
        }
        if (list) cand[atomicAdd(&st->ncand, 1)] = tok;
      } else {
        sh.slow[atomicAdd(&sh.nslow, 1)] = tok;
      }
    }
    __syncthreads();
    // ---- slow path: one warp per token over the full row --------------------------------------------
    const int nslow = sh.nslow;
    for (int s = warp; s < nslow; s += 8) {
      const int t2 = sh.slow[s];
      const uint32_t flat = (uint32_t)t2 * (uint32_t)E;
      const float* row = M + (size_t)t2 * E;
      const int mine = lane < k ? expert_idx[(size_t)t2 * k + lane] : -1;
      long long key[kEPLf], val[kEPLf]; bool in[kEPLf]; float xr[kEPLf];
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        const int e = lane + 32 * q;
        xr[q] = e < E ? __ldg(row + e) : 0.f;
        key[q] = e < E ? make_key(g, xr[q], flat + e) : -kInf;
        val[q] = e < E ? key[q] - sh.sp[e] : -kInf;
        in[q] = false;
      }
      for (int j = 0; j < k; ++j) {
        const int ej = __shfl_sync(0xffffffffu, mine, j);
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) in[q] |= (ej == lane + 32 * q) && (ej < E);
      }
      int cnt = 0;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) cnt += __popc(__ballot_sync(0xffffffffu, in[q]));
      long long min_held = kInf, max_non = -kInf;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        if (lane + 32 * q >= E) continue;
        if (in[q]) min_held = val[q] < min_held ? val[q] : min_held;
        else max_non = val[q] > max_non ? val[q] : max_non;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const long long a = __shfl_xor_sync(0xffffffffu, min_held, o), c = __shfl_xor_sync(0xffffffffu, max_non, o);
        min_held = a < min_held ? a : min_held; max_non = c > max_non ? c : max_non;
      }
      const bool keep = cnt == k && min_held >= max_non;
      long long gap = keep ? ((E > k) ? min_held - max_non : kInf) : kInf;
      if (!keep) {
        if (lane == 0) ++t_viol;
        if (!final_pass) {
          long long vk = -kInf, vk1 = -kInf;
          warp_select(val, E, k + 1, in, vk, vk1, k);
          gap = (E > k) ? vk - vk1 : kInf;
        }
      }
      // the experts in ascending order: word q of the held mask is the vote over in[q]
      unsigned words[kEPLf]; int below = 0;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) words[q] = __ballot_sync(0xffffffffu, in[q]);
      if (keep || !final_pass) {
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) {
          if (in[q]) {
            const int rank = below + __popc(words[q] & ((1u << lane) - 1u));
            if (rank < k) expert_idx[(size_t)t2 * k + rank] = lane + 32 * q;
          }
          below += __popc(words[q]);
        }
      }
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) if (in[q]) atomicAdd(&sh.sload[lane + 32 * q], 1);
      {
        bool rsel[kEPLf]; long long kth_raw = -kInf, next_raw = -kInf;
        warp_select(key, E, k, rsel, kth_raw, next_raw, k);
        int rer = 0; double sc = 0.0;
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) {
          rer += (in[q] && key[q] < kth_raw) ? 1 : 0;
          if (in[q]) sc += g.mode == 0 ? (double)xr[q] : (double)key[q];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { sc += __shfl_xor_sync(0xffffffffu, sc, o); rer += __shfl_xor_sync(0xffffffffu, rer, o); }
        if (lane == 0) { t_rer += rer; t_score += sc; }
      }
      if (gap < kInf && gap <= theta && lane == 0) cand[atomicAdd(&st->ncand, 1)] = t2;
    }
    __syncthreads();
  }
  if (t_viol) atomicAdd(&sh.viol, t_viol);
  if (t_rer) atomicAdd(&sh.rer, t_rer);
  if (t_score != 0.0) atomicAdd(&sh.score, t_score);
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x)
    if (sh.sload[e]) atomicAdd(&st->load[e], sh.sload[e]);
  if (tid == 0) {
    if (sh.viol) atomicAdd(&st->violations, sh.viol);
    if (sh.rer) atomicAdd(&st->rerouted, sh.rer);
    if (sh.score != 0.0) atomicAdd(&st->total_score, sh.score);
  }
  if (!last_block_arrives(&st->ticket)) return;
  // ---- last CTA: is the state a certificate? ---------------------------------------------------
  __shared__ int s_badload;
  if (tid == 0) s_badload = 0;
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) {
    const int load = __ldcg(&st->load[e]);
    st->load_cur[e] = load;
    st->load[e] = 0;
    if (expert_load_out) expert_load_out[e] = load;
    // primal feasibility and complementary slackness on the expert -> sink arcs
    if (load > C || (sh.sp[e] > 0 && load < C)) atomicAdd(&s_badload, 1);
  }
  __syncthreads();
  if (tid == 0) {
    const int viol = *(volatile int*)&st->violations;
    const bool ok = viol == 0 && s_badload == 0;
#ifdef MAXSCORE_TRACE
    printf("check round %d: violations %d experts off %d listed %d theta %lld\n", st->round, viol, s_badload, st->ncand, theta);
#endif
    st->violations = 0;
    st->ticket = 0;
    if (ok || final_pass) {
      unsigned status = *(volatile unsigned*)&st->status;
      if (!ok) status |= 1u;
      if (error_flag && *error_flag) status |= 4u;
      // layout of maxscore_stats: status, capacity, sweeps, augmentations, rounds, candidates,
      // rerouted, reserved, total_score
      int* so = reinterpret_cast<int*>(stats_out);
      so[0] = (int)(status & 7u);
      so[1] = C; so[2] = st->sweep; so[3] = st->naug; so[4] = st->round;
      so[5] = st->ncand_last; so[6] = *(volatile int*)&st->rerouted; so[7] = 0;
      *reinterpret_cast<double*>(so + 8) = *(volatile double*)&st->total_score;
      st->converged = 1;
      __threadfence();
      st->done = 1;
    } else {
      // the next round looks further: its candidates were listed with this pass's theta
      const long long th = theta;
      st->round = st->round + 1;
      st->theta_used = th;
      st->theta = (th > (kInf >> 8)) ? kInf : th * 4;
      st->rerouted = 0; st->total_score = 0.0;
      st->converged = 0;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Exact phase: successive shortest augmenting paths on the expert-level residual graph of Table 1's
// network (E experts + one node Z for the sink side).
//
// Only candidate tokens (gap <= theta) are in the graph.  A round stops BEFORE an augmentation whose
// price update would spread the experts' price changes of this round by more than theta: up to that
// point no token outside the list can have lost its top-k, so the state handed to the next check
// pass is consistent, and that pass only has to list more tokens.
//
// The graph is never materialised as an E x E matrix.  Each candidate carries a short record: the
// experts it holds that could be given up within the arc window, and the experts it does not hold
// that could be taken within it, each with value0 = key - price at the start of the round.  A token
// that holds e and not f is a residual arc e -> f of reduced cost value(e) - value(f) >= 0, where
// value = value0 - (price now - price at round start).  One round of the Bellman-Ford search is then
// one pass over the records: A = min over held entries of dist[e] + value(e), and every entry f not
// held is offered A - value(f).  Moving a token flips two flags of its record; nothing is rebuilt.
constexpr int kP2Group = 4;                // threads that share one node of the graph in a search round
constexpr int kP2Threads = kP2Group * kMaxE + 32;   // a group per expert node and one warp for node Z
constexpr int kP2Own = 8;                  // candidates per thread whose experts and flags stay packed in registers during a search
constexpr int kRecSmemBytes = 96 * 1024;   // records up to this size are mirrored in shared memory
constexpr long long kDistLimit = 1LL << 58;  // distances stay below this, so that sums cannot overflow
constexpr long long kExactCycleBudget = 4000000000LL;   // about two seconds: the exact phase gives up beyond this

struct Records {
  long long* val;          // [cap] value0 of each entry
  unsigned short* meta;    // [cap] expert index | held << 8
  int* off;                // [T] first entry of candidate c
  int* cnt;                // [T] number of its entries
  // scratch of the exact phase when the records do not fit in shared memory
  int* pos;                // [cap] position of the entry in the by-expert order
  int* bxc;                // [cap] by-expert order: position in the candidate list of the entry's token
  long long* ndv;          // [cap] by-expert order: the offer the entry makes to its expert in this search round
  int* aarg;               // [T] the held expert through which the candidate is reached most cheaply
  int cap;
};

// Records of one round, built by the whole GPU: one warp per candidate token reads the token's row once.
__global__ void __launch_bounds__(256)
flow_records_kernel(const float* __restrict__ M, FlowState* st, const int32_t* __restrict__ expert_idx,
                    const int32_t* __restrict__ cand, Records rec, int T, int E, int k, KeyGen g) {
  if (*(volatile const int*)&st->converged) return;
  __shared__ long long sp[kMaxE];
  for (int e = threadIdx.x; e < E; e += blockDim.x) sp[e] = st->p[e];
  __syncthreads();
  const int n = min(st->ncand, T);
  const long long theta = st->theta_used;
  const long long arc_window = theta >= (kInf >> 2) ? kInf : 2 * theta;
  const int lane = threadIdx.x & 31;
  const int nwarps = gridDim.x * (blockDim.x >> 5);
  for (int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); c < n; c += nwarps) {
    const int tok = cand[c];
    int h[kMaxK];
#pragma unroll
    for (int j = 0; j < kMaxK; ++j) h[j] = j < k ? expert_idx[(size_t)tok * k + j] : -1;
    const float* row = M + (size_t)tok * E;
    const uint32_t flat = (uint32_t)tok * (uint32_t)E;
    long long val[kEPLf]; bool in[kEPLf];
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      const int f = lane + 32 * q;
      val[q] = f < E ? make_key(g, __ldg(row + f), flat + f) - sp[f] : -kInf;
      bool hd = false;
#pragma unroll
      for (int j = 0; j < kMaxK; ++j) hd |= (h[j] == f);
      in[q] = hd;
    }
    long long best_out = -kInf;                         // best value among the experts the token does not hold
#pragma unroll
    for (int q = 0; q < kEPLf; ++q)
      if (!in[q] && lane + 32 * q < E) best_out = val[q] > best_out ? val[q] : best_out;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const long long ov = __shfl_xor_sync(0xffffffffu, best_out, o);
      best_out = ov > best_out ? ov : best_out;
    }
    // a held expert further than the arc window above every alternative cannot be given up this round
    bool inc[kEPLf];
    long long low_held = kInf;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      inc[q] = in[q] && best_out > -kInf && (arc_window >= kInf || val[q] - best_out <= arc_window);
      if (inc[q]) low_held = val[q] < low_held ? val[q] : low_held;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const long long ov = __shfl_xor_sync(0xffffffffu, low_held, o);
      low_held = ov < low_held ? ov : low_held;
    }
    // an expert not held further than the window below every held one that can move cannot be taken
#pragma unroll
    for (int q = 0; q < kEPLf; ++q)
      if (!in[q]) inc[q] = lane + 32 * q < E && low_held < kInf && (arc_window >= kInf || low_held - val[q] <= arc_window);
    unsigned words[kEPLf]; int total = 0;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) { words[q] = __ballot_sync(0xffffffffu, inc[q]); total += __popc(words[q]); }
    int base = 0;
    if (lane == 0) {
      base = atomicAdd(&st->nrec, total);
      if (base + total > rec.cap) { base = -1; st->rec_overflow = 1; }     // no room: the token stays out of the graph
      rec.off[c] = base < 0 ? 0 : base;
      rec.cnt[c] = base < 0 ? 0 : total;
    }
    base = __shfl_sync(0xffffffffu, base, 0);
    if (base < 0) continue;
    int before = 0;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      if (inc[q]) {
        const int pos = base + before + __popc(words[q] & ((1u << lane) - 1u));
        rec.val[pos] = val[q];
        rec.meta[pos] = (unsigned short)((lane + 32 * q) | (in[q] ? 256 : 0));
      }
      before += __popc(words[q]);
    }
  }
}

constexpr int kRecUnroll = 6;      // records up to this many entries are handled with all loads in flight

struct P2Shared {
  long long p[kMaxE + 1];        // potentials: prices of the experts, then Z
  long long dp[kMaxE + 1];       // potentials now minus potentials at the start of the round
  long long p0[kMaxE + 1];
  long long dist[2][kMaxE + 1];  // distances as of the last search round / of the running one
  int lvl[kMaxE + 1];            // search round in which the node's distance became final
  int imb[kMaxE + 1];            // + excess, - deficit
  int flow[kMaxE];               // units on expert -> sink
  int estart[kMaxE + 2], efill[kMaxE + 1];   // entries grouped by expert: first position, fill counter
  int path_v[kMaxE + 2], path_u[kMaxE + 2], path_tok[kMaxE + 2], path_c[kMaxE + 2];
  unsigned char failed[kMaxE + 4];   // deficit nodes whose walk came to a dead end in this search
  unsigned char front[2][kMaxE + 4]; // nodes whose distance changed in the last search round / in the running one
  unsigned char dirty[kMaxE + 4];    // nodes that were made a new offer in the running round
  int nact;                          // candidates listed for the running round
  int act[kP2Own * kP2Threads];      // their positions in the candidate list
  int npath, target, stop;
  long long dt, dtb;             // distance of the chosen target; best distance of any node with a deficit so far
};

// kSmem = true: the records are mirrored in shared memory (the kernel returns at once if they do not fit);
// kSmem = false: they stay in global memory (the kernel returns at once if they would have fitted).  The
// host launches both, one after the other; exactly one of them does the work.
template <bool kSmem>
__global__ void __launch_bounds__(kP2Threads)
flow_exact_kernel(FlowState* st, int32_t* expert_idx, const int32_t* __restrict__ cand, Records rec, int T, int E,
                  int k, int C, int max_aug) {
  if (*(volatile int*)&st->done) return;
  if (*(volatile int*)&st->converged) {             // nothing to repair; the check pass starts a fresh list
    if (threadIdx.x == 0) { st->ncand = 0; st->nrec = 0; }
    return;
  }
  extern __shared__ __align__(16) unsigned char p2smem[];
  __shared__ P2Shared s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = min(st->ncand, T);
  const int nent = min(st->nrec, rec.cap);
  const int nZ = E;
  const long long theta = st->theta_used;
  const long long t_start = clock64();

  if ((((size_t)nent * 26 + (size_t)n * 16 + 64) <= (size_t)kRecSmemBytes) != kSmem) return;
  // ---- mirror the records in shared memory when they fit ------------------------------------------
  long long* v_s = reinterpret_cast<long long*>(p2smem);
  long long* nd_s = v_s + nent;
  int* off_s = reinterpret_cast<int*>(nd_s + nent);
  int* cnt_s = off_s + n;
  int* tok_s = cnt_s + n;
  int* aarg_s = tok_s + n;
  int* pos_s = aarg_s + n;
  int* bxc_s = pos_s + nent;
  unsigned short* m_s = reinterpret_cast<unsigned short*>(bxc_s + nent);
  if (kSmem) {
    for (int i = tid; i < nent; i += blockDim.x) { v_s[i] = rec.val[i]; m_s[i] = rec.meta[i]; }
    for (int i = tid; i < n; i += blockDim.x) { off_s[i] = rec.off[i]; cnt_s[i] = rec.cnt[i]; tok_s[i] = cand[i]; }
  }
  const long long* rval = kSmem ? v_s : rec.val; unsigned short* rmeta = kSmem ? m_s : rec.meta;
  const int* roff = kSmem ? off_s : rec.off; const int* rcnt = kSmem ? cnt_s : rec.cnt; const int* rtok = kSmem ? tok_s : cand;
  int* rpos = kSmem ? pos_s : rec.pos; int* bxc = kSmem ? bxc_s : rec.bxc; long long* ndv = kSmem ? nd_s : rec.ndv;
  int* aarg = kSmem ? aarg_s : rec.aarg;
  for (int e = tid; e <= E + 1; e += blockDim.x) { s.estart[e] = 0; if (e <= E) s.efill[e] = 0; }
  for (int e = tid; e < E; e += blockDim.x) {
    s.p[e] = st->p[e]; s.p0[e] = s.p[e]; s.dp[e] = 0;
    const int load = st->load_cur[e];
    const int fl = s.p[e] > 0 ? C : min(load, C);
    s.flow[e] = fl; s.imb[e] = load - fl;
  }
  __syncthreads();
  // ---- the entries grouped by expert (counting sort over the candidates' records) ---------------------
  for (int c = tid; c < n; c += blockDim.x) {
    const int o = roff[c], m = rcnt[c];
    for (int i = o; i < o + m; ++i) atomicAdd(&s.estart[(rmeta[i] & 255) + 1], 1);
  }
  __syncthreads();
  if (tid == 0) {
    int tot = 0;
    for (int e = 0; e < E; ++e) tot += s.imb[e];
    s.imb[nZ] = -tot; s.p[nZ] = 0; s.p0[nZ] = 0; s.dp[nZ] = 0; s.stop = 0;
    for (int e = 0; e <= E; ++e) s.estart[e + 1] += s.estart[e];
  }
  __syncthreads();
  for (int c = tid; c < n; c += blockDim.x) {
    const int o = roff[c], m = rcnt[c];
    for (int i = o; i < o + m; ++i) {
      const int e = rmeta[i] & 255;
      const int ps = s.estart[e] + atomicAdd(&s.efill[e], 1);
      rpos[i] = ps; bxc[ps] = c;
    }
  }
  __syncthreads();

  int naug = 0;
  const int naug_before = st->naug;
  long long* d0 = s.dist[0]; long long* dn = s.dist[1];
  for (;;) {
    {
      if (tid == 0 && clock64() - t_start > kExactCycleBudget) s.stop = 1;
      const int any = __syncthreads_or(tid <= E && s.imb[tid] > 0);
      if (s.stop) { if (tid == 0) atomicOr(&st->status, 4u); break; }
      if (!any || naug_before + naug >= max_aug) break;
    }
    // ---- shortest paths from every node with excess: synchronous Bellman-Ford, frontier by frontier ------
    // A candidate's offers only change when the distance of an expert it holds has changed, so a round
    //   (0) lists the candidates that hold an expert of the frontier (the nodes whose distance changed in the
    //       round before; at first the nodes with excess): one thread per candidate, from a packed copy of the
    //       record's experts and flags that stays in registers;
    //   (A) one thread per LISTED candidate: A = the cheapest way to reach the token through an expert it holds;
    //       every entry it does not hold is offered A - value, written where the entry sits in the by-expert
    //       order, and that expert is marked dirty;
    //   (B) a group of threads per dirty node (and per node with a Z arc when Z moved): the best offer over the
    //       node's stretch of the by-expert order, and the arcs through Z.
    // Offers of candidates that were not listed are still those of their last evaluation, which used the same
    // distances.  No atomics on distances, and distances only ever come from the previous round's, so the round
    // in which a node's distance became final orders the nodes.  Offers that cannot beat the nearest node with a
    // deficit found so far (plus theta) are dropped: all costs are non-negative, and beyond that distance the
    // price update only needs to know "at least that far".
    for (int v = tid; v <= E; v += blockDim.x) {
      d0[v] = s.imb[v] > 0 ? 0 : kInf; s.lvl[v] = 0; s.dirty[v] = 0;
      s.front[0][v] = s.imb[v] > 0 ? 1 : 0; s.front[1][v] = 0;
    }
    for (int i = tid; i < nent; i += blockDim.x) ndv[i] = kInf;        // no offers yet in this search
    if (tid == 0) { s.dtb = kDistLimit; s.nact = 0; }
    // packed copies of this thread's candidates: bytes 0..5 the experts of up to six entries, byte 6 their held
    // flags, byte 7 the entry count (0xff: a record too long to pack, always evaluated)
    unsigned long long own[kP2Own];
#pragma unroll
    for (int r = 0; r < kP2Own; ++r) {
      const int c = tid + r * kP2Threads;
      unsigned long long pk = 0;
      if (c < n) {
        const int o = roff[c], m = rcnt[c];
        if (m > kRecUnroll) pk = 0xffULL << 56;
        else {
          unsigned hb = 0;
          for (int j = 0; j < m; ++j) {
            const int mt = rmeta[o + j];
            pk |= (unsigned long long)(mt & 255) << (8 * j);
            if (mt & 256) hb |= 1u << j;
          }
          pk |= (unsigned long long)hb << 48 | (unsigned long long)m << 56;
        }
      }
      own[r] = pk;
    }
    __syncthreads();
    int more = 1, cur = 0;
    for (int round = 1; round <= E + 2 && more; ++round) {
      const unsigned char* fr = s.front[cur];
      // (0) list the candidates touched by the frontier
#pragma unroll
      for (int r = 0; r < kP2Own; ++r) {
        const unsigned long long pk = own[r];
        const int m = (int)(pk >> 56);
        if (__all_sync(0xffffffffu, m == 0)) continue;               // nobody in the warp owns a candidate in this slot
        bool hit = m == 0xff;
        const unsigned hb = (unsigned)(pk >> 48) & 0xffu;
#pragma unroll
        for (int j = 0; j < kRecUnroll; ++j)
          if (j < m && ((hb >> j) & 1u)) hit |= fr[(pk >> (8 * j)) & 255u] != 0;
        const unsigned hits = __ballot_sync(0xffffffffu, hit);        // one shared-memory atomic per warp, not per hit
        if (hits) {
          int base = 0;
          if (lane == 0) base = atomicAdd(&s.nact, __popc(hits));
          base = __shfl_sync(0xffffffffu, base, 0);
          if (hit) s.act[base + __popc(hits & ((1u << lane) - 1u))] = tid + r * kP2Threads;
        }
      }
      __syncthreads();
      // (A) offers of the listed candidates
      const int nact = s.nact;
      // (candidates beyond the packed copies are evaluated every round)
      for (int ai = tid; ai < nact + max(0, n - kP2Own * kP2Threads); ai += blockDim.x) {
        const int c = ai < nact ? s.act[ai] : kP2Own * kP2Threads + (ai - nact);
        const int o = roff[c], m = rcnt[c];
        long long A = kInf; int ae = 0;
        if (m <= kRecUnroll) {
          long long vc[kRecUnroll], x[kRecUnroll]; int ex[kRecUnroll], ps[kRecUnroll]; bool held[kRecUnroll];
#pragma unroll
          for (int j = 0; j < kRecUnroll; ++j) {
            const int i = j < m ? o + j : o;
            const int mt = rmeta[i];
            ex[j] = mt & 255; held[j] = (mt & 256) != 0; ps[j] = rpos[i];
            const long long dv = d0[ex[j]];
            vc[j] = rval[i] - s.dp[ex[j]];
            x[j] = (j < m && held[j] && dv < kInf) ? dv + vc[j] : kInf;
          }
#pragma unroll
          for (int j = 0; j < kRecUnroll; ++j)
            if (x[j] < A || (x[j] == A && x[j] < kInf && ex[j] < ae)) { A = x[j]; ae = ex[j]; }
#pragma unroll
          for (int j = 0; j < kRecUnroll; ++j)
            if (j < m && !held[j]) { ndv[ps[j]] = A < kInf ? A - vc[j] : kInf; s.dirty[ex[j]] = 1; }
        } else {
          for (int i = o; i < o + m; ++i) {
            const int mt = rmeta[i];
            if (!(mt & 256)) continue;
            const int e = mt & 255;
            const long long du = d0[e];
            if (du >= kInf) continue;
            const long long x = du + (rval[i] - s.dp[e]);
            if (x < A || (x == A && e < ae)) { A = x; ae = e; }
          }
          for (int i = o; i < o + m; ++i) {
            const int mt = rmeta[i];
            if (mt & 256) continue;
            ndv[rpos[i]] = A < kInf ? A - (rval[i] - s.dp[mt & 255]) : kInf; s.dirty[mt & 255] = 1;
          }
        }
        aarg[c] = ae;
      }
      __syncthreads();
      // (B) nodes
      bool changed = false;
      // beyond the nearest deficit's distance plus theta no target can be used: its price update would leave the window
      const long long dtb = (theta < kInf && s.dtb < kDistLimit - theta) ? s.dtb + theta + 1 : kDistLimit;
      unsigned char* fn = s.front[cur ^ 1];
      const bool zmoved = fr[nZ] != 0;
      {
        const int f = tid / kP2Group, sub = tid % kP2Group;      // every thread takes part in the group shuffles
        long long best = kInf;
        const bool work = f < E && (s.dirty[f] || (zmoved && s.flow[f] > 0));
        if (work) {
          const int hi = s.estart[f + 1];
          for (int idx = s.estart[f] + sub; idx < hi; idx += 4 * kP2Group) {
            long long a[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) a[u] = idx + u * kP2Group < hi ? ndv[idx + u * kP2Group] : kInf;
#pragma unroll
            for (int u = 0; u < 4; ++u) best = a[u] < best ? a[u] : best;
          }
          if (sub == 0) {                                 // one unit less on f -> sink
            const long long dz = d0[nZ];
            if (dz < kInf && s.flow[f] > 0) {
              long long rc = -s.p[nZ] + s.p[f]; if (rc < 0) rc = 0;
              best = dz + rc < best ? dz + rc : best;
            }
          }
        }
#pragma unroll
        for (int o = kP2Group / 2; o > 0; o >>= 1) {
          const long long ob = __shfl_xor_sync(0xffffffffu, best, o);
          best = ob < best ? ob : best;
        }
        if (f < E && sub == 0) {
          const long long old = d0[f];
          const bool better = work && best < old && best < dtb;
          dn[f] = better ? best : old;
          fn[f] = better ? 1 : 0;
          s.dirty[f] = 0;
          if (better) {
            s.lvl[f] = round; changed = true;
            if (s.imb[f] < 0) atomicMin(&s.dtb, best);
          }
        }
      }
      if (warp == kP2Threads / 32 - 1) {                  // node Z: one more unit on e -> sink, for any expert with room
        long long off[kEPLf];
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) {
          const int e = lane + 32 * q;
          off[q] = kInf;
          if (e < E) {
            const long long de = d0[e]; const int fl = s.flow[e];
            long long rc = -s.p[e] + s.p[nZ]; if (rc < 0) rc = 0;
            if (de < kInf && fl < C) off[q] = de + rc;
          }
        }
        long long best = kInf;
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) best = off[q] < best ? off[q] : best;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const long long ob = __shfl_xor_sync(0xffffffffu, best, o);
          best = ob < best ? ob : best;
        }
        if (lane == 0) {
          const long long old = d0[nZ];
          const bool better = best < old && best < dtb;
          dn[nZ] = better ? best : old;
          fn[nZ] = better ? 1 : 0;
          if (better) {
            s.lvl[nZ] = round; changed = true;
            if (s.imb[nZ] < 0) atomicMin(&s.dtb, best);
          }
          s.nact = 0;
        }
      }
      more = __syncthreads_or(changed);
      { long long* t = d0; d0 = dn; dn = t; }
      cur ^= 1;
    }
    // ---- augment along tight arcs, nearest deficit first, by one warp ------------------------------------
    // With potentials lowered by min(dist, D), every arc u -> v with dist[u] + cost == dist[v] <= D has reduced
    // cost zero, and so has its reverse: pushing a unit along ANY path of such arcs keeps all reduced costs
    // non-negative.  One search therefore serves several augmentations: the deficit nodes are taken in order
    // of distance (lowest index on ties) as long as the price update for D = their distance stays within theta.
    // The walk back from a target: an arc u -> v is eligible when it is tight and u's distance was final before
    // v's; such an arc exists for every reached node, and following them strictly lowers the level, so the walk
    // ends at a node that had excess when the search began without repeating a node.  Among the eligible arcs
    // the Z arc wins, then the smallest token index, then the smallest tail: the choice does not depend on the
    // order of the candidate list.  The offers of the last search round (which changed nothing) are still in
    // place: an entry whose offer equals its node's distance is a tight arc from the expert its candidate is
    // reached through.  A token that has moved takes its offers off the table for the rest of this search.
    if (warp == 0) {
      int napplied = 0, result = -1; long long dmax = 0;
      for (int v = lane; v <= E; v += 32) s.failed[v] = 0;
      __syncwarp();
      const bool trusted = more == 0;                    // a search that never settled is not used
      for (int attempt = 0; trusted && attempt < 4 * kMaxE; ++attempt) {
        long long dt = kInf; int t = 0x7fffffff;
        for (int v = lane; v <= E; v += 32)
          if (s.imb[v] < 0 && !s.failed[v] && d0[v] < dt) { dt = d0[v]; t = v; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const long long od = __shfl_xor_sync(0xffffffffu, dt, o);
          const int ot = __shfl_xor_sync(0xffffffffu, t, o);
          if (od < dt || (od == dt && ot < t)) { dt = od; t = ot; }
        }
        if (dt >= kInf) break;                           // no reachable deficit is left
        {
          long long lo = kInf, hi = -kInf;
          for (int e = lane; e < E; e += 32) {
            const long long d = d0[e];
            const long long chg = s.dp[e] - (d < dt ? d : dt);
            lo = chg < lo ? chg : lo; hi = chg > hi ? chg : hi;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const long long ol = __shfl_xor_sync(0xffffffffu, lo, o), oh = __shfl_xor_sync(0xffffffffu, hi, o);
            lo = ol < lo ? ol : lo; hi = oh > hi ? oh : hi;
          }
          if (theta < kInf && hi - lo > theta) {
            if (napplied == 0) {
              result = -2;                                // stop here; the next round lists more tokens:
              if (lane == 0 && st->theta < 2 * (hi - lo)) st->theta = 2 * (hi - lo);   // enough of them for this price update
            }
            break;
          }
        }
        // ---- walk back from t ----
        int len = 0, v = t; bool dead = false;
        while (s.lvl[v] > 0 && len <= E + 1) {
          unsigned long long code = ~0ULL; int cc = -1;
          const long long dv = d0[v]; const int lv = s.lvl[v];
          if (v == nZ) {
            for (int e = lane; e < E; e += 32) {
              const long long de = d0[e];
              if (de < kInf && s.flow[e] < C && s.lvl[e] < lv) {
                long long rc = -s.p[e] + s.p[nZ]; if (rc < 0) rc = 0;
                if (de + rc == dv && (unsigned long long)e < code) code = (unsigned long long)e;
              }
            }
          } else {
            const long long dz = d0[nZ];
            bool zarc = false;
            if (dz < kInf && s.flow[v] > 0 && s.lvl[nZ] < lv) {
              long long rc = -s.p[nZ] + s.p[v]; if (rc < 0) rc = 0;
              zarc = dz + rc == dv;
            }
            if (zarc) {
              code = (unsigned long long)nZ;
            } else {
              for (int idx = s.estart[v] + lane; idx < s.estart[v + 1]; idx += 32) {
                if (ndv[idx] != dv) continue;
                const int c = bxc[idx];
                const unsigned long long tk = ((unsigned long long)(unsigned)rtok[c] + 1ULL) << 8;
                const int e1 = aarg[c];
                if (s.lvl[e1] < lv) {
                  if ((tk | (unsigned long long)e1) < code) { code = tk | (unsigned long long)e1; cc = c; }
                  continue;
                }
                // the offer came through A = min over the candidate's held experts; any of them that attains A
                // gives a tight arc as well
                const int o = roff[c], m = rcnt[c];
                long long Ac = kInf;
                for (int j = o; j < o + m; ++j) {
                  const int mj = rmeta[j];
                  if (!(mj & 256)) continue;
                  const long long de = d0[mj & 255];
                  if (de >= kInf) continue;
                  const long long x = de + (rval[j] - s.dp[mj & 255]);
                  Ac = x < Ac ? x : Ac;
                }
                for (int j = o; j < o + m; ++j) {
                  const int mj = rmeta[j];
                  if (!(mj & 256)) continue;
                  const int e = mj & 255;
                  const long long de = d0[e];
                  if (de >= kInf || s.lvl[e] >= lv) continue;
                  if (de + (rval[j] - s.dp[e]) == Ac && (tk | (unsigned long long)e) < code) { code = tk | (unsigned long long)e; cc = c; }
                }
              }
            }
          }
          {   // smallest code of the warp: its high word (token + 1), then its low byte (the tail) among the lanes that match
            const unsigned hi = __reduce_min_sync(0xffffffffu, (unsigned)(code >> 8));
            const unsigned lo = __reduce_min_sync(0xffffffffu, (unsigned)(code >> 8) == hi ? (unsigned)(code & 255ULL) : 0xffffffffu);
            const unsigned who = __ballot_sync(0xffffffffu, (unsigned)(code >> 8) == hi && (unsigned)(code & 255ULL) == lo);
            const bool none = hi == 0xffffffffu;
            cc = __shfl_sync(0xffffffffu, cc, none ? 0 : __ffs(who) - 1);
            code = none ? ~0ULL : (((unsigned long long)hi << 8) | lo);
          }
          if (code == ~0ULL) { dead = true; break; }      // every tight arc into v was used up earlier in this search
          const int u = (int)(code & 255ULL);
          if (lane == 0) { s.path_v[len] = v; s.path_u[len] = u; s.path_tok[len] = (int)(code >> 8) - 1; s.path_c[len] = cc; }
          ++len; v = u;
        }
        if (!dead && (s.lvl[v] > 0 || s.imb[v] <= 0)) dead = true;      // the walk must end at a node that still has excess
        if (dead) {
          if (napplied == 0 && attempt == 0 && s.lvl[v] > 0 && len > E + 1) { result = -3; break; }   // cannot happen
          if (lane == 0) s.failed[t] = 1;
          __syncwarp();
          continue;
        }
        // ---- move one unit along the path ----
        __syncwarp();
        for (int a = lane; a < len; a += 32) {
          const int pu = s.path_u[a], pv = s.path_v[a], tok = s.path_tok[a];
          if (tok >= 0) {
            const int c = s.path_c[a];
            const int o = roff[c], m = rcnt[c];
            for (int i = o; i < o + m; ++i) {
              const int e = rmeta[i] & 255;
              if (e == pu) rmeta[i] = (unsigned short)pu;             // given up
              if (e == pv) rmeta[i] = (unsigned short)(pv | 256);     // taken
              ndv[rpos[i]] = kInf;
            }
            int rowv[kMaxK];                                   // all loads in flight before the one store
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) rowv[j] = j < k ? expert_idx[(size_t)tok * k + j] : -1;
#pragma unroll
            for (int j = 0; j < kMaxK; ++j)
              if (j < k && rowv[j] == pu) expert_idx[(size_t)tok * k + j] = pv;
          } else if (pv == nZ) {
            atomicAdd(&s.flow[pu], 1);
          } else {
            atomicAdd(&s.flow[pv], -1);
          }
        }
        if (lane == 0) { s.imb[v] -= 1; s.imb[t] += 1; }
        __syncwarp();
        ++napplied; dmax = dt;
      }
      if (lane == 0) { s.target = napplied > 0 ? napplied : result; s.dt = dmax; if (!trusted || result == -3) s.stop = 1; }
    }
    __syncthreads();
    if (s.stop) { if (tid == 0) atomicOr(&st->status, 4u); break; }
    if (s.target < 0) break;        // -1: no augmenting path inside the candidate graph; -2: theta reached
    {
      const long long dt = s.dt;
      for (int v = tid; v <= E; v += blockDim.x) {
        const long long d = d0[v];
        const long long step = d < dt ? d : dt;
        s.p[v] -= step; s.dp[v] -= step;
      }
    }
    naug += s.target;
    __syncthreads();
  }
  // ---- write back ---------------------------------------------------------------------------------
  __syncthreads();
#ifdef MAXSCORE_TRACE
  if (tid == 0) {
    int ex = 0, de = 0;
    for (int e = 0; e < E; ++e) { if (s.imb[e] > 0) ex += s.imb[e]; if (s.imb[e] < 0) de -= s.imb[e]; }
    printf("exact round %d: cand %d entries %d aug %d last %d excess %d deficit %d z %d theta %lld\n", st->round, n, nent, naug,
           s.target, ex, de, s.imb[nZ], theta);
  }
#endif
  if (tid == 0) s.dt = 0;
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) {
    long long pe = s.p[e] - s.p[nZ];
    pe = pe < 0 ? 0 : pe;           // only an expert that holds nothing can come out negative
    st->p[e] = pe;
    if (s.p0[e] - pe > 0) atomicMax(&s.dt, s.p0[e] - pe);
  }
  __syncthreads();
  // the caches' bounds on uncached experts must keep up with prices that fell during this round
  if (tid == 0) {
    st->cumdrop += s.dt; st->naug += naug; st->ncand_last = n; st->ncand = 0; st->nrec = 0;
    // Excess left and no path to a deficit among the listed tokens at all: the list is far too short (a price spread
    // that stopped the round tells how far to look; this tells nothing), so the next listing looks four times further
    // than it would have.
    if (s.target == -1 && theta < (kInf >> 8)) {
      bool left = false;
      for (int e = 0; e <= E; ++e) left |= s.imb[e] > 0;
      const long long th = st->theta;
      if (left && th < (kInf >> 8)) st->theta = th * 4;
    }
  }
}

}  // namespace msr
