// Token -> expert assignment: the min-cost max-flow of Eq. 7-8 on the network of Table 1, solved
// exactly on the GPU.
//
// Structure used.  The dual of the flow problem has one price p_e >= 0 per expert; given prices every
// token independently holds its k largest values of key(i, e) - p_e.  The solver therefore works on
// the E prices, never on the T x E arcs:
//
//   sweeps    (data parallel, one thread per token)  every token re-picks its top-k under the
//             current prices; per expert a load count, two histograms of margins (how much a price
//             rise makes a holder leave / how much a price cut makes an outsider join) and the exact
//             smallest margin are collected.  The first sweep scans whole rows and caches each
//             token's 16 best experts with a bound on everything else; later sweeps re-evaluate the
//             cached entries only, and rescan a row (one warp) when the bound no longer vouches for
//             them.  A one-CTA kernel then moves each over- or under-loaded expert's price to the
//             histogram quantile that balances it, plus a step eps that is halved as the sweeps go
//             on; small imbalances move one exact margin at a time.  This is an epsilon-scaled
//             simultaneous price adjustment (auction-style); it ends a few dozen token moves away
//             from the optimum and stops early once a small imbalance has stopped shrinking.
//   collect   every token's top-k under the final prices is written out; tokens whose k-th and
//             (k+1)-th values differ by at most theta are listed as candidates.
//   build     the cost matrix D[e][f] = cheapest move of one candidate token from e to f is built by
//             the whole GPU (one warp per candidate, 64-bit atomicMin).
//   exact     one CTA runs successive shortest augmenting paths on the expert-level residual graph
//             (E experts + one node Z for the sink side) with D as arc costs; node potentials keep reduced costs non-negative, so each search is a
//             Bellman-Ford over E+1 nodes held in shared memory.  It ends with every expert within
//             capacity and complementary slackness satisfied for the candidates.
//   verify    a last data-parallel pass checks complementary slackness for EVERY token under the
//             final prices.  If a non-candidate token is violated, theta grows and collect/exact run
//             again.  Passing this check is a proof of optimality (LP duality of Eq. 7-8).
//
// All arithmetic is on int64 keys: key = rne(A * 2^40) (+ a 12-bit position hash) for float
// affinities, or the quantised logit with a hashed tie-break.
#pragma once
#include <cstddef>
#include "common.cuh"

namespace msr {

constexpr int kNB = 256;                  // histogram bins per expert: 4 per octave of the margin
constexpr int kTopN = kMaxK + 2;          // sorted values kept per token in a sweep
constexpr long long kInf = 1LL << 62;
constexpr long long kArcLimit = 1LL << 58; // arcs with a larger reduced cost are ignored by the exact phase
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
  if (!isfinite(x)) x = 0.f;   // reported separately by the collect pass
  // x * 2^40 is exact in fp32; the low 12 bits carry a multiplicative hash of the entry's position so
  // that identical rows do not tie exactly (it moves the optimum by less than 4e-9 per chosen pair)
  if (g.mode == 0) return __float2ll_rn(x * 1099511627776.0f) + (long long)((flat_idx * 2654435761u) >> 20);
  float sc = rintf(ldexpf(x, g.quant_shift));
  sc = fminf(fmaxf(sc, -32768.f), 32767.f);
  long long q = (long long)sc;
  uint32_t r = fmix32(flat_idx + g.seed_mul) >> 12;
  return q * (1LL << g.S) + (long long)r;
}

struct FlowState {
  int trace[128];            // diagnostics: [0..23] imbalance per sweep, [64..] rows scanned in full per sweep
  long long p[kMaxE];        // expert prices
  long long eps, eps_min;
  long long theta;           // candidate threshold of the next collect pass
  long long theta_used;      // threshold the current candidate list was collected with
  double total_score;
  int load[kMaxE];           // accumulated by the running pass, consumed by its last CTA
  int load_cur[kMaxE];       // loads of the assignment currently written in expert_idx
  alignas(16) unsigned hist_up[2][kMaxE * kNB];   // [sweep parity]; read and cleared with 16-byte accesses
  alignas(16) unsigned hist_dn[2][kMaxE * kNB];
  long long cumdrop;                              // sum over sweeps of the largest price decrease of that sweep
  int cut_max;                                    // log2 of the largest margin worth recording at all
  long long min_up[kMaxE], min_dn[kMaxE];   // smallest margin recorded by the running sweep (reset by the price update)
  int cap_up[kMaxE], cap_dn[kMaxE];   // log2 of the largest margin worth recording
  int flag_dn[kMaxE];                 // expert whose join-histogram came out short: scan it in full next sweep
  unsigned ticket;
  int sweep, p1_done, balanced;
  int best_imb, stall;                // smallest imbalance seen so far; sweeps since it last improved
  int round, converged, ncand, violations, naug, rerouted;
  unsigned status;
  int ncand_last;
};

static_assert(offsetof(FlowState, hist_up) % 16 == 0 && offsetof(FlowState, hist_dn) % 16 == 0 && (kMaxE * kNB * 4) % 16 == 0,
              "histograms are accessed as uint4");

// ---------------------------------------------------------------------------------------------
__global__ void flow_init_kernel(FlowState* st, long long eps0, long long eps_min, int cap0,
                                 long long theta0, int balanced, int E) {
  {   // both histogram buffers, by all CTAs of the launch
    uint4* zu = reinterpret_cast<uint4*>(st->hist_up[0]); uint4* zd = reinterpret_cast<uint4*>(st->hist_dn[0]);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 2 * kMaxE * kNB / 4; i += gridDim.x * blockDim.x) {
      zu[i] = make_uint4(0, 0, 0, 0); zd[i] = make_uint4(0, 0, 0, 0);
    }
  }
  if (blockIdx.x != 0) return;
  for (int e = threadIdx.x; e < kMaxE; e += blockDim.x) {
    st->p[e] = 0; st->load[e] = 0; st->load_cur[e] = 0; st->min_up[e] = kInf; st->min_dn[e] = kInf; st->cap_up[e] = cap0; st->cap_dn[e] = cap0; st->flag_dn[e] = 0;
  }
  if (threadIdx.x == 0) {
    st->eps = eps0; st->eps_min = eps_min; st->theta = theta0; st->total_score = 0.0;
    st->ticket = 0; st->sweep = 0; st->p1_done = 0; st->balanced = balanced; st->best_imb = 0x7fffffff; st->stall = 0;
    for (int i = 64; i < 128; ++i) st->trace[i] = 0;
    st->round = 0; st->converged = 0; st->ncand = 0; st->violations = 0; st->naug = 0;
    st->rerouted = 0; st->status = 0; st->ncand_last = 0; st->cut_max = cap0; st->cumdrop = 0;
  }
}

// Insert (val, id) into a list sorted by descending value, lower expert index first on equal values.
template <int N>
__device__ __forceinline__ void top_insert_tb(long long (&v)[N], int (&id)[N], long long val, int e) {
  if (val > v[N - 1] || (val == v[N - 1] && e < id[N - 1])) {
    v[N - 1] = val; id[N - 1] = e;
#pragma unroll
    for (int j = N - 1; j > 0; --j) {
      if (v[j] > v[j - 1] || (v[j] == v[j - 1] && id[j] < id[j - 1])) {
        long long tv = v[j]; v[j] = v[j - 1]; v[j - 1] = tv;
        int ti = id[j]; id[j] = id[j - 1]; id[j - 1] = ti;
      }
    }
  }
}

// Key in fp32 (24 significant bits): good enough to FIND the largest few entries of a row cheaply.
__device__ __forceinline__ float approx_key(const KeyGen& g, float x) {
  if (!isfinite(x)) x = 0.f;
  if (g.mode == 0) return x * 1099511627776.0f;
  return fminf(fmaxf(rintf(x * g.fshift), -32768.f), 32767.f) * g.fS;
}

// The N largest entries of key(e) - price(e) over one row, exact and sorted (value descending, lower
// expert index first on equal values).
//   1. a branch-free pass keeps the N largest fp32 approximations; the expert index rides in the low
//      7 mantissa bits, so each slot costs one max and one min;
//   2. the exact int64 values of those N experts are computed and sorted;
//   3. if `exact`, a second pass checks that no other expert beats the N-th one exactly; in the rare
//      case one does (values closer than fp32 resolves), the row is redone by exact insertion.
// Without `exact` the result may miss an entry that differs from the N-th by less than ~2^-17 relative.
template <int N>
__device__ __forceinline__ void select_top(const float* row, const long long* sp, const float* spf, const KeyGen& g,
                                           uint32_t flat, int E, int start, bool exact, long long (&v)[N],
                                           int (&id)[N]) {
  float pk[N];
#pragma unroll
  for (int j = 0; j < N; ++j) pk[j] = -INFINITY;
  int e = start;
  auto feed = [&](float val, int ee) {
    const float vf = approx_key(g, val) - (spf ? spf[ee] : 0.f);
    float x = __uint_as_float((__float_as_uint(vf) & ~127u) | (unsigned)ee);
#pragma unroll
    for (int j = 0; j < N; ++j) { const float hi = fmaxf(pk[j], x); x = fminf(pk[j], x); pk[j] = hi; }
  };
  if (start < 0) {
    // row in global memory: 16-byte loads, so that each 32-byte sector is fetched by two adjacent
    // instructions instead of eight that the L1 may not keep apart
    for (int e4 = 0; e4 < E; e4 += 4) {
      const float4 x4 = __ldg(reinterpret_cast<const float4*>(row + e4));
      feed(x4.x, e4); feed(x4.y, e4 + 1); feed(x4.z, e4 + 2); feed(x4.w, e4 + 3);
    }
    start = 0;
  } else {
    for (int jj = 0; jj < E; ++jj) {
      feed(row[e], e);
      if (++e == E) e = 0;
    }
  }
#pragma unroll
  for (int j = 0; j < N; ++j) {
    const bool ok = pk[j] != -INFINITY;
    const int ee = (int)(__float_as_uint(pk[j]) & 127u);
    id[j] = ok ? ee : -1;
    v[j] = ok ? make_key(g, row[ee], flat + ee) - (sp ? sp[ee] : 0) : -kInf;
  }
#pragma unroll
  for (int pass = 0; pass < N; ++pass) {
#pragma unroll
    for (int j = (pass & 1); j + 1 < N; j += 2) {
      if (v[j + 1] > v[j] || (v[j + 1] == v[j] && id[j + 1] >= 0 && id[j + 1] < id[j])) {
        const long long tv = v[j]; v[j] = v[j + 1]; v[j + 1] = tv;
        const int ti = id[j]; id[j] = id[j + 1]; id[j + 1] = ti;
      }
    }
  }
  if (!exact || id[N - 1] < 0) return;                 // E <= N: every expert is in the list
  const long long tv = v[N - 1]; const int ti = id[N - 1];
  bool missed = false;
  e = start;
  for (int jj = 0; jj < E; ++jj) {
    const long long val = make_key(g, row[e], flat + e) - (sp ? sp[e] : 0);
    if (val > tv || (val == tv && e < ti)) {
      bool in = false;
#pragma unroll
      for (int j = 0; j < N; ++j) in |= (id[j] == e);
      missed |= !in;
    }
    if (++e == E) e = 0;
  }
  if (!missed) return;
#pragma unroll
  for (int j = 0; j < N; ++j) { v[j] = -kInf; id[j] = -1; }
  for (e = 0; e < E; ++e) top_insert_tb(v, id, make_key(g, row[e], flat + e) - (sp ? sp[e] : 0), e);
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

// ---------------------------------------------------------------------------------------------
// One price sweep.
constexpr int kSweepThreads = 128;

// Per-token candidate cache of the sweeps.  A full scan of a token's row keeps its kCacheN best experts
// (score and index) and `bound` = the smallest of their values minus the total price drop so far.  A
// later sweep re-evaluates only those kCacheN entries; every other expert is worth at most
// bound + (total price drop now), so while the (k+2)-th cached value stays at or above that, the cached
// entries still contain the token's k+2 best experts and the row need not be read again.
constexpr int kCacheN = 16;
struct SweepCache {
  float* x;              // [kCacheN][T] scores of the cached experts
  unsigned char* id;     // [T][kCacheN] their indices (255 = none)
  long long* bound;      // [T]
};

struct SweepShared {
  long long sp[kMaxE];
  float spf[kMaxE];
  int sload[kMaxE], scu[kMaxE], scd[kMaxE], sflag[kMaxE];
  int nflag, nslow;
  unsigned short slow[kSweepThreads];
};

__device__ __forceinline__ void emit_margin(unsigned* hist, long long* mins, const int* caplog, int e, long long m) {
  if (m >= 0 && m < (1LL << caplog[e])) {
    atomicAdd(&hist[e * kNB + log_bin(m)], 1u);
    // the exact smallest margin, for steps that move one token; it only ever drops, so a stale read
    // can only let a useless atomic through
    if (m < __ldcg(&mins[e])) atomicMin(&mins[e], m);
  }
}

template <bool kFirst>   // the first sweep scans every row (one thread per token) and fills the cache
__global__ void __launch_bounds__(kSweepThreads)
flow_sweep_kernel(const float* __restrict__ M, FlowState* st, SweepCache cache, int T, int E, int k, int C,
                  KeyGen g, int sweep_index) {
  // the token's cache entries do not depend on anything the prologue reads: fetch them first, so that
  // their latency overlaps the state loads and barriers below
  uint4 pre_id = make_uint4(0, 0, 0, 0); float pre_x[kCacheN]; long long pre_bound = kInf;
  {
    const int tok = blockIdx.x * blockDim.x + threadIdx.x;
#pragma unroll
    for (int j = 0; j < kCacheN; ++j) pre_x[j] = 0.f;
    if (!kFirst && sweep_index > 0 && tok < T) {
      pre_id = *reinterpret_cast<const uint4*>(cache.id + (size_t)tok * kCacheN);
#pragma unroll
      for (int j = 0; j < kCacheN; ++j) pre_x[j] = cache.x[(size_t)j * T + tok];
      pre_bound = cache.bound[tok];
    }
  }
  if (*(volatile int*)&st->p1_done) return;
  // histograms alternate between two buffers: this sweep fills one while every CTA clears a slice of
  // the other for the next sweep (its last reader, the previous price update, has finished)
  const int sweep0 = sweep_index;                     // sweeps run in launch order; a finished phase returns above
  const long long cumdrop = st->cumdrop;
  const int par = sweep0 & 1;
  unsigned* hup = st->hist_up[par]; unsigned* hdn = st->hist_dn[par];
  long long* mup = st->min_up; long long* mdn = st->min_dn;
  {
    uint4* zu = reinterpret_cast<uint4*>(st->hist_up[par ^ 1]); uint4* zd = reinterpret_cast<uint4*>(st->hist_dn[par ^ 1]);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < kMaxE * kNB / 4; i += gridDim.x * blockDim.x) {
      zu[i] = make_uint4(0, 0, 0, 0); zd[i] = make_uint4(0, 0, 0, 0);
    }
  }
  __shared__ SweepShared sh;
  long long (&sp)[kMaxE] = sh.sp;
  int (&sload)[kMaxE] = sh.sload; int (&scu)[kMaxE] = sh.scu; int (&scd)[kMaxE] = sh.scd;
  if (threadIdx.x == 0) { sh.nflag = 0; sh.nslow = 0; }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    sp[e] = st->p[e]; sh.spf[e] = (float)sp[e]; sload[e] = 0; scu[e] = st->cap_up[e]; scd[e] = st->cap_dn[e];
    if (st->flag_dn[e]) sh.sflag[atomicAdd(&sh.nflag, 1)] = e;
  }
  __syncthreads();
  const int tok0 = blockIdx.x * blockDim.x;
  const int need = min(k + 2, E);                       // sorted values a token has to know
  const int nflag = sh.nflag;
  // ---- pass A, one thread per token: re-evaluate the cached experts -----------------------------
  {
    const int tok = tok0 + threadIdx.x;
    if (tok < T) {
      bool valid = false;
      if (kFirst) {
        const uint32_t flat = (uint32_t)tok * (uint32_t)E;
        const float* row = M + (size_t)tok * E;
        long long v[kCacheN]; int id[kCacheN];
        select_top(row, sp, sh.spf, g, flat, E, (E & 3) == 0 ? -1 : 0, false, v, id);
        unsigned idws[4] = {0, 0, 0, 0};
#pragma unroll
        for (int j = 0; j < kCacheN; ++j) {
          cache.x[(size_t)j * T + tok] = id[j] >= 0 ? __ldg(row + id[j]) : 0.f;
          idws[j >> 2] |= (unsigned)(id[j] >= 0 ? id[j] : 255) << (8 * (j & 3));
        }
        *reinterpret_cast<uint4*>(cache.id + (size_t)tok * kCacheN) = make_uint4(idws[0], idws[1], idws[2], idws[3]);
        cache.bound[tok] = id[kCacheN - 1] >= 0 ? v[kCacheN - 1] - cumdrop : -kInf;
        long long vk = -kInf, vk1 = -kInf;
#pragma unroll
        for (int j = 0; j < kCacheN; ++j) { if (j == k - 1) vk = v[j]; if (j == k) vk1 = v[j]; }
#pragma unroll
        for (int j = 0; j < kMaxK + 2; ++j) {
          const int e = id[j];
          if (j < k) {
            atomicAdd(&sload[e], 1);
            if (E > k) emit_margin(hup, mup, scu, e, v[j] - vk1);
          } else if (j <= k + 1 && e >= 0) {
            emit_margin(hdn, mdn, scd, e, vk - v[j]);
          }
        }
        valid = true;                                   // no expert is flagged before the first sweep
      } else if (sweep0 > 0) {
        const uint32_t flat = (uint32_t)tok * (uint32_t)E;
        const unsigned idws[4] = {pre_id.x, pre_id.y, pre_id.z, pre_id.w};
        long long v[kCacheN]; int rank[kCacheN];
#pragma unroll
        for (int j = 0; j < kCacheN; ++j) {
          const int e = (int)((idws[j >> 2] >> (8 * (j & 3))) & 255u);
          const float x = pre_x[j];
          v[j] = e < E ? make_key(g, x, flat + e) - sp[e] : -kInf;
          rank[j] = 0;
        }
#pragma unroll
        for (int j = 1; j < kCacheN; ++j)
#pragma unroll
          for (int i = 0; i < j; ++i) {
            const bool first = v[i] >= v[j];            // the earlier entry wins a tie
            rank[j] += first ? 1 : 0; rank[i] += first ? 0 : 1;
          }
        long long vk = -kInf, vk1 = -kInf, vneed = -kInf;
#pragma unroll
        for (int j = 0; j < kCacheN; ++j) {
          if (rank[j] == k - 1) vk = v[j];
          if (rank[j] == k) vk1 = v[j];
          if (rank[j] == need - 1) vneed = v[j];
        }
        const long long bound = pre_bound;
        valid = bound <= -kInf || vneed >= bound + cumdrop;
        if (valid) {
          const bool has_alt = E > k;
#pragma unroll
          for (int j = 0; j < kCacheN; ++j) {
            const int e = (int)((idws[j >> 2] >> (8 * (j & 3))) & 255u);
            if (rank[j] < k) {
              atomicAdd(&sload[e], 1);
              if (has_alt) emit_margin(hup, mup, scu, e, v[j] - vk1);        // price rise at which the token leaves e
            } else if (rank[j] <= k + 1 && e < E) {
              emit_margin(hdn, mdn, scd, e, vk - v[j]);                      // price cut at which the token joins e
            }
          }
          // experts whose join-histogram was short last time: count this token even if the expert is
          // not among its best alternatives
          for (int q = 0; q < nflag; ++q) {
            const int e = sh.sflag[q];
            bool seen = false;
#pragma unroll
            for (int j = 0; j < kCacheN; ++j)
              seen |= (rank[j] <= k + 1) && ((int)((idws[j >> 2] >> (8 * (j & 3))) & 255u) == e);
            if (seen) continue;
            emit_margin(hdn, mdn, scd, e, vk - (make_key(g, __ldg(M + (size_t)tok * E + e), flat + e) - sp[e]));
          }
        }
      }
      if (!valid) sh.slow[atomicAdd(&sh.nslow, 1)] = (unsigned short)threadIdx.x;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0 && sweep0 < 64 && sh.nslow) atomicAdd(&st->trace[64 + sweep0], sh.nslow);
  // ---- pass B, one warp per token whose cache no longer vouches for itself: scan the whole row ----
  {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nslow = sh.nslow;
    for (int s = warp; s < nslow; s += kSweepThreads / 32) {
      const int tok = tok0 + sh.slow[s];
      const uint32_t flat = (uint32_t)tok * (uint32_t)E;
      const float* row = M + (size_t)tok * E;
      // lane l looks at experts l, l+32, l+64, l+96.  fp32 approximations, the expert index in the low
      // 7 mantissa bits, mapped to unsigned integers that order the same way; 0 = absent
      unsigned u[kEPLf];
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        const int e = lane + 32 * q;
        u[q] = 0;
        if (e < E) {
          const float vf = approx_key(g, __ldg(row + e)) - sh.spf[e];
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
      // lanes 0..kCacheN-1 now hold the winners in descending approximate order; make them exact
      int ee = 255; float xv = 0.f; long long val = -kInf;
      if (lane < kCacheN && mine != 0) {
        const unsigned bits = (mine & 0x80000000u) ? (mine & 0x7fffffffu) : ~mine;
        ee = (int)(bits & 127u);
        xv = __ldg(row + ee);
        val = make_key(g, xv, flat + ee) - sp[ee];
      }
      if (lane < kCacheN) {
        cache.x[(size_t)lane * T + tok] = xv;
        cache.id[(size_t)tok * kCacheN + lane] = (unsigned char)ee;
      }
      // every expert outside the cache is worth no more than the last winner (none if E <= kCacheN)
      const long long vlast = __shfl_sync(0xffffffffu, val, kCacheN - 1);
      if (lane == 0) cache.bound[tok] = (vlast <= -kInf) ? -kInf : vlast - cumdrop;
      int rank = 0;
#pragma unroll
      for (int i = 0; i < kCacheN; ++i) {
        const long long vi = __shfl_sync(0xffffffffu, val, i);
        rank += (vi > val || (vi == val && i < lane)) ? 1 : 0;
      }
      const bool listed = lane < kCacheN && ee < E;
      const unsigned bk = __ballot_sync(0xffffffffu, listed && rank == k - 1);
      const unsigned bk1 = __ballot_sync(0xffffffffu, listed && rank == k);
      const long long vk = __shfl_sync(0xffffffffu, val, bk ? __ffs(bk) - 1 : 0);
      const long long vk1 = bk1 ? __shfl_sync(0xffffffffu, val, __ffs(bk1) - 1) : -kInf;
      if (listed) {
        if (rank < k) {
          atomicAdd(&sload[ee], 1);
          if (E > k) emit_margin(hup, mup, scu, ee, val - vk1);
        } else if (rank <= k + 1) {
          emit_margin(hdn, mdn, scd, ee, vk - val);
        }
      }
      for (int q = 0; q < nflag; ++q) {
        const int e = sh.sflag[q];
        const unsigned seen = __ballot_sync(0xffffffffu, listed && rank <= k + 1 && ee == e);
        if (!seen && lane == 0) emit_margin(hdn, mdn, scd, e, vk - (make_key(g, __ldg(row + e), flat + e) - sp[e]));
      }
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x)
    if (sload[e]) atomicAdd(&st->load[e], sload[e]);

}

// Price update that closes a sweep: one CTA, one warp per expert (four experts per warp, all their
// histograms in flight at once).
constexpr int kPriceThreads = 1024;
__global__ void __launch_bounds__(kPriceThreads)
flow_price_kernel(FlowState* st, int E, int C, int n_sweeps, int decay_every, int sweep_index) {
  // every input is loaded up front, independently of the others, so that the kernel pays two global
  // round trips (state, then the histogram rows picked by the sign of the imbalance), not one per field
  __shared__ long long sp[kMaxE];
  __shared__ int s_imb;
  __shared__ long long pmin, s_drop;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kPriceThreads / 32, kBatch = kMaxE / kWarps;
  const int par = sweep_index & 1;                    // the sweep this update closes filled these buffers
  const unsigned* hup = st->hist_up[par]; const unsigned* hdn = st->hist_dn[par];
  const int done_before = __ldcg(&st->p1_done);
  const long long eps = __ldcg(&st->eps), eps_min = __ldcg(&st->eps_min);
  const bool balanced = __ldcg(&st->balanced) != 0;
  const int cut_max = __ldcg(&st->cut_max), best_imb = __ldcg(&st->best_imb), stall_before = __ldcg(&st->stall);
  int xs[kBatch], cup[kBatch], cdn[kBatch]; long long ps[kBatch], mu[kBatch], md[kBatch];
#pragma unroll
  for (int b = 0; b < kBatch; ++b) {
    const int e = warp + b * kWarps;
    xs[b] = 0; ps[b] = 0; mu[b] = kInf; md[b] = kInf; cup[b] = 0; cdn[b] = 0;
    if (e < E) {
      xs[b] = __ldcg(&st->load[e]) - C; ps[b] = __ldcg(&st->p[e]);
      cup[b] = __ldcg(&st->cap_up[e]); cdn[b] = __ldcg(&st->cap_dn[e]);
      mu[b] = __ldcg(&st->min_up[e]); md[b] = __ldcg(&st->min_dn[e]);
    }
  }
  if (done_before) return;
  if (threadIdx.x == 0) { s_imb = 0; s_drop = 0; }
  uint4 ha[kBatch], hb[kBatch]; long long m1[kBatch];
#pragma unroll
  for (int b = 0; b < kBatch; ++b) {
    const int e = warp + b * kWarps;
    m1[b] = kInf; ha[b] = make_uint4(0, 0, 0, 0); hb[b] = ha[b];
    if (e < E) {
      const int x = xs[b];
      const bool up = x > 0, dn = x < 0 && (balanced || ps[b] > 0);
      if (up || dn) {
        const uint4* h = reinterpret_cast<const uint4*>((up ? hup : hdn) + e * kNB) + 2 * lane;
        ha[b] = __ldcg(h); hb[b] = __ldcg(h + 1);
        m1[b] = up ? mu[b] : md[b];
      }
    }
  }
  __syncthreads();
  int imb = 0; long long drop = 0;
#pragma unroll
  for (int b = 0; b < kBatch; ++b) {
    const int e = warp + b * kWarps;
    if (e >= E) continue;
    const int x = xs[b];
    long long p = ps[b];
    int flag = 0;
    if (x > 0) {
      int cl = cup[b]; bool shortw;
      p += price_step_warp(ha[b], hb[b], x, eps, cl, shortw, cut_max, m1[b]);
      if (lane == 0) st->cap_up[e] = cl;
      imb += x;
    } else if (x < 0 && (balanced || p > 0)) {
      int cl = cdn[b]; bool shortw;
      p -= price_step_warp(ha[b], hb[b], -x, eps, cl, shortw, cut_max, m1[b]);
      if (!balanced && p < 0) p = 0;
      if (lane == 0) st->cap_dn[e] = cl;
      flag = shortw ? 1 : 0;
      imb += -x;
    }
    p = p > kPriceLimit ? kPriceLimit : (p < -kPriceLimit ? -kPriceLimit : p);
    // when nothing was out of balance the prices stay put and the collect pass reproduces this state
    if (x == 0) p = ps[b];
    if (lane == 0) {
      st->flag_dn[e] = flag;
      st->load[e] = 0;
      st->min_up[e] = kInf; st->min_dn[e] = kInf;
      if (ps[b] - p > drop) drop = ps[b] - p;
      sp[e] = p;
    }
  }
  if (lane == 0) { if (imb) atomicAdd(&s_imb, imb); if (drop > 0) atomicMax(&s_drop, drop); }
  __syncthreads();
  const int sweep = sweep_index + 1;
  // a small imbalance that has stopped shrinking is a price war between a few experts: the exact phase
  // ends it faster than more sweeps would
  const int stall = s_imb < best_imb ? 0 : stall_before + 1;
  const bool done = (s_imb == 0) || sweep >= n_sweeps || (stall >= kStallSweeps && s_imb <= kStallImbalance);
  if (threadIdx.x == 0) {
    // prices are only defined up to a shift when every expert must be full; anchor the minimum at 0
    long long m = 0;
    if (done && balanced) { m = sp[0]; for (int e = 1; e < E; ++e) m = sp[e] < m ? sp[e] : m; }
    pmin = m;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) st->p[e] = sp[e] - pmin;
  if (threadIdx.x == 0) {
    if (sweep <= 40) st->trace[sweep - 1] = s_imb;
    st->sweep = sweep;
    st->stall = stall; if (stall == 0) st->best_imb = s_imb;
    st->cumdrop += s_drop;
    if (sweep % decay_every == 0) { long long ne = eps >> 1; st->eps = ne < eps_min ? eps_min : ne; }
    if (done) st->p1_done = 1;
  }
}

// fp32 <-> unsigned integers that order the same way (for the integer warp reductions)
__device__ __forceinline__ unsigned flip_f32(float f) {
  const unsigned b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float unflip_f32(unsigned u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// Approximate selection over one row held by a warp: the `count` largest fp32 values, one warp reduction
// each (the expert index rides in the low 7 mantissa bits, so values are distinct and the winner's
// owner is known).  sel[] marks the first `nsel`; v_a / v_b are the values picked as number nsel and
// nsel+1 (-inf where there is none).  The caller decides whether v_a - v_b is large enough to trust.
__device__ __forceinline__ void warp_select_f32(const float (&val)[kEPLf], int E, int count, bool (&sel)[kEPLf],
                                                float& v_a, float& v_b, int nsel) {
  const int lane = threadIdx.x & 31;
  unsigned u[kEPLf];
#pragma unroll
  for (int q = 0; q < kEPLf; ++q) {
    const int e = lane + 32 * q;
    u[q] = e < E ? flip_f32(__uint_as_float((__float_as_uint(val[q]) & ~127u) | (unsigned)e)) : 0u;
    sel[q] = false;
  }
  v_a = -INFINITY; v_b = -INFINITY;
  for (int r = 0; r < count && r < E; ++r) {
    unsigned m = u[0];
#pragma unroll
    for (int q = 1; q < kEPLf; ++q) m = max(m, u[q]);
    const unsigned w = __reduce_max_sync(0xffffffffu, m);
    const float v = unflip_f32(w);
    if (r == nsel - 1) v_a = v;
    if (r == nsel) v_b = v;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q)
      if (u[q] == w) { u[q] = 0u; if (r < nsel) sel[q] = true; }
  }
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
// Collect / verify pass.  The first pass picks every token's top-k under the sweep prices.  Later ones
// keep a token's experts when they still are a top-k under the current prices (ties included) and
// re-pick otherwise.  verify_only never re-picks: it only counts violations and gathers statistics.
__global__ void __launch_bounds__(kSweepThreads)
flow_collect_kernel(const float* __restrict__ M, FlowState* st, int32_t* __restrict__ expert_idx,
                    int32_t* __restrict__ cand, int T, int E, int k, int C, KeyGen g, int first,
                    int verify_only, long long theta_scale, int32_t* __restrict__ expert_load_out,
                    void* stats_out, const unsigned* __restrict__ error_flag, int unbounded, long long* __restrict__ Dg) {
  if (!verify_only && *(volatile int*)&st->converged) return;
  if (Dg)   // the move-cost matrix the build kernel fills next starts out empty
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < E * (E | 1); i += gridDim.x * blockDim.x) Dg[i] = kInf;
  __shared__ long long sp[kMaxE];
  __shared__ float spf[kMaxE];
  __shared__ int sload[kMaxE];
  __shared__ int s_viol, s_rer;
  __shared__ double s_score;
  __shared__ unsigned s_flags;
  for (int e = threadIdx.x; e < E; e += blockDim.x) { sp[e] = st->p[e]; spf[e] = (float)sp[e]; sload[e] = 0; }
  if (threadIdx.x == 0) { s_viol = 0; s_rer = 0; s_score = 0.0; s_flags = 0; }
  __syncthreads();
  const long long theta = unbounded ? kInf : st->theta;   // the last round lists every token
  // One warp per token, lane l holds experts l, l+32, l+64, l+96: coalesced row loads, every decision
  // by warp votes and reductions.  Decisions are first tried on fp32 approximations of key - price with
  // a rigorous error bound; only a token whose decision the bound cannot settle (a near-tie) is redone
  // on the exact int64 values.  A token may be listed as a candidate on the approximate gap: the list
  // only has to be a superset.
  const int lane = threadIdx.x & 31;
  const int wid = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), nwarp = gridDim.x * (blockDim.x >> 5);
  const float hash_bound = g.mode == 0 ? 4096.f : 1048576.f;      // key - approx_key lies in [-0.5, this)
  const float thetaf = theta >= kInf ? INFINITY : (float)theta * 1.0000005f;
  int w_viol = 0, w_rer = 0; double w_score = 0.0; bool w_bad = false;
  // the next token's row and experts are fetched while the current token is worked on
  float nx[kEPLf]; int nmine = -1;
  auto fetch = [&](int t) {
    if (t >= T) return;
    const float* r = M + (size_t)t * E;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) { const int e = lane + 32 * q; nx[q] = e < E ? __ldg(r + e) : 0.f; }
    nmine = (!first && lane < k) ? expert_idx[(size_t)t * k + lane] : -1;
  };
  fetch(wid);
  for (int tok = wid; tok < T; tok += nwarp) {
    const uint32_t flat = (uint32_t)tok * (uint32_t)E;
    float x[kEPLf], kf[kEPLf], vf[kEPLf]; bool in[kEPLf];
    const int mine = nmine;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) x[q] = nx[q];
    fetch(tok + nwarp);
    float mag = 0.f;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      const int e = lane + 32 * q;
      w_bad |= !isfinite(x[q]);
      kf[q] = e < E ? approx_key(g, x[q]) : -INFINITY;
      const float pf = e < E ? spf[e] : 0.f;
      vf[q] = kf[q] - pf;
      if (e < E) mag = fmaxf(mag, fabsf(kf[q]) + fabsf(pf));
      in[q] = false;
    }
    // |approximation - exact| <= hash_bound + 2^-15 * (|key| + |price|): float conversion of the price,
    // one rounding of the difference, and the 7 mantissa bits that carry the expert index in selections
    mag = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mag)));
    const float err3 = 3.f * (hash_bound + mag * (1.f / 32768.f));
    if (!first)
      for (int j = 0; j < k; ++j) {
        const int ej = __shfl_sync(0xffffffffu, mine, j);
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) in[q] |= (ej == lane + 32 * q);
      }
    bool settled = false, list = false, keep = false;
    if (!first) {
      float mh = INFINITY, mn = -INFINITY;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        if (lane + 32 * q >= E) continue;
        if (in[q]) mh = fminf(mh, vf[q]); else mn = fmaxf(mn, vf[q]);
      }
      mh = unflip_f32(__reduce_min_sync(0xffffffffu, flip_f32(mh)));
      mn = unflip_f32(__reduce_max_sync(0xffffffffu, flip_f32(mn)));
      const float diff = mh - mn;
      if (diff > err3) {                                // certainly still a top-k (E == k: diff = inf)
        settled = true; keep = true;
        list = E > k && (diff - err3 <= thetaf);
      }
    } else {
      float vkf, vk1f; bool sel[kEPLf];
      warp_select_f32(vf, E, k + 1, sel, vkf, vk1f, k);
      if (vkf - vk1f > err3) {                          // the approximate top-k is certainly the exact one
        settled = true;
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) in[q] = sel[q];
        list = E > k && (vkf - vk1f - err3 <= thetaf);
      }
    }
    long long key[kEPLf];
    bool have_keys = false;
    if (!settled) {
      long long val[kEPLf];
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        const int e = lane + 32 * q;
        key[q] = e < E ? make_key(g, x[q], flat + e) : -kInf;
        val[q] = e < E ? key[q] - sp[e] : -kInf;
      }
      have_keys = true;
      // exact check of the experts the token holds now: the worst held value against the best other one
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
      keep = !first && (min_held >= max_non);
      long long gap = keep ? ((E > k) ? min_held - max_non : kInf) : kInf;
      if (!verify_only && !keep) {
        long long vk = -kInf, vk1 = -kInf;
        warp_select(val, E, k + 1, in, vk, vk1, k);
        gap = (E > k) ? vk - vk1 : kInf;
      }
      list = gap < kInf && gap <= theta;
    }
    if (!keep && !first) ++w_viol;
    // the experts in ascending order: word q of the held mask is the vote over in[q]
    unsigned words[kEPLf]; int below = 0;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) words[q] = __ballot_sync(0xffffffffu, in[q]);
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      if (in[q]) {
        const int rank = below + __popc(words[q] & ((1u << lane) - 1u));
        if (rank < k) expert_idx[(size_t)tok * k + rank] = lane + 32 * q;
        atomicAdd(&sload[lane + 32 * q], 1);
      }
      below += __popc(words[q]);
    }
    if (verify_only) {
      // statistics: the score of the held pairs, and how many of them are not in the token's own top-k
      // of raw keys (the k-th and (k+1)-th raw keys must be told apart for certain, else exact keys decide)
      float rkf, rk1f; bool rsel[kEPLf];
      warp_select_f32(kf, E, k + 1, rsel, rkf, rk1f, k);
      int rer = 0; double sc = 0.0;
      if (rkf - rk1f > err3) {
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) rer += (in[q] && !rsel[q]) ? 1 : 0;
      } else {
        if (!have_keys) {
#pragma unroll
          for (int q = 0; q < kEPLf; ++q) { const int e = lane + 32 * q; key[q] = e < E ? make_key(g, x[q], flat + e) : -kInf; }
          have_keys = true;
        }
        long long kth_raw = -kInf, next_raw = -kInf;
        warp_select(key, E, k, rsel, kth_raw, next_raw, k);
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) rer += (in[q] && key[q] < kth_raw) ? 1 : 0;
      }
#pragma unroll
      for (int q = 0; q < kEPLf; ++q)
        if (in[q]) sc += (g.mode == 0) ? (double)x[q] : (double)(have_keys ? key[q] : make_key(g, x[q], flat + lane + 32 * q));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) { sc += __shfl_xor_sync(0xffffffffu, sc, o); rer += __shfl_xor_sync(0xffffffffu, rer, o); }
      w_score += sc; w_rer += rer;
    }
    if (!verify_only && list && lane == 0)
      cand[atomicAdd(&st->ncand, 1)] = tok;     // the list has room for every token
  }
  if (__any_sync(0xffffffffu, w_bad) && lane == 0) atomicOr(&s_flags, 2u);
  if (lane == 0) {
    if (w_viol) atomicAdd(&s_viol, w_viol);
    if (verify_only) { atomicAdd(&s_score, w_score); if (w_rer) atomicAdd(&s_rer, w_rer); }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x)
    if (sload[e]) atomicAdd(&st->load[e], sload[e]);
  if (threadIdx.x == 0) {
    if (s_viol) atomicAdd(&st->violations, s_viol);
    if (s_flags) atomicOr(&st->status, s_flags);
    if (verify_only) { atomicAdd(&st->total_score, s_score); if (s_rer) atomicAdd(&st->rerouted, s_rer); }
  }
  if (!last_block_arrives(&st->ticket)) return;
  // ---- last CTA: is the state a certificate? ---------------------------------------------------
  __shared__ int s_badload;
  if (threadIdx.x == 0) s_badload = 0;
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const int load = __ldcg(&st->load[e]);
    st->load_cur[e] = load;
    st->load[e] = 0;
    if (verify_only && expert_load_out) expert_load_out[e] = load;
    // primal feasibility and complementary slackness on the expert -> sink arcs
    if (load > C || (sp[e] > 0 && load < C)) atomicAdd(&s_badload, 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int viol = *(volatile int*)&st->violations;
    const bool ok = (first || viol == 0) && s_badload == 0;
    {   // diagnostics: per round, violations / experts out of balance / augmentations so far / candidates
      const int r = st->round < 4 ? st->round : 3;
      st->trace[48 + 4 * r] = viol; st->trace[49 + 4 * r] = s_badload; st->trace[50 + 4 * r] = st->naug;
      st->trace[51 + 4 * r] = st->ncand;
    }
    st->violations = 0;
    st->ticket = 0;
    if (!verify_only) {
      st->round = st->round + 1;
      st->theta_used = theta;
      st->theta = (theta > (kInf >> 8)) ? kInf : theta * theta_scale;   // next round looks further
    }
    if (verify_only && !ok) atomicOr(&st->status, 1u);
    if (verify_only && error_flag && *error_flag) atomicOr(&st->status, 4u);
    __threadfence();
    if (ok) st->converged = 1;
    if (verify_only && stats_out) {
      // layout of maxscore_stats: status, capacity, sweeps, augmentations, rounds, candidates,
      // rerouted, reserved, total_score
      int* so = reinterpret_cast<int*>(stats_out);
      so[0] = (int)(*(volatile unsigned*)&st->status & 7u);
      so[1] = C; so[2] = st->sweep; so[3] = st->naug; so[4] = st->round;
      so[5] = st->ncand_last; so[6] = *(volatile int*)&st->rerouted; so[7] = 0;
      *reinterpret_cast<double*>(so + 8) = *(volatile double*)&st->total_score;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Exact phase: successive shortest augmenting paths on the expert-level residual graph, one CTA.
//
// Only candidate tokens (gap <= theta) are in the graph.  A round stops BEFORE an augmentation whose
// price update would spread the experts' price changes of this round by more than theta: up to that
// point no token outside the list can have lost its top-k, so the state handed to the next collect
// pass is consistent, and that pass only has to list more tokens.
//
// D[e][f] (shared memory) is the cheapest move of one candidate token from e to f.  After a token
// moves u -> v only row u is rebuilt; the rows of its other experts and of v are patched from the
// token's own keys.  The experts of the first kHeldCache candidates are mirrored in shared memory
// (expert_idx itself is edited in place as well); the list is sorted first, so ties are broken by
// the smallest token index whatever order the collect pass appended the tokens in.
constexpr int kP2Threads = 1024;
constexpr int kHeldCache = 4096;
constexpr int kMaxFix = 256;
constexpr int kMaxArcs = 8192;      // finite arcs of D the Bellman-Ford search can list
constexpr int kSortMax = 16384;     // candidate lists up to this length are sorted (they fit in D's space)

// First build of D for a round, spread over the whole GPU: one warp per candidate token, results
// merged into global memory with 64-bit atomicMin.  (Inside the exact phase's single CTA the same
// work costs a quarter of a millisecond at 1 600 candidates.)
__global__ void __launch_bounds__(256)
flow_build_kernel(const float* __restrict__ M, const FlowState* st, const int32_t* __restrict__ expert_idx,
                  const int32_t* __restrict__ cand, long long* __restrict__ Dg, int T, int E, int k, KeyGen g) {
  if (*(volatile const int*)&st->converged) return;
  __shared__ long long sp[kMaxE];
  for (int e = threadIdx.x; e < E; e += blockDim.x) sp[e] = st->p[e];
  __syncthreads();
  const int n = min(st->ncand, T);
  const int ES = E | 1;
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
    long long key[kEPLf]; bool in[kEPLf];
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      const int f = lane + 32 * q;
      key[q] = f < E ? make_key(g, __ldg(row + f), flat + f) : 0;
      bool hd = f >= E;
#pragma unroll
      for (int j = 0; j < kMaxK; ++j) hd |= (h[j] == f);
      in[q] = hd;
    }
    long long vmax = -kInf;
#pragma unroll
    for (int q = 0; q < kEPLf; ++q) {
      const int f = lane + 32 * q;
      if (!in[q]) { const long long val = key[q] - sp[f]; vmax = val > vmax ? val : vmax; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const long long ov = __shfl_xor_sync(0xffffffffu, vmax, o);
      vmax = ov > vmax ? ov : vmax;
    }
#pragma unroll
    for (int j = 0; j < kMaxK; ++j) {
      if (j >= k) continue;
      const int e = h[j];
      long long mine = 0;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) if ((e >> 5) == q) mine = key[q];
      const long long we = __shfl_sync(0xffffffffu, mine, e & 31);
      const long long pe = sp[e];
      if (arc_window < kInf && (we - pe) - vmax > arc_window) continue;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        const int f = lane + 32 * q;
        if (!in[q]) {
          const long long cst = we - key[q];
          if (cst - pe + sp[f] <= arc_window && cst < Dg[e * ES + f]) atomicMin(&Dg[e * ES + f], cst);
        }
      }
    }
  }
}

struct P2Shared {
  long long p[kMaxE + 1];        // potentials: prices of the experts, then Z
  long long p0[kMaxE + 1];       // potentials at the start of the round
  long long dist[2][kMaxE + 1];  // [0] current, [1] snapshot of the previous round
  int pred[kMaxE + 1];
  unsigned char act[2][kMaxE + 4];   // nodes whose distance changed in the last round
  int imb[kMaxE + 1];            // + excess, - deficit
  int flow[kMaxE];               // units on expert -> sink
  int dirty[kMaxE];
  unsigned char fixrow[kMaxE];   // rows that have a stale entry to recompute
  int path[kMaxE + 2];
  int npath, changed, who, target, stop, any_pos, qn, nfix, narc, bf_bad, dup;
  int who_a[kMaxE + 2];          // per arc of the path: the candidate that moves
  int fix_e[kMaxFix], fix_f[kMaxFix];   // stale D entries to recompute after a move
  long long dt;
};

__global__ void __launch_bounds__(kP2Threads)
flow_exact_kernel(const float* __restrict__ M, FlowState* st, int32_t* expert_idx, int32_t* cand, int T, int E,
                  int k, int C, KeyGen g, int max_aug, const long long* __restrict__ Dg) {
  if (*(volatile int*)&st->converged) return;
  extern __shared__ __align__(16) unsigned char p2smem[];
  long long* D = reinterpret_cast<long long*>(p2smem);                              // [E][E] raw arc costs
  unsigned char* held_s = reinterpret_cast<unsigned char*>(D + (size_t)E * (E | 1));       // [kHeldCache][kMaxK]
  int* cand_s = reinterpret_cast<int*>(held_s + (size_t)kHeldCache * kMaxK);          // [kHeldCache]
  int* queue_s = cand_s + kHeldCache;                                                // [kHeldCache]
  unsigned short* arcs_s = reinterpret_cast<unsigned short*>(queue_s + kHeldCache);  // [kMaxArcs] (u << 8 | v)
  __shared__ P2Shared s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = min(st->ncand, T);
  const int nZ = E;   // index of Z
  const int ES = E | 1;   // odd row stride of D: a warp walking down a column hits different banks
  const long long theta = st->theta_used;
  const long long arc_window = theta >= (kInf >> 2) ? kInf : 2 * theta;

  // ---- sort the candidate list (in D's space, not yet in use) ----------------------------------------
  if (n > 1 && n <= kSortMax && (size_t)n * 4 <= (size_t)E * (E | 1) * 8) {
    int* buf = reinterpret_cast<int*>(D);
    int npow = 1; while (npow < n) npow <<= 1;
    if ((size_t)npow * 4 <= (size_t)E * (E | 1) * 8) {
      for (int i = tid; i < npow; i += blockDim.x) buf[i] = i < n ? cand[i] : 0x7fffffff;
      __syncthreads();
      for (int size = 2; size <= npow; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
          for (int i = tid; i < npow; i += blockDim.x) {
            const int j = i ^ stride;
            if (j > i) {
              const bool up = (i & size) == 0;
              const int a = buf[i], b = buf[j];
              if ((a > b) == up) { buf[i] = b; buf[j] = a; }
            }
          }
          __syncthreads();
        }
      for (int i = tid; i < n; i += blockDim.x) cand[i] = buf[i];
      __syncthreads();
    }
  }
  const int nc = min(n, kHeldCache);
  for (int i = tid; i < nc; i += blockDim.x) cand_s[i] = cand[i];
  __syncthreads();
  for (int i = tid; i < nc * k; i += blockDim.x) {
    const int c = i / k, j = i - c * k;
    held_s[c * kMaxK + j] = (unsigned char)expert_idx[(size_t)cand_s[c] * k + j];
  }
  auto tok_of = [&](int c) -> int { return c < nc ? cand_s[c] : cand[c]; };
  auto held_of = [&](int c, int tok, int j) -> int {
    return c < nc ? (int)held_s[c * kMaxK + j] : expert_idx[(size_t)tok * k + j];
  };

  for (int e = tid; e < E; e += blockDim.x) {
    s.p[e] = st->p[e]; s.p0[e] = s.p[e];
    const int load = st->load_cur[e];
    const int fl = s.p[e] > 0 ? C : min(load, C);
    s.flow[e] = fl; s.imb[e] = load - fl; s.dirty[e] = 0;
  }
  for (int i = tid; i < E * ES; i += blockDim.x) D[i] = Dg[i];       // built by flow_build_kernel
  __syncthreads();
  if (tid == 0) {
    int tot = 0;
    for (int e = 0; e < E; ++e) tot += s.imb[e];
    s.imb[nZ] = -tot; s.p[nZ] = 0; s.p0[nZ] = 0; s.stop = 0;
  }
  __syncthreads();

  int naug = 0;
  int bf_rounds = 0; long long q_total = 0, t_first = 0;
  long long t_who = 0, t_patch = 0, t_fix = 0; int n_arcs = 0;
  long long t_rebuild = 0, t_bf = 0, t_move = 0, t0 = clock64();   // phase timers (thread 0), diagnostics
  for (;;) {
    // ---- rebuild the rows of D marked dirty: D[e][f] = min over candidates in e, not in f ----------
    for (int i = tid; i < E * ES; i += blockDim.x)
      if (s.dirty[i / ES]) D[i] = kInf;
    __syncthreads();
    // cached candidates that hold a dirty row are queued first (one thread each, shared memory only);
    // the warps then work through the queue and through the uncached tail of the list
    if (tid == 0) s.qn = 0;
    __syncthreads();
    for (int c0 = 0; c0 < nc; c0 += blockDim.x) {
      const int c = c0 + tid;
      bool any = false;
      if (c < nc)
        for (int j = 0; j < k; ++j) any |= (s.dirty[held_s[c * kMaxK + j]] != 0);
      const unsigned mask = __ballot_sync(0xffffffffu, any);
      int base = 0;
      if (lane == 0 && mask) base = atomicAdd(&s.qn, __popc(mask));
      base = __shfl_sync(0xffffffffu, base, 0);
      if (any) queue_s[base + __popc(mask & ((1u << lane) - 1u))] = c;
    }
    __syncthreads();
    const int work = s.qn + (n - nc);
    q_total += work; if (naug == 0 && t_first == 0) t_first = -1;
    for (int i = warp; i < work; i += kP2Threads / 32) {
      const int c = i < s.qn ? queue_s[i] : nc + (i - s.qn);
      const int tok = tok_of(c);
      int h[kMaxK];
      bool any = false;
#pragma unroll
      for (int j = 0; j < kMaxK; ++j) {
        h[j] = j < k ? held_of(c, tok, j) : -1;
        if (j < k) any |= (s.dirty[h[j]] != 0);
      }
      if (!any) continue;
      const float* row = M + (size_t)tok * E;
      const uint32_t flat = (uint32_t)tok * (uint32_t)E;
      long long key[kEPLf];
      bool in[kEPLf];
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        const int f = lane + 32 * q;
        key[q] = f < E ? make_key(g, __ldg(row + f), flat + f) : 0;
        bool hd = f >= E;
#pragma unroll
        for (int j = 0; j < kMaxK; ++j) hd |= (h[j] == f);
        in[q] = hd;
      }
      // best value among the experts the token does not hold: a held expert further than the arc
      // window above it has no usable move at all
      long long vmax = -kInf;
#pragma unroll
      for (int q = 0; q < kEPLf; ++q) {
        const int f = lane + 32 * q;
        if (!in[q]) { const long long val = key[q] - s.p[f]; vmax = val > vmax ? val : vmax; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const long long ov = __shfl_xor_sync(0xffffffffu, vmax, o);
        vmax = ov > vmax ? ov : vmax;
      }
#pragma unroll
      for (int j = 0; j < kMaxK; ++j) {
        if (j >= k) continue;
        const int e = h[j];
        if (!s.dirty[e]) continue;
        long long mine = 0;
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) if ((e >> 5) == q) mine = key[q];
        const long long we = __shfl_sync(0xffffffffu, mine, e & 31);
        // only moves whose reduced cost is within 2*theta can be used before this round ends
        const long long pe = s.p[e];
        if (arc_window < kInf && (we - pe) - vmax > arc_window) continue;
#pragma unroll
        for (int q = 0; q < kEPLf; ++q) {
          const int f = lane + 32 * q;
          if (!in[q]) {
            const long long cst = we - key[q];
            // D only ever decreases, so a stale read can only let a useless atomic through
            if (cst - pe + s.p[f] <= arc_window && cst < D[e * ES + f]) atomicMin(&D[e * ES + f], cst);
          }
        }
      }
    }
    __syncthreads();
    for (int e = tid; e < E; e += blockDim.x) s.dirty[e] = 0;
    {
      const int any = __syncthreads_or(tid <= E && s.imb[tid] > 0);
      if (tid == 0) s.any_pos = any;
    }
    __syncthreads();
    { const long long t1 = clock64(); t_rebuild += t1 - t0; if (t_first == -1) t_first = t1 - t0; t0 = t1; }
    if (!s.any_pos || naug >= max_aug) break;

    // ---- shortest paths from every node with excess ---------------------------------------------------
    // First choice: synchronous Bellman-Ford over the list of finite arcs of D (a few thousand after the
    // window filter), all threads, distance and predecessor packed in one word (dist << 8 | pred) so
    // that one atomicMin keeps them consistent.  A node is only updated when its distance strictly
    // drops against the previous round, so the predecessor graph has no cycle.  If the arc list does
    // not fit, or distances leave the packed range, the single-warp Dijkstra below takes over.
    bool have_paths = false;
    {
      if (tid == 0) s.narc = 0;
      __syncthreads();
      for (int i0 = 0; i0 < E * ES; i0 += blockDim.x) {      // one counter update per warp, not per arc
        const int i = i0 + tid;
        const int u = i / ES, v = i - u * ES;
        const bool finite = i < E * ES && v < E && D[i] < kInf;
        const unsigned mask = __ballot_sync(0xffffffffu, finite);
        int base = 0;
        if (lane == 0 && mask) base = atomicAdd(&s.narc, __popc(mask));
        base = __shfl_sync(0xffffffffu, base, 0);
        const int slot = base + __popc(mask & ((1u << lane) - 1u));
        if (finite && slot < kMaxArcs) arcs_s[slot] = (unsigned short)((u << 8) | v);
      }
      __syncthreads();
      if (s.narc <= kMaxArcs) {
        const int narc = s.narc;
        constexpr long long kPInf = 0x7fffffffffffffffLL;
        constexpr long long kBfLimit = 1LL << 46;     // arcs and distances beyond this leave the packed range
        long long* pd0 = s.dist[0]; long long* pd1 = s.dist[1];
        for (int v = tid; v <= E; v += blockDim.x) pd0[v] = s.imb[v] > 0 ? 255LL : kPInf;   // dist 0, no pred
        if (tid == 0) s.bf_bad = 0;
        __syncthreads();
        for (int round = 0; round <= E + 1; ++round) {
          for (int v = tid; v <= E; v += blockDim.x) pd1[v] = pd0[v];
          if (tid == 0) s.changed = 0;
          __syncthreads();
          for (int a = tid; a < narc; a += blockDim.x) {
            const int u = arcs_s[a] >> 8, v = arcs_s[a] & 255;
            const long long pu = pd0[u];
            if (pu == kPInf) continue;
            long long rc = D[u * ES + v] - s.p[u] + s.p[v];
            if (rc < 0) rc = 0;
            if (rc >= kBfLimit) { s.bf_bad = 1; continue; }
            const long long nd = (pu >> 8) + rc;
            if (nd >= kBfLimit) { s.bf_bad = 1; continue; }
            const long long old = pd0[v];
            if (old == kPInf || nd < (old >> 8)) { atomicMin(&pd1[v], (nd << 8) | u); s.changed = 1; }
          }
          for (int e = tid; e < E; e += blockDim.x) {      // the arcs through Z
            const long long pe = pd0[e], pz = pd0[nZ];
            if (pe != kPInf && s.flow[e] < C) {
              long long rc = -s.p[e] + s.p[nZ]; if (rc < 0) rc = 0;
              const long long nd = (pe >> 8) + rc;
              if (rc >= kBfLimit || nd >= kBfLimit) s.bf_bad = 1;
              else if (pz == kPInf || nd < (pz >> 8)) { atomicMin(&pd1[nZ], (nd << 8) | e); s.changed = 1; }
            }
            if (pz != kPInf && s.flow[e] > 0) {
              long long rc = -s.p[nZ] + s.p[e]; if (rc < 0) rc = 0;
              const long long nd = (pz >> 8) + rc;
              if (rc >= kBfLimit || nd >= kBfLimit) s.bf_bad = 1;
              else if (pe == kPInf || nd < (pe >> 8)) { atomicMin(&pd1[e], (nd << 8) | nZ); s.changed = 1; }
            }
          }
          __syncthreads();
          long long* t = pd0; pd0 = pd1; pd1 = t;
          ++bf_rounds;
          const bool more = s.changed != 0;
          __syncthreads();
          if (!more) break;
        }
        if (!s.bf_bad) {
          // unpack; nearest node with a deficit (lowest index on ties)
          long long dv = kInf; int pv = -1;
          if (tid <= E) {
            const long long w = pd0[tid];
            if (w != kPInf) { dv = w >> 8; pv = (int)(w & 255); if (pv == 255) pv = -1; }
          }
          __syncthreads();
          if (tid <= E) { s.dist[0][tid] = dv; s.pred[tid] = pv; }
          __syncthreads();
          if (warp == 0) {
            long long dt = kInf; int t = 0x7fffffff;
            for (int v = lane; v <= E; v += 32)
              if (s.imb[v] < 0 && s.dist[0][v] < dt) { dt = s.dist[0][v]; t = v; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              const long long od = __shfl_xor_sync(0xffffffffu, dt, o);
              const int ot = __shfl_xor_sync(0xffffffffu, t, o);
              if (od < dt || (od == dt && ot < t)) { dt = od; t = ot; }
            }
            if (lane == 0) { s.target = dt < kInf ? t : -1; s.dt = dt; }
          }
          __syncthreads();
          have_paths = s.target >= 0;
        }
      }
    }
    // ---- Dijkstra from every node with excess (reduced costs rc = cost - p[u] + p[v] are >= 0) ---------
    if (!have_paths)

    // One warp, nodes spread over its lanes; it stops when the first node with a deficit is settled:
    // every node still open is at least that far away, which is all the price update needs to know.
    if (warp == 0) {
      constexpr int NQ = (kMaxE + 1 + 31) / 32;
      long long d[NQ]; int pr[NQ]; bool open[NQ];
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const int v = lane + 32 * q;
        open[q] = v <= E;
        d[q] = (v <= E && s.imb[v] > 0) ? 0 : kInf;
        pr[q] = -1;
      }
      int target = -1; long long dt = kInf;
      // all nodes with excess start at distance 0: settle them together and relax their arcs in one go
#pragma unroll
      for (int q = 0; q < NQ; ++q) if (open[q] && d[q] == 0) open[q] = false;
      for (int u = 0; u <= E; ++u) {
        if (s.imb[u] <= 0) continue;
        const long long pu = s.p[u];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          const int v = lane + 32 * q;
          if (!open[q]) continue;
          long long rc;
          if (u < E && v < E) {
            const long long c = D[u * ES + v];
            if (c >= kInf) continue;
            rc = c - pu + s.p[v];
          } else if (v == nZ) {
            if (s.flow[u] >= C) continue;
            rc = -pu + s.p[nZ];
          } else {
            if (s.flow[v] <= 0) continue;
            rc = -pu + s.p[v];
          }
          if (rc < 0) rc = 0;
          if (rc >= kArcLimit) continue;
          if (rc < d[q]) { d[q] = rc; pr[q] = u; }
        }
      }
      for (int it = 0; it <= E; ++it) {
        long long best = kInf; int bv = 0x7fffffff;
#pragma unroll
        for (int q = 0; q < NQ; ++q)
          if (open[q] && d[q] < best) { best = d[q]; bv = lane + 32 * q; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const long long ob = __shfl_xor_sync(0xffffffffu, best, o);
          const int ov = __shfl_xor_sync(0xffffffffu, bv, o);
          if (ob < best || (ob == best && ov < bv)) { best = ob; bv = ov; }
        }
        if (best >= kInf) break;                       // nothing reachable is left
        const int u = bv; const long long du = best;
#pragma unroll
        for (int q = 0; q < NQ; ++q) if (lane + 32 * q == u) open[q] = false;
        ++bf_rounds;
        if (s.imb[u] < 0) { target = u; dt = du; break; }
        const long long pu = s.p[u];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          const int v = lane + 32 * q;
          if (!open[q]) continue;
          long long rc;
          if (u < E && v < E) {
            const long long c = D[u * ES + v];
            if (c >= kInf) continue;
            rc = c - pu + s.p[v];
          } else if (v == nZ) {          // expert u -> Z: one more unit on u -> sink
            if (s.flow[u] >= C) continue;
            rc = -pu + s.p[nZ];
          } else {                       // Z -> expert v: one unit less on v -> sink
            if (s.flow[v] <= 0) continue;
            rc = -pu + s.p[v];
          }
          if (rc < 0) rc = 0;            // cannot happen while the potentials are valid
          if (rc >= kArcLimit) continue;
          if (du + rc < d[q]) { d[q] = du + rc; pr[q] = u; }
        }
      }
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const int v = lane + 32 * q;
        if (v <= E) {
          // settled nodes keep their distance; open ones are at least dt away
          s.dist[0][v] = open[q] ? kInf : d[q];
          s.pred[v] = pr[q];
        }
      }
      if (lane == 0) { s.target = target; s.dt = dt; }
    }
    __syncthreads();
    const int cur = 0;
    // ---- nearest node with a deficit; would the price update stay within theta? -----------------------
    if (warp == 0) {
      const int t = s.target; const long long dt = s.dt;
      if (lane == 0) s.npath = 0;
      if (t >= 0) {
        if (lane == 0) {
          int len = 0, v = t;
          while (v >= 0 && len <= E + 1) { s.path[len++] = v; v = s.pred[v]; }
          s.npath = len;
        }
        long long lo = kInf, hi = -kInf;
        for (int e = lane; e < E; e += 32) {
          const long long d = s.dist[cur][e];
          const long long chg = s.p[e] - (d < dt ? d : dt) - s.p0[e];
          lo = chg < lo ? chg : lo; hi = chg > hi ? chg : hi;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const long long ol = __shfl_xor_sync(0xffffffffu, lo, o), oh = __shfl_xor_sync(0xffffffffu, hi, o);
          lo = ol < lo ? ol : lo; hi = oh > hi ? oh : hi;
        }
        __syncwarp();
        if (lane == 0 && theta < kInf && hi - lo > theta) {
          s.target = -2;                                // stop here; the next round lists more tokens:
          if (st->theta < 2 * (hi - lo)) st->theta = 2 * (hi - lo);   // enough of them for this price update
        }
      }
    }
    __syncthreads();
    { const long long t1 = clock64(); t_bf += t1 - t0; t0 = t1; }
    if (s.target < 0) break;        // -1: no augmenting path inside the candidate graph
    for (int v = tid; v <= E; v += blockDim.x) {
      const long long d = s.dist[cur][v];
      s.p[v] -= (d < s.dt ? d : s.dt);
    }
    __syncthreads();
    // ---- push one unit along the path (stored target first) ------------------------------------------
    // All arcs of the path at once: (W) every thread looks up, for its candidates, which arcs they are
    // the cheapest token of; (P) one warp per arc patches D from that token's keys and lists the entries
    // that became stale; (F) one pass recomputes the listed entries.  The path's nodes are distinct, so
    // arcs touch different (row, column) pairs except where a min-update is used.  If one token is the
    // cheapest of two arcs the arcs are taken one by one instead (below).
    auto fix_pass = [&]() {
        if (s.nfix > 0 && n <= kHeldCache) {
          // recompute the listed entries: candidates that hold one of the listed rows are queued by one
          // thread each; a warp then takes a queued candidate with its lanes spread over the entries,
          // so that the loads of one candidate are in flight together
          const int nfix = s.nfix;
          for (int e = tid; e < E; e += blockDim.x) s.fixrow[e] = 0;
          if (tid == 0) s.qn = 0;
          __syncthreads();
          if (tid < nfix) s.fixrow[s.fix_e[tid]] = 1;
          __syncthreads();
          for (int c0 = 0; c0 < n; c0 += blockDim.x) {
            const int c = c0 + tid;
            bool any = false;
            if (c < n)
              for (int j = 0; j < k; ++j) any |= (s.fixrow[held_s[c * kMaxK + j]] != 0);
            const unsigned mask = __ballot_sync(0xffffffffu, any);
            int base = 0;
            if (lane == 0 && mask) base = atomicAdd(&s.qn, __popc(mask));
            base = __shfl_sync(0xffffffffu, base, 0);
            if (any) queue_s[base + __popc(mask & ((1u << lane) - 1u))] = c;
          }
          __syncthreads();
          const int qn = s.qn;
          for (int qi = warp; qi < qn; qi += kP2Threads / 32) {
            const int c = queue_s[qi];
            const int tok = cand_s[c];
            int h[kMaxK];
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) h[j] = j < k ? (int)held_s[c * kMaxK + j] : -1;
            const uint32_t flat = (uint32_t)tok * (uint32_t)E;
            for (int i = lane; i < nfix; i += 32) {
              const int e = s.fix_e[i], f = s.fix_f[i];
              bool he = false, hf = false;
#pragma unroll
              for (int j = 0; j < kMaxK; ++j) { he |= (h[j] == e); hf |= (h[j] == f); }
              if (!he || hf) continue;
              const long long cst = make_key(g, __ldg(M + (size_t)tok * E + e), flat + e) -
                                    make_key(g, __ldg(M + (size_t)tok * E + f), flat + f);
              if (cst - s.p[e] + s.p[f] <= arc_window && cst < D[e * ES + f]) atomicMin(&D[e * ES + f], cst);
            }
          }
          __syncthreads();
        } else if (s.nfix > 0) {
          // one thread per candidate (lists longer than the shared-memory mirror)
          for (int c = tid; c < n; c += blockDim.x) {
            const int tok = tok_of(c);
            int h[kMaxK];
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) h[j] = j < k ? held_of(c, tok, j) : -1;
            const uint32_t flat = (uint32_t)tok * (uint32_t)E;
            for (int i = 0; i < s.nfix; ++i) {
              const int e = s.fix_e[i], f = s.fix_f[i];
              bool he = false, hf = false;
#pragma unroll
              for (int j = 0; j < kMaxK; ++j) { he |= (h[j] == e); hf |= (h[j] == f); }
              if (!he || hf) continue;
              const long long cst = make_key(g, __ldg(M + (size_t)tok * E + e), flat + e) -
                                    make_key(g, __ldg(M + (size_t)tok * E + f), flat + f);
              if (cst - s.p[e] + s.p[f] <= arc_window && cst < D[e * ES + f]) atomicMin(&D[e * ES + f], cst);
            }
          }
          __syncthreads();
        }
    };
    bool batched = false;
    {
      const int L = s.npath - 1;
      long long ta = clock64();
      for (int a = tid; a <= L; a += blockDim.x) s.who_a[a] = 0x7fffffff;
      if (tid == 0) { s.dup = 0; s.nfix = 0; }
      __syncthreads();
      for (int c = tid; c < n; c += blockDim.x) {
        const int tok = tok_of(c);
        unsigned hm[4] = {0, 0, 0, 0};
        for (int j = 0; j < k; ++j) { const int e = held_of(c, tok, j); hm[e >> 5] |= 1u << (e & 31); }
        const uint32_t flat = (uint32_t)tok * (uint32_t)E;
        for (int a = L; a >= 1; --a) {
          const int u = s.path[a], v = s.path[a - 1];
          if (u >= E || v >= E) continue;
          if (!((hm[u >> 5] >> (u & 31)) & 1u) || ((hm[v >> 5] >> (v & 31)) & 1u)) continue;
          const long long cost = make_key(g, __ldg(M + (size_t)tok * E + u), flat + u) -
                                 make_key(g, __ldg(M + (size_t)tok * E + v), flat + v);
          if (cost == D[u * ES + v]) atomicMin(&s.who_a[a], c);    // sorted list: smallest c = smallest token
        }
      }
      __syncthreads();
      for (int idx = tid; idx < L * L; idx += blockDim.x) {
        const int i = idx / L + 1, j = idx - (i - 1) * L + 1;
        if (i < j && s.who_a[i] != 0x7fffffff && s.who_a[i] == s.who_a[j]) s.dup = 1;
      }
      __syncthreads();
      batched = !s.dup;
      { const long long tb = clock64(); t_who += tb - ta; ta = tb; }
      if (batched) {
        n_arcs += L;
        for (int a = L - warp; a >= 1; a -= kP2Threads / 32) {
          const int u = s.path[a], v = s.path[a - 1];
          if (u >= E || v >= E) continue;
          const int c = s.who_a[a];
          if (c == 0x7fffffff) { if (lane == 0) { atomicOr(&st->status, 4u); s.stop = 1; } continue; }
          const int tok = tok_of(c);
          int h[kMaxK];
#pragma unroll
          for (int j = 0; j < kMaxK; ++j) {
            h[j] = j < k ? held_of(c, tok, j) : -1;
            if (h[j] == u) h[j] = v;                   // experts after the move
          }
          const uint32_t flat = (uint32_t)tok * (uint32_t)E;
          long long key[kEPLf]; bool in[kEPLf];
#pragma unroll
          for (int q = 0; q < kEPLf; ++q) {
            const int f = lane + 32 * q;
            key[q] = f < E ? make_key(g, __ldg(M + (size_t)tok * E + f), flat + f) : 0;
            bool hd = f >= E;
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) hd |= (h[j] == f);
            in[q] = hd;
          }
          auto key_of = [&](int e) -> long long {
            long long mine = 0;
#pragma unroll
            for (int q = 0; q < kEPLf; ++q) if ((e >> 5) == q) mine = key[q];
            return __shfl_sync(0xffffffffu, mine, e & 31);
          };
          const long long ku = key_of(u), kv = key_of(v);
#pragma unroll
          for (int q = 0; q < kEPLf; ++q) {
            const int f = lane + 32 * q;
            if (!in[q]) {                               // row v gains the token
              const long long cst = kv - key[q];
              if (cst - s.p[v] + s.p[f] <= arc_window && cst < D[v * ES + f]) atomicMin(&D[v * ES + f], cst);
            }
            const bool was_out = f < E && f != u && (!in[q] || f == v);
            if (was_out && D[u * ES + f] == ku - key[q]) {      // the token's own offer from u is gone
              const int slot = atomicAdd(&s.nfix, 1);
              if (slot < kMaxFix) { s.fix_e[slot] = u; s.fix_f[slot] = f; }
            }
          }
#pragma unroll
          for (int j = 0; j < kMaxK; ++j) {
            if (j >= k || h[j] == v) continue;
            const int gg = h[j];
            const long long kg = key_of(gg);
            if (lane == 0) {
              if (kg - ku - s.p[gg] + s.p[u] <= arc_window && kg - ku < D[gg * ES + u]) atomicMin(&D[gg * ES + u], kg - ku);
              if (D[gg * ES + v] == kg - kv) {
                const int slot = atomicAdd(&s.nfix, 1);
                if (slot < kMaxFix) { s.fix_e[slot] = gg; s.fix_f[slot] = v; }
              }
            }
          }
          __syncwarp();
          if (lane == 0)
            for (int j = 0; j < k; ++j)
              if (held_of(c, tok, j) == u) {
                if (c < nc) held_s[c * kMaxK + j] = (unsigned char)v;
                expert_idx[(size_t)tok * k + j] = v;
              }
        }
        if (tid == 0)
          for (int a = L; a >= 1; --a) {
            const int u = s.path[a], v = s.path[a - 1];
            if (u < E && v < E) continue;
            if (v == nZ) s.flow[u] += 1; else s.flow[v] -= 1;
          }
        __syncthreads();
        if (s.nfix > kMaxFix) {
          // too many stale entries: rebuild the rows they sit in.  The tokens have moved already, so a
          // token's other experts are what it holds now, minus the arc's target
          for (int a = L - warp; a >= 1; a -= kP2Threads / 32) {
            const int u = s.path[a], v = s.path[a - 1];
            if (u >= E || v >= E || lane != 0) continue;
            const int c = s.who_a[a];
            if (c == 0x7fffffff) continue;
            const int tok = tok_of(c);
            s.dirty[u] = 1;
            for (int j = 0; j < k; ++j) { const int e = held_of(c, tok, j); if (e != v) s.dirty[e] = 1; }
          }
          __syncthreads();
          if (tid == 0) s.nfix = 0;
        } else {
          for (int i = tid; i < s.nfix; i += blockDim.x) D[s.fix_e[i] * ES + s.fix_f[i]] = kInf;
        }
        __syncthreads();
        { const long long tb = clock64(); t_patch += tb - ta; ta = tb; }
        fix_pass();
        t_fix += clock64() - ta;
      }
    }
    if (!batched)
    for (int a = s.npath - 1; a >= 1; --a) {
      const int u = s.path[a], v = s.path[a - 1];
      if (u < E && v < E) {
        long long ta = clock64(); ++n_arcs;
        if (tid == 0) s.who = 0x7fffffff;
        __syncthreads();
        const long long want = D[u * ES + v];
        for (int c = tid; c < n; c += blockDim.x) {
          const int tok = tok_of(c);
          bool hu = false, hv = false;
          for (int j = 0; j < k; ++j) {
            const int e = held_of(c, tok, j);
            hu |= (e == u); hv |= (e == v);
          }
          if (!hu || hv) continue;
          const uint32_t flat = (uint32_t)tok * (uint32_t)E;
          const long long cost = make_key(g, __ldg(M + (size_t)tok * E + u), flat + u) -
                                 make_key(g, __ldg(M + (size_t)tok * E + v), flat + v);
          if (cost == want) atomicMin(&s.who, c);      // the list is sorted: smallest c = smallest token
        }
        __syncthreads();
        if (s.who == 0x7fffffff) {   // internal inconsistency: stop, the verify pass will report it
          if (tid == 0) { atomicOr(&st->status, 4u); s.stop = 1; }
          __syncthreads();
          break;
        }
        { const long long tb = clock64(); t_who += tb - ta; ta = tb; }
        if (warp == 0) {
          // the token leaves u for v: patch D from its own keys instead of rebuilding every row it touches
          const int c = s.who, tok = tok_of(c);
          int h[kMaxK];
#pragma unroll
          for (int j = 0; j < kMaxK; ++j) {
            h[j] = j < k ? held_of(c, tok, j) : -1;
            if (h[j] == u) h[j] = v;                   // experts after the move
          }
          const uint32_t flat = (uint32_t)tok * (uint32_t)E;
          long long key[kEPLf]; bool in[kEPLf];
#pragma unroll
          for (int q = 0; q < kEPLf; ++q) {
            const int f = lane + 32 * q;
            key[q] = f < E ? make_key(g, __ldg(M + (size_t)tok * E + f), flat + f) : 0;
            bool hd = f >= E;
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) hd |= (h[j] == f);
            in[q] = hd;
          }
          auto key_of = [&](int e) -> long long {
            long long mine = 0;
#pragma unroll
            for (int q = 0; q < kEPLf; ++q) if ((e >> 5) == q) mine = key[q];
            return __shfl_sync(0xffffffffu, mine, e & 31);
          };
          const long long ku = key_of(u), kv = key_of(v);
          // row v gains the token: new moves v -> f for every expert f it does not hold
#pragma unroll
          for (int q = 0; q < kEPLf; ++q) {
            const int f = lane + 32 * q;
            if (!in[q]) {
              const long long cst = kv - key[q];
              if (cst - s.p[v] + s.p[f] <= arc_window && cst < D[v * ES + f]) D[v * ES + f] = cst;
            }
          }
          // D entries whose cheapest move was this token's become stale: (u, f) for the experts f it
          // offered from u, and (g, v) for its other experts g.  They are listed and recomputed below
          // from the candidates that hold the row's expert; a full row rebuild is the fallback.
          if (lane == 0) s.nfix = 0;
          __syncwarp();
#pragma unroll
          for (int q = 0; q < kEPLf; ++q) {
            const int f = lane + 32 * q;
            // before the move the token held u and not f (f != v is covered by in[], v itself is the used arc)
            const bool was_out = f < E && f != u && (!in[q] || f == v);
            if (was_out && D[u * ES + f] == ku - key[q]) {
              const int slot = atomicAdd(&s.nfix, 1);
              if (slot < kMaxFix) { s.fix_e[slot] = u; s.fix_f[slot] = f; }
            }
          }
#pragma unroll
          for (int j = 0; j < kMaxK; ++j) {
            if (j >= k || h[j] == v) continue;
            const int gg = h[j];
            const long long kg = key_of(gg);
            if (lane == 0) {
              if (kg - ku - s.p[gg] + s.p[u] <= arc_window && kg - ku < D[gg * ES + u]) D[gg * ES + u] = kg - ku;   // g -> u is a new move
              if (D[gg * ES + v] == kg - kv) {                            // g -> v is gone
                const int slot = atomicAdd(&s.nfix, 1);
                if (slot < kMaxFix) { s.fix_e[slot] = gg; s.fix_f[slot] = v; }
              }
            }
          }
          __syncwarp();
          if (lane == 0) {
            if (s.nfix > kMaxFix) {                    // too many: rebuild the rows instead
              s.dirty[u] = 1;
              for (int j = 0; j < k; ++j) if (h[j] != v) s.dirty[h[j]] = 1;
              s.nfix = 0;
            }
            for (int j = 0; j < k; ++j) {
              const int e = held_of(c, tok, j);
              if (e == u) {
                if (c < nc) held_s[c * kMaxK + j] = (unsigned char)v;
                expert_idx[(size_t)tok * k + j] = v;
              }
            }
          }
          __syncwarp();
          for (int i = lane; i < s.nfix; i += 32) D[s.fix_e[i] * ES + s.fix_f[i]] = kInf;
        }
        __syncthreads();
        { const long long tb = clock64(); t_patch += tb - ta; ta = tb; }
        fix_pass();
        t_fix += clock64() - ta;
      } else if (tid == 0) {
        if (v == nZ) s.flow[u] += 1; else s.flow[v] -= 1;
      }
    }
    if (s.stop) break;
    if (tid == 0) { s.imb[s.path[s.npath - 1]] -= 1; s.imb[s.target] += 1; }
    ++naug;
    __syncthreads();
    { const long long t1 = clock64(); t_move += t1 - t0; t0 = t1; }
  }
  // ---- write back ---------------------------------------------------------------------------------
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) {
    long long pe = s.p[e] - s.p[nZ];
    st->p[e] = pe < 0 ? 0 : pe;     // only an expert that holds nothing can come out negative
  }
  if (tid == 0) {
    st->naug += naug; st->ncand_last = n; st->ncand = 0;
    st->trace[44] = (int)(t_rebuild >> 10); st->trace[45] = (int)(t_bf >> 10); st->trace[46] = (int)(t_move >> 10); st->trace[47] = bf_rounds; st->trace[41] = (int)q_total; st->trace[42] = (int)(t_first >> 10);   // kilo-cycles
    st->trace[34] = (int)(t_who >> 10); st->trace[35] = (int)(t_patch >> 10); st->trace[36] = (int)(t_fix >> 10); st->trace[37] = n_arcs;
  }
}

}  // namespace msr
