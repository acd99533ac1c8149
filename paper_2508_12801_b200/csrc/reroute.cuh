// Iterative rerouting (Sec. 2.3, the Switch Transformers paragraph; the assignment step of "MaxScore-I",
// Sec. 4.1): top-k with capacity, then the dropped pairs are greedily given to the best expert that still
// has room.  The paper calls it the speed end of the quality/speed trade-off for k > 2 (Sec. 3.2).
//
// Orders (the paper fixes none; these are the library's reading, the same as the CPU checker's):
//   stage 1  choice level 1 of every token is served before level 2, ...; within a level tokens in
//            ascending index; a pair is accepted while its expert holds fewer than C tokens;
//   stage 2  dropped pairs in ascending token index, within a token in level order; each goes to the
//            expert of highest affinity among those with room that the token does not hold (ties: lowest
//            index), or stays empty if there is none.
// Stage 1 needs no sequential pass: a pair is accepted iff fewer than C pairs of the same expert come before
// it in level-major order, and that rank is what the index-build kernels compute when they are handed the
// level-major choice array as k*T "tokens" with one expert each.
// Stage 2 is sequential by definition (every placement changes what the next token may take), but what a token
// takes depends on the earlier ones only through the set of experts that still have room, and that set changes
// at most E times.  So one CTA places up to 1024 tokens at a time speculatively: every token proposes to the
// first experts of its candidate list that have room now, the proposals to an expert are ranked in token order,
// and the first token whose proposal finds its expert used up by earlier proposals marks the end of the prefix
// that is final.  Everything before it is placed, the expert that ran out is closed, and the next round starts
// at that token.  A round therefore places everything up to the next expert that fills up.
// A token's candidate order holds every expert that it does not hold and that has room after stage 1, by descending
// affinity (ties by ascending index), a byte each; it is made once, by one warp per listed token across the whole GPU,
// and a thread reads its token's order 16 experts at a time as far as it has to.
#pragma once
#include "common.cuh"
#include "softtopk.cuh"

namespace msr {

// Every token's k choices in level order: choice[r * T + tok].
__global__ void __launch_bounds__(256)
reroute_choices_kernel(const float* __restrict__ A, int32_t* __restrict__ choice, int T, int E, int k) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = A + (size_t)tok * E;
    float a[kEPL]; bool live[kEPL];
#pragma unroll
    for (int j = 0; j < kEPL; ++j) { const int e = lane + 32 * j; live[j] = e < E; a[j] = live[j] ? __ldg(row + e) : 0.f; }
    for (int r = 0; r < k; ++r) {
      float best = -INFINITY; int bidx = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < kEPL; ++j)
        if (live[j] && (a[j] > best || bidx == 0x7fffffff)) { best = a[j]; bidx = lane + 32 * j; }
      warp_argmax(best, bidx);
#pragma unroll
      for (int j = 0; j < kEPL; ++j) if (lane + 32 * j == bidx) live[j] = false;
      if (lane == 0) choice[(size_t)r * T + tok] = bidx;
    }
  }
}

// Stage 1 acceptance from the level-major ranks: held mask (128 bits) and dropped-level bits of every token,
// and per block of 256 tokens how many of them have a dropped pair (for the ordered list of such tokens).
constexpr int kRrTokBlock = 256;
__global__ void __launch_bounds__(kRrTokBlock)
reroute_accept_kernel(const int32_t* __restrict__ choice, const int32_t* __restrict__ rank, uint4* __restrict__ held,
                      unsigned char* __restrict__ dropped, int32_t* __restrict__ blk_cnt, int32_t* __restrict__ counts,
                      int T, int E, int k, int C) {
  const int tok = blockIdx.x * kRrTokBlock + threadIdx.x;
  unsigned db = 0;
  if (tok < T) {
    unsigned hm[4] = {0, 0, 0, 0};
    for (int r = 0; r < k; ++r) {
      const int e = choice[(size_t)r * T + tok];
      if (rank[(size_t)r * T + tok] < C) hm[e >> 5] |= 1u << (e & 31);
      else db |= 1u << r;
    }
    held[tok] = make_uint4(hm[0], hm[1], hm[2], hm[3]);
    dropped[tok] = (unsigned char)db;
  }
  const int has = __syncthreads_count(db != 0);
  if (threadIdx.x == 0) blk_cnt[blockIdx.x] = has;
  int nd = __popc(db);
#pragma unroll
  for (int d = 16; d; d >>= 1) nd += __shfl_xor_sync(0xffffffffu, nd, d);
  if ((threadIdx.x & 31) == 0 && nd) atomicAdd(&counts[0], nd);
}

// Exclusive scan of the block counts (one CTA): blk_off[b] = tokens with a dropped pair in the blocks before b,
// blk_off[nblk] = their total.
__global__ void __launch_bounds__(1024)
reroute_scan_kernel(const int32_t* __restrict__ blk_cnt, int32_t* __restrict__ blk_off, int nblk) {
  __shared__ int wsum[32];
  __shared__ int s_total;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int carry = 0;
  for (int base = 0; base < nblk; base += 1024) {
    const int i = base + tid;
    const int v = i < nblk ? blk_cnt[i] : 0;
    int x = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, d); if (lane >= d) x += y; }
    if (lane == 31) wsum[warp] = x;
    __syncthreads();
    if (warp == 0) {
      const int w = wsum[lane];
      int xs = w;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) { const int y = __shfl_up_sync(0xffffffffu, xs, d); if (lane >= d) xs += y; }
      wsum[lane] = xs - w;
      if (lane == 31) s_total = xs;
    }
    __syncthreads();
    if (i < nblk) blk_off[i] = carry + wsum[warp] + x - v;
    carry += s_total;
    __syncthreads();
  }
  if (tid == 0) blk_off[nblk] = carry;
}

constexpr int kRrChunk = 16;               // experts of a token's order that a thread holds at a time
constexpr int kRrRow = kMaxE;              // bytes per row of the order array

__device__ __forceinline__ bool rr_bit(const unsigned (&w)[4], int e) {
  const unsigned x = (e & 64) ? ((e & 32) ? w[3] : w[2]) : ((e & 32) ? w[1] : w[0]);
  return (x >> (e & 31)) & 1u;
}
__device__ __forceinline__ unsigned rr_byte(const unsigned (&w)[4], int j) {
  const unsigned x = (j & 8) ? ((j & 4) ? w[3] : w[2]) : ((j & 4) ? w[1] : w[0]);
  return (x >> (8 * (j & 3))) & 255u;
}

// Position of the n-th set bit of x (n counts from 1; x has at least n bits set).
__device__ __forceinline__ int rr_nth_bit(unsigned x, int n) {
  int pos = 0;
#pragma unroll
  for (int h = 16; h; h >>= 1) {
    const int c = __popc(x & ((1u << h) - 1u));
    if (n > c) { n -= c; pos += h; x >>= h; }
  }
  return pos;
}

// The tokens with a dropped pair, in token order (dtok), with their number of dropped pairs (dnum).
__global__ void __launch_bounds__(kRrTokBlock)
reroute_compact_kernel(const unsigned char* __restrict__ dropped, const int32_t* __restrict__ blk_off,
                       int32_t* __restrict__ dtok, unsigned char* __restrict__ dnum, int T) {
  __shared__ int wbase[kRrTokBlock / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int off = blk_off[blockIdx.x];
  if (blk_off[blockIdx.x + 1] == off) return;
  const int tok = blockIdx.x * kRrTokBlock + tid;
  const unsigned db = tok < T ? dropped[tok] : 0u;
  const unsigned bal = __ballot_sync(0xffffffffu, db != 0);
  if (lane == 0) wbase[warp] = __popc(bal);
  __syncthreads();
  int before = 0;
#pragma unroll
  for (int w = 0; w < kRrTokBlock / 32; ++w) before += w < warp ? wbase[w] : 0;
  if (db) {
    const int pos = off + before + __popc(bal & ((1u << lane) - 1u));
    dtok[pos] = tok; dnum[pos] = (unsigned char)__popc(db);
  }
}

// Every listed token's candidates (one warp per token): the experts that have room after stage 1 and that the token
// does not hold, by descending affinity, ties by ascending index, a byte each, kRrNone after the last.  A
// candidate's place is the number of candidates that come before it, counted against all of them.
constexpr unsigned kRrNone = 255u;
__global__ void __launch_bounds__(256)
reroute_order_kernel(const float* __restrict__ A, const int32_t* __restrict__ total, const uint4* __restrict__ held,
                     const int32_t* __restrict__ nd_ptr, const int32_t* __restrict__ dtok,
                     unsigned char* __restrict__ order, int E, int C) {
  __shared__ unsigned openw[4];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (warp < 4) {
    const unsigned ob = __ballot_sync(0xffffffffu, (int)threadIdx.x < E && total[threadIdx.x] < C);
    if (lane == 0) openw[warp] = ob;
  }
  __syncthreads();
  const int nd = *nd_ptr;
  for (int q = blockIdx.x * 8 + warp; q < nd; q += gridDim.x * 8) {
    const int t = dtok[q];
    const float* row = A + (size_t)t * E;
    const uint4 hv = held[t];
    const unsigned hw[4] = {hv.x, hv.y, hv.z, hv.w};
    float a[kEPL]; int place[kEPL]; bool cand[kEPL];
    int ncand = 0;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      const int e = lane + 32 * j;
      cand[j] = e < E && ((openw[j] >> lane) & 1u) && !((hw[j] >> lane) & 1u);
      a[j] = cand[j] ? __ldg(row + e) : 0.f;
      place[j] = 0;
      ncand += __popc(__ballot_sync(0xffffffffu, cand[j]));
    }
#pragma unroll
    for (int j2 = 0; j2 < kEPL; ++j2) {
      if (32 * j2 >= E) break;
      const unsigned there = __ballot_sync(0xffffffffu, cand[j2]);
      for (unsigned rest = there; rest; rest &= rest - 1) {
        const int src = __ffs(rest) - 1;
        const float o = __shfl_sync(0xffffffffu, a[j2], src);
        const int oe = src + 32 * j2;
#pragma unroll
        for (int j = 0; j < kEPL; ++j) place[j] += (o > a[j] || (o == a[j] && oe < lane + 32 * j)) ? 1 : 0;
      }
    }
    unsigned char* out = order + (size_t)q * kRrRow;
#pragma unroll
    for (int j = 0; j < kEPL; ++j)
      if (cand[j]) out[min(place[j], kRrRow - 1)] = (unsigned char)(lane + 32 * j);
    for (int p = ncand + lane; p < kRrRow; p += 32) out[p] = (unsigned char)kRrNone;
  }
}

constexpr int kRrThreads = 1024;          // tokens of one speculative block
struct RerouteShared {
  unsigned mask[kRrThreads / 32][kMaxE + 1];   // lanes of a warp that propose to the expert
  int resid[kMaxE];                       // room left
  unsigned openw[4];
  int qstar, nempty;
};

// Stage 2, one CTA (see the head of this file).  Thread i owns the i-th listed token of the current block of
// kRrThreads tokens until the whole block is placed: its held mask, its picks, the 16 experts of its order it is
// reading and how far it has read stay in registers from round to round.
__global__ void __launch_bounds__(kRrThreads)
reroute_place_kernel(const int32_t* __restrict__ total, uint4* __restrict__ held, const int32_t* __restrict__ nd_ptr,
                     const int32_t* __restrict__ dtok, const unsigned char* __restrict__ dnum,
                     const unsigned char* __restrict__ order, int32_t* __restrict__ expert_load,
                     int32_t* __restrict__ counts, int E, int C) {
  __shared__ RerouteShared s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < kMaxE) {
    const int r = tid < E ? C - min(C, total[tid]) : 0;
    s.resid[tid] = r;
    const unsigned ob = __ballot_sync(0xffffffffu, r > 0);
    if (lane == 0) s.openw[warp] = ob;
  }
  if (tid == 0) { s.nempty = 0; s.qstar = 0x7fffffff; }
  const int nd = *nd_ptr;
  int my_empty = 0;
  __syncthreads();
  for (int qb = 0; qb < nd; qb += kRrThreads) {
    const int nb = min(kRrThreads, nd - qb);
    const bool active = tid < nb;
    unsigned lw[4] = {0, 0, 0, 0};
    unsigned long long picks = 0;                  // the experts proposed to, a byte each
    int m = 0, np = 0, cur = 0, t = 0;             // cur: entries of the order read so far
    const uint4* myrow = reinterpret_cast<const uint4*>(order + (size_t)(qb + tid) * kRrRow);
    if (active) {
      t = dtok[qb + tid];
      m = dnum[qb + tid];
    }
    int q0 = 0;                                    // tokens of the block before q0 are placed
    while (q0 < nb) {
      for (int e = lane; e < kMaxE; e += 32) s.mask[warp][e] = 0u;     // a warp's row is written by that warp alone
      __syncwarp();
      const unsigned open[4] = {s.openw[0], s.openw[1], s.openw[2], s.openw[3]};
      const bool live = active && tid >= q0;
      if (live) {
        // picks whose expert has filled up meanwhile are given back; the order is read on from where it was left
        // (what was skipped before had no room then and has none now)
        for (int i = 0; i < np;) {
          const int e = (int)((picks >> (8 * i)) & 255u);
          if (rr_bit(open, e)) { ++i; continue; }
          --np;
          const unsigned long long last = (picks >> (8 * np)) & 255u;
          picks = (picks & ~(255ull << (8 * i))) | (last << (8 * i));
        }
        while (np < m && cur < E) {
          if ((cur & (kRrChunk - 1)) == 0) {
            const uint4 lv = __ldg(myrow + cur / kRrChunk);
            lw[0] = lv.x; lw[1] = lv.y; lw[2] = lv.z; lw[3] = lv.w;
          }
          const int e = (int)rr_byte(lw, cur & (kRrChunk - 1));
          ++cur;
          if (e >= E) { cur = E; break; }            // past the last candidate
          if (rr_bit(open, e)) {
            picks = (picks & ~(255ull << (8 * np))) | ((unsigned long long)e << (8 * np));
            ++np;
          }
        }
        for (int i = 0; i < np; ++i) atomicOr(&s.mask[warp][(picks >> (8 * i)) & 255u], 1u << lane);
      }
      __syncthreads();
      unsigned mw[kRrThreads / 32];
      if (tid < kMaxE) {  // the first proposal, in token order, that finds expert tid used up by the ones before it
#pragma unroll
        for (int w = 0; w < kRrThreads / 32; ++w) mw[w] = s.mask[w][tid];      // rows of placed warps are empty
        const int room = s.resid[tid];
        int cum = 0, wsel = -1, nth = 0; unsigned msel = 0;
#pragma unroll
        for (int w = 0; w < kRrThreads / 32; ++w) {
          const int c = __popc(mw[w]);
          if (wsel < 0 && cum + c > room) { wsel = w; msel = mw[w]; nth = room - cum + 1; }
          cum += c;
        }
        if (wsel >= 0) atomicMin(&s.qstar, 32 * wsel + rr_nth_bit(msel, nth));
      }
      __syncthreads();
      const int qe = min(s.qstar, nb);              // the first token that has to think again
      if (live && tid < qe) my_empty += m - np;     // placed: its picks stay until the block is written back
      if (tid < kMaxE) {
        int taken = 0;
        const int wq = qe >> 5;
#pragma unroll
        for (int w = 0; w < kRrThreads / 32; ++w) {
          const unsigned part = w < wq ? 0xffffffffu : (w == wq ? (1u << (qe & 31)) - 1u : 0u);
          taken += __popc(mw[w] & part);
        }
        const int r = s.resid[tid] - taken;
        s.resid[tid] = r;
        const unsigned ob = __ballot_sync(0xffffffffu, r > 0);
        if (lane == 0) s.openw[warp] = ob;
      }
      q0 = qe;
      __syncthreads();
      if (tid == 0) s.qstar = 0x7fffffff;
    }
    if (active && np) {                             // the block's placements into the held masks
      const uint4 hv = held[t];
      unsigned hm[4] = {hv.x, hv.y, hv.z, hv.w};
      for (int i = 0; i < np; ++i) {
        const unsigned e = (unsigned)((picks >> (8 * i)) & 255u);
#pragma unroll
        for (int w = 0; w < 4; ++w) if ((int)(e >> 5) == w) hm[w] |= 1u << (e & 31u);
      }
      held[t] = make_uint4(hm[0], hm[1], hm[2], hm[3]);
    }
  }
  if (my_empty) atomicAdd(&s.nempty, my_empty);
  __syncthreads();
  for (int e = tid; e < E; e += kRrThreads) expert_load[e] = C - s.resid[e];
  if (tid == 0) counts[1] = s.nempty;
}

// The held masks as rows of expert_idx: ascending expert index, empty slots (-1) last.
__global__ void __launch_bounds__(256)
reroute_write_kernel(const uint4* __restrict__ held, int32_t* __restrict__ expert_idx, int T, int k) {
  for (int tok = blockIdx.x * blockDim.x + threadIdx.x; tok < T; tok += gridDim.x * blockDim.x) {
    const uint4 hv = held[tok];
    const unsigned hm[4] = {hv.x, hv.y, hv.z, hv.w};
    int n = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      unsigned m = hm[w];
      while (m && n < k) { const int b = __ffs(m) - 1; m &= m - 1; expert_idx[(size_t)tok * k + n++] = 32 * w + b; }
    }
    while (n < k) expert_idx[(size_t)tok * k + n++] = -1;
  }
}

}  // namespace msr
