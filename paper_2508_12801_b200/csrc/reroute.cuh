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
// Stage 1 needs no sequential pass: with cnt[r][e] tokens choosing e at level r, the expert starts level r
// with base[r][e] = min(C, base[r-1][e] + cnt[r-1][e]) tokens and accepts the first C - base[r][e] of them
// in token order, so a pair is accepted iff base + (its rank among that level's choosers) < C.  The ranks
// come from the index-build kernels.  Stage 2 is sequential by definition (every placement changes what the
// next pair may take); it runs in one CTA that stages the rows, held masks and dropped bits of the next 64 dropped
// tokens in shared memory, after which one warp places them without touching global memory.
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

// base[r][e] = tokens expert e holds when level r starts (base[k] = its load after stage 1).
__global__ void reroute_base_kernel(const int32_t* __restrict__ cnt, int32_t* __restrict__ base, int E, int k, int C) {
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int b = 0;
    for (int r = 0; r <= k; ++r) {
      base[r * E + e] = b;
      if (r < k) b = min(C, b + cnt[r * E + e]);
    }
  }
}

// Stage 1 acceptance: held mask (128 bits) and dropped-level bits of every token.
__global__ void __launch_bounds__(256)
reroute_accept_kernel(const int32_t* __restrict__ choice, const int32_t* __restrict__ rank, const int32_t* __restrict__ base,
                      uint4* __restrict__ held, unsigned char* __restrict__ dropped, int32_t* __restrict__ counts,
                      int T, int E, int k, int C) {
  int ndrop = 0;
  for (int tok = blockIdx.x * blockDim.x + threadIdx.x; tok < T; tok += gridDim.x * blockDim.x) {
    unsigned hm[4] = {0, 0, 0, 0}; unsigned db = 0;
    for (int r = 0; r < k; ++r) {
      const int e = choice[(size_t)r * T + tok];
      if (base[r * E + e] + rank[(size_t)r * T + tok] < C) hm[e >> 5] |= 1u << (e & 31);
      else { db |= 1u << r; ++ndrop; }
    }
    held[tok] = make_uint4(hm[0], hm[1], hm[2], hm[3]);
    dropped[tok] = (unsigned char)db;
  }
  if (ndrop) atomicAdd(&counts[0], ndrop);
}

constexpr int kRerouteThreads = 1024, kRerouteBatch = 64;
struct RerouteShared {
  int load[kMaxE];
  int list[kRerouteThreads];       // tokens of the chunk that have a dropped pair, in token order
  int nlist, nempty;
  int wcount[kRerouteThreads / 32];
  float rows[kRerouteBatch][kMaxE];
  uint4 hrow[kRerouteBatch];       // held masks and dropped-level bits of the staged tokens
  unsigned drow[kRerouteBatch];
};

// Stage 2, one CTA.  Tokens are scanned in chunks of kRerouteThreads; the chunk's tokens with a dropped pair are
// listed in order (ballot + scan), their score rows are staged in shared memory kRerouteBatch at a time by all
// warps, and warp 0 places the pairs one after the other (lanes over experts, one arg-max per pair).
__global__ void __launch_bounds__(kRerouteThreads)
reroute_place_kernel(const float* __restrict__ A, const int32_t* __restrict__ base, uint4* __restrict__ held,
                     const unsigned char* __restrict__ dropped, int32_t* __restrict__ expert_load,
                     int32_t* __restrict__ counts, int T, int E, int k, int C) {
  extern __shared__ __align__(16) unsigned char reroute_smem[];
  RerouteShared& s = *reinterpret_cast<RerouteShared*>(reroute_smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < E; e += blockDim.x) s.load[e] = base[k * E + e];
  if (tid == 0) s.nempty = 0;
  __syncthreads();
  for (int chunk = 0; chunk < T; chunk += kRerouteThreads) {
    const int tok = chunk + tid;
    const bool has = tok < T && dropped[tok] != 0;
    const unsigned bal = __ballot_sync(0xffffffffu, has);
    if (lane == 0) s.wcount[warp] = __popc(bal);
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int w = 0; w < kRerouteThreads / 32; ++w) { const int c = s.wcount[w]; s.wcount[w] = run; run += c; }
      s.nlist = run;
    }
    __syncthreads();
    if (has) s.list[s.wcount[warp] + __popc(bal & ((1u << lane) - 1u))] = tok;
    __syncthreads();
    const int nlist = s.nlist;
    for (int b0 = 0; b0 < nlist; b0 += kRerouteBatch) {
      const int nb = min(kRerouteBatch, nlist - b0);
      for (int i = tid; i < nb * E; i += blockDim.x) {
        const int q = i / E, e = i - q * E;
        s.rows[q][e] = __ldg(A + (size_t)s.list[b0 + q] * E + e);
      }
      if (tid < nb) { s.hrow[tid] = held[s.list[b0 + tid]]; s.drow[tid] = dropped[s.list[b0 + tid]]; }
      __syncthreads();
      if (warp == 0) {
        for (int q = 0; q < nb; ++q) {
          const int t2 = s.list[b0 + q];
          const uint4 hv = s.hrow[q];
          unsigned hm[4] = {hv.x, hv.y, hv.z, hv.w};
          const unsigned db = s.drow[q];
          for (int r = 0; r < k; ++r) {
            if (!((db >> r) & 1u)) continue;
            float best = -INFINITY; int bidx = 0x7fffffff;
#pragma unroll
            for (int j = 0; j < kEPL; ++j) {
              const int e = lane + 32 * j;
              if (e < E && s.load[e] < C && !((hm[j] >> lane) & 1u)) {
                const float v = s.rows[q][e];
                if (v > best || bidx == 0x7fffffff) { best = v; bidx = e; }
              }
            }
            const unsigned anyone = __ballot_sync(0xffffffffu, bidx != 0x7fffffff);
            if (!anyone) { if (lane == 0) s.nempty += 1; continue; }
            if (bidx == 0x7fffffff) best = -INFINITY;
            warp_argmax(best, bidx);
            // lanes without a candidate carried -inf and the sentinel index: a real candidate always wins, and
            // among equal affinities the lowest expert index
            hm[bidx >> 5] |= 1u << (bidx & 31);
            if (lane == 0) s.load[bidx] += 1;
            __syncwarp();
          }
          if (lane == 0) held[t2] = make_uint4(hm[0], hm[1], hm[2], hm[3]);
        }
      }
      __syncthreads();
    }
  }
  for (int e = tid; e < E; e += blockDim.x) expert_load[e] = s.load[e];
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
