// Algorithm 1 (Sec. 3.2): maximum score routing for top-2 as the paper trains it: every token's best expert first,
// then Sinkhorn on what is left.  The steps follow the algorithm's numbering; what the paper leaves open (the
// regulariser and iteration count of Sinkhorn, how the real-valued plan becomes a binary P) is this library's
// reading, stated in include/maxscore.h.
//   top-1      warp per token: arg-max of the affinities (ties: lowest index), counts per expert     (steps 4, 6)
//   Sinkhorn   K_ij = exp((a_ij - m_i) / eps) over the pairs that are not masked; one launch per iteration:
//              a warp per token forms u_i = 1 / sum_j K_ij v_j and adds u_i K_ij into per-lane column sums;
//              the CTA's sums are merged in a fixed order and the last CTA turns them into
//              v_j = min(1, c_j / t_j)                                                                (steps 7-9)
//   rounding   warp per token: arg-max of K_ij v_j; the index-build kernels then rank the tokens of every expert in
//              token order and the first c_j keep their second expert.
// All floating point is fp64: the arg-max of the rounding is a discrete decision, and the CPU checker takes it in
// double precision as well.  Column sums are added in a fixed order (lane-local, then warps, then CTAs), so the
// result does not change from run to run.
#pragma once
#include "common.cuh"
#include "softtopk.cuh"

namespace msr {

__global__ void __launch_bounds__(256)
alg1_top1_kernel(const float* __restrict__ A, int32_t* __restrict__ first, int32_t* __restrict__ cnt, int T, int E) {
  __shared__ int scnt[kMaxE];
  for (int e = threadIdx.x; e < E; e += blockDim.x) scnt[e] = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = A + (size_t)tok * E;
    float best = -INFINITY; int bidx = 0x7fffffff;
    for (int e = lane; e < E; e += 32) {
      const float v = __ldg(row + e);
      if (v > best || bidx == 0x7fffffff) { best = v; bidx = e; }
    }
    warp_argmax(best, bidx);
    if (lane == 0) { first[tok] = bidx; atomicAdd(&scnt[bidx], 1); }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) if (scnt[e]) atomicAdd(&cnt[e], scnt[e]);
}

// residual capacities (step 6), the first column scaling, and the count of top-1 pairs beyond C
__global__ void alg1_resid_kernel(const int32_t* __restrict__ cnt, int32_t* __restrict__ resid, double* __restrict__ v,
                                  int32_t* __restrict__ counts, int E, int C) {
  __shared__ int over;
  if (threadIdx.x == 0) over = 0;
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const int r = C - cnt[e] > 0 ? C - cnt[e] : 0;
    resid[e] = r; v[e] = r > 0 ? 1.0 : 0.0;
    if (cnt[e] > C) atomicAdd(&over, cnt[e] - C);
  }
  __syncthreads();
  if (threadIdx.x == 0) counts[0] = over;
}

constexpr int kAlg1Blocks = 296, kAlg1Threads = 256;

// One Sinkhorn iteration: row scaling with the current v, column sums, new v.
__global__ void __launch_bounds__(kAlg1Threads)
alg1_sinkhorn_kernel(const float* __restrict__ A, const int32_t* __restrict__ first, const int32_t* __restrict__ resid,
                     double* __restrict__ v, double* __restrict__ partial, unsigned* __restrict__ ticket, int T, int E,
                     double inv_eps) {
  __shared__ double sv[kMaxE];
  __shared__ double wsum[kAlg1Threads / 32][kMaxE];
  __shared__ bool is_last;
  for (int e = threadIdx.x; e < E; e += blockDim.x) sv[e] = v[e];
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_per_block = blockDim.x >> 5;
  double col[kEPL];
#pragma unroll
  for (int q = 0; q < kEPL; ++q) col[q] = 0.0;
  for (int tok = blockIdx.x * warps_per_block + warp; tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = A + (size_t)tok * E;
    const int f = first[tok];
    double a[kEPL], m = -INFINITY;
#pragma unroll
    for (int q = 0; q < kEPL; ++q) {
      const int e = lane + 32 * q;
      a[q] = (e < E && e != f) ? (double)__ldg(row + e) : -INFINITY;
      m = fmax(m, a[q]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double K[kEPL], s = 0.0;
#pragma unroll
    for (int q = 0; q < kEPL; ++q) {
      const int e = lane + 32 * q;
      K[q] = (e < E && e != f) ? exp((a[q] - m) * inv_eps) : 0.0;
      s += e < E ? K[q] * sv[e] : 0.0;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const double u = s > 0.0 ? 1.0 / s : 0.0;
#pragma unroll
    for (int q = 0; q < kEPL; ++q) col[q] += u * K[q];
  }
#pragma unroll
  for (int q = 0; q < kEPL; ++q) { const int e = lane + 32 * q; if (e < E) wsum[warp][e] = col[q]; }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    double t = 0.0;
    for (int w = 0; w < kAlg1Threads / 32; ++w) t += wsum[w][e];      // fixed order
    partial[(size_t)blockIdx.x * E + e] = t;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    double t = 0.0;
    for (int b = 0; b < (int)gridDim.x; ++b) t += __ldcg(partial + (size_t)b * E + e);   // fixed order
    const int r = resid[e];
    v[e] = r <= 0 ? 0.0 : (t > (double)r ? (double)r / t : 1.0);
  }
  if (threadIdx.x == 0) *ticket = 0;
}

// Rounding: the token's best expert under the plan (its row scaling does not change the arg-max), and the plan row.
__global__ void __launch_bounds__(256)
alg1_round_kernel(const float* __restrict__ A, const int32_t* __restrict__ first, const double* __restrict__ v,
                  int32_t* __restrict__ second, double* __restrict__ plan, int T, int E, double inv_eps) {
  __shared__ double sv[kMaxE];
  for (int e = threadIdx.x; e < E; e += blockDim.x) sv[e] = v[e];
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = A + (size_t)tok * E;
    const int f = first[tok];
    double a[kEPL], m = -INFINITY;
#pragma unroll
    for (int q = 0; q < kEPL; ++q) {
      const int e = lane + 32 * q;
      a[q] = (e < E && e != f) ? (double)__ldg(row + e) : -INFINITY;
      m = fmax(m, a[q]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double p[kEPL], s = 0.0;
#pragma unroll
    for (int q = 0; q < kEPL; ++q) {
      const int e = lane + 32 * q;
      p[q] = (e < E && e != f) ? exp((a[q] - m) * inv_eps) * sv[e] : 0.0;
      s += p[q];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const double u = s > 0.0 ? 1.0 / s : 0.0;
    double best = 0.0; int bidx = 0x7fffffff;
#pragma unroll
    for (int q = 0; q < kEPL; ++q) {
      const int e = lane + 32 * q;
      p[q] *= u;
      if (e < E && plan) plan[(size_t)tok * E + e] = p[q];
      if (p[q] > best) { best = p[q]; bidx = e; }          // strictly larger: the lowest index keeps a tie
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
      if (ob > best || (ob == best && oi < bidx)) { best = ob; bidx = oi; }
    }
    if (lane == 0) second[tok] = best > 0.0 ? bidx : -1;
  }
}

// Keep the first resid[e] seconds of every expert (rank = position among the expert's seconds in token order),
// write the two experts of every token in ascending order (-1 = dropped, last), count loads and drops.
__global__ void __launch_bounds__(256)
alg1_finish_kernel(const int32_t* __restrict__ first, const int32_t* __restrict__ second, const int32_t* __restrict__ rank,
                   const int32_t* __restrict__ resid, int32_t* __restrict__ expert_idx, int32_t* __restrict__ expert_load,
                   int32_t* __restrict__ counts, int T, int E) {
  __shared__ int sload[kMaxE];
  __shared__ int sdrop;
  for (int e = threadIdx.x; e < E; e += blockDim.x) sload[e] = 0;
  if (threadIdx.x == 0) sdrop = 0;
  __syncthreads();
  for (int tok = blockIdx.x * blockDim.x + threadIdx.x; tok < T; tok += gridDim.x * blockDim.x) {
    const int f = first[tok];
    int s2 = second[tok];
    if (s2 >= 0 && rank[tok] >= resid[s2]) s2 = -1;
    if (s2 < 0) atomicAdd(&sdrop, 1); else atomicAdd(&sload[s2], 1);
    atomicAdd(&sload[f], 1);
    expert_idx[2 * (size_t)tok] = (s2 >= 0 && s2 < f) ? s2 : f;
    expert_idx[2 * (size_t)tok + 1] = (s2 >= 0 && s2 < f) ? f : s2;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) if (sload[e]) atomicAdd(&expert_load[e], sload[e]);
  if (threadIdx.x == 0 && sdrop) atomicAdd(&counts[1], sdrop);
}

}  // namespace msr
