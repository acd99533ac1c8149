// SoftTopk forward and backward (Eq. 6 and its derivative), one warp per token.
//
// Level j (1-based) of Eq. 6 adds a softmax with temperature t over the entries that are not among
// the j-1 largest (ties: lowest expert index).  A lane holds experts lane, lane+32, ... so every
// global access of a warp is one contiguous row segment, and each level costs two shuffle
// reductions (arg-max, sum).  The exponentials are taken once, relative to the row maximum: a level's
// softmax is z_i / (sum of z over its unmasked entries) whatever the reference point.  Only when a
// level's own maximum lies so far below the row maximum that z would leave the normal fp32 range are
// they recomputed relative to that level's maximum.
#pragma once
#include "common.cuh"

namespace msr {

constexpr int kEPL = kMaxE / 32;  // experts per lane

// arg-max over the warp of (value, index) pairs, lowest index on equal values: two integer warp
// reductions (the largest value through an order-preserving map to unsigned, then the lowest index
// among the lanes that hold it) instead of five shuffle rounds.  Adding +0.0 first turns -0.0 into +0.0,
// so the two zeros tie as they do in a floating-point comparison.
__device__ __forceinline__ void warp_argmax(float& v, int& idx) {
  const unsigned b = __float_as_uint(v + 0.f);
  const unsigned u = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  const unsigned best = __reduce_max_sync(0xffffffffu, u);
  idx = (int)__reduce_min_sync(0xffffffffu, u == best ? (unsigned)idx : 0x7fffffffu);
  v = __uint_as_float((best & 0x80000000u) ? (best & 0x7fffffffu) : ~best);
}

__global__ void __launch_bounds__(256)
softtopk_fwd_kernel(const float* __restrict__ logits, float* __restrict__ scores, int T, int E, int k,
                    float t) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T;
       tok += gridDim.x * warps_per_block) {
    const float* row = logits + (size_t)tok * E;
    float a[kEPL], y[kEPL];
    bool live[kEPL];
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      int e = lane + 32 * j;
      live[j] = e < E;
      a[j] = live[j] ? __ldg(row + e) : 0.f;
      y[j] = 0.f;
    }
    float z[kEPL];
    float ref = 0.f;                                  // reference point of the current z
    for (int level = 0; level < k; ++level) {
      float best = -INFINITY; int bidx = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < kEPL; ++j)
        if (live[j] && (a[j] > best || bidx == 0x7fffffff)) { best = a[j]; bidx = lane + 32 * j; }
      warp_argmax(best, bidx);
      if (level == 0 || (ref - best) > 60.f * t) {    // (re)base the exponentials on this level's maximum
        ref = best;
#pragma unroll
        for (int j = 0; j < kEPL; ++j) z[j] = live[j] ? expf((a[j] - ref) / t) : 0.f;
      }
      float zs = 0.f;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) zs += z[j];
      zs = warp_sum(zs);
      const float inv = 1.f / zs;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) {
        y[j] = fmaf(z[j], inv, y[j]);
        if (lane + 32 * j == bidx) { live[j] = false; z[j] = 0.f; }   // masked from the next level on
      }
    }
    float* out = scores + (size_t)tok * E;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      int e = lane + 32 * j;
      if (e < E) out[e] = y[j];
    }
  }
}

// dlogits = J^T g with g = the k gradients of the token's assigned experts plus, if given, a per-expert
// term shared by all tokens (the gradient of the auxiliary loss, Eq. 9).  The masks are constants.
//   da_l = (1/t) * sum_{levels j with l unmasked} q_l * (g_l - sum_i g_i q_i),  q = level-j softmax
__global__ void __launch_bounds__(256)
softtopk_bwd_kernel(const float* __restrict__ logits, const int32_t* __restrict__ expert_idx,
                    const float* __restrict__ dgate_w, const float* __restrict__ dscores_col,
                    float* __restrict__ dlogits, int T, int E, int k, float t) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T;
       tok += gridDim.x * warps_per_block) {
    const float* row = logits + (size_t)tok * E;
    float a[kEPL], g[kEPL], da[kEPL];
    bool live[kEPL];
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      int e = lane + 32 * j;
      live[j] = e < E;
      a[j] = live[j] ? __ldg(row + e) : 0.f;
      g[j] = (live[j] && dscores_col) ? __ldg(dscores_col + e) : 0.f; da[j] = 0.f;
    }
    for (int c = 0; c < k; ++c) {
      int e = __ldg(expert_idx + (size_t)tok * k + c);
      float gv = __ldg(dgate_w + (size_t)tok * k + c);
#pragma unroll
      for (int j = 0; j < kEPL; ++j)
        if (lane + 32 * j == e) g[j] += gv;
    }
    float z[kEPL];
    float ref = 0.f;
    const float inv_t = 1.f / t;
    for (int level = 0; level < k; ++level) {
      float best = -INFINITY; int bidx = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < kEPL; ++j)
        if (live[j] && (a[j] > best || bidx == 0x7fffffff)) { best = a[j]; bidx = lane + 32 * j; }
      warp_argmax(best, bidx);
      if (level == 0 || (ref - best) > 60.f * t) {
        ref = best;
#pragma unroll
        for (int j = 0; j < kEPL; ++j) z[j] = live[j] ? expf((a[j] - ref) / t) : 0.f;
      }
      float zs = 0.f, gz = 0.f;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) { zs += z[j]; gz += g[j] * z[j]; }
      zs = warp_sum(zs);
      gz = warp_sum(gz);
      const float inv = 1.f / zs;
      const float gq = gz * inv;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) {
        da[j] = fmaf(z[j] * inv, (g[j] - gq) * inv_t, da[j]);
        if (lane + 32 * j == bidx) { live[j] = false; z[j] = 0.f; }
      }
    }
    float* out = dlogits + (size_t)tok * E;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      int e = lane + 32 * j;
      if (e < E) out[e] = da[j];
    }
  }
}

// The literal readings of Eq. 6 ("rank-scaled softmax"): y_i = p_i * (beta + t * min(rank_i - delta, k)) with
// p = Softmax(a) over all experts and rank 1 = largest (ties: lowest index first).  Only the k + delta - 1
// largest entries have a count below k, so that many arg-max rounds give every entry its scale.  The same
// routine serves the backward pass, where the ranks are constants:
//   da_l = p_l * (g_l s_l - sum_i g_i s_i p_i),   s_i = beta + t * min(rank_i - delta, k).
template <bool kBackward>
__global__ void __launch_bounds__(256)
softtopk_rankscale_kernel(const float* __restrict__ logits, const int32_t* __restrict__ expert_idx,
                          const float* __restrict__ dgate_w, const float* __restrict__ dscores_col,
                          float* __restrict__ out, int T, int E, int k, float t, float beta, int delta) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = logits + (size_t)tok * E;
    float a[kEPL], sc[kEPL]; bool live[kEPL];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      const int e = lane + 32 * j;
      live[j] = e < E;
      a[j] = live[j] ? __ldg(row + e) : -INFINITY;
      mx = fmaxf(mx, a[j]);
      sc[j] = beta + t * (float)k;                      // every entry of rank >= k + delta
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float p[kEPL], zs = 0.f;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) { p[j] = live[j] ? expf(a[j] - mx) : 0.f; zs += p[j]; }
    zs = warp_sum(zs);
    const float inv = 1.f / zs;
    for (int r = 1; r < k + delta && r <= E; ++r) {     // the entry of rank r
      float best = -INFINITY; int bidx = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < kEPL; ++j)
        if (live[j] && (a[j] > best || bidx == 0x7fffffff)) { best = a[j]; bidx = lane + 32 * j; }
      warp_argmax(best, bidx);
#pragma unroll
      for (int j = 0; j < kEPL; ++j)
        if (lane + 32 * j == bidx) { live[j] = false; sc[j] = beta + t * (float)(r - delta); }
    }
    float* o = out + (size_t)tok * E;
    if (!kBackward) {
#pragma unroll
      for (int j = 0; j < kEPL; ++j) { const int e = lane + 32 * j; if (e < E) o[e] = p[j] * inv * sc[j]; }
    } else {
      float g[kEPL];
#pragma unroll
      for (int j = 0; j < kEPL; ++j) {
        const int e = lane + 32 * j;
        g[j] = (e < E && dscores_col) ? __ldg(dscores_col + e) : 0.f;
      }
      for (int c = 0; c < k; ++c) {
        const int e = __ldg(expert_idx + (size_t)tok * k + c);
        const float gv = __ldg(dgate_w + (size_t)tok * k + c);
#pragma unroll
        for (int j = 0; j < kEPL; ++j) if (lane + 32 * j == e) g[j] += gv;
      }
      float dot = 0.f;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) dot += g[j] * sc[j] * p[j] * inv;
      dot = warp_sum(dot);
#pragma unroll
      for (int j = 0; j < kEPL; ++j) { const int e = lane + 32 * j; if (e < E) o[e] = p[j] * inv * (g[j] * sc[j] - dot); }
    }
  }
}

// IterTopk of Table 2: y^(0) = 0, y^(l) = y^(l-1) + g(x; 1 - y^(l-1)) with g(x; w) = w e^x / sum(w e^x), for
// l = 1..k.  One warp per token, a lane holds experts lane, lane+32, ...; a level is one weighted sum.  The
// backward pass (kBackward) keeps the weights of all k levels in registers and runs the recursion in reverse:
// with z = e^{x - max}, u = w z, s = sum u, r = u / s and rb the gradient of r,
//   ub = (rb - sum_i rb_i r_i) / s,   zb += ub w,   gradient of y^(l-1) = gradient of y^(l) - ub z,
// and dx = zb z at the end.  Table 2 has no temperature: the logits enter as they are.
template <bool kBackward>
__global__ void __launch_bounds__(256)
itertopk_kernel(const float* __restrict__ logits, const int32_t* __restrict__ expert_idx,
                const float* __restrict__ dgate_w, const float* __restrict__ dscores_col,
                float* __restrict__ out, int T, int E, int k) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = logits + (size_t)tok * E;
    float z[kEPL], w[kMaxK][kEPL], sl[kMaxK];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      const int e = lane + 32 * j;
      z[j] = e < E ? __ldg(row + e) : -INFINITY;
      mx = fmaxf(mx, z[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
#pragma unroll
    for (int j = 0; j < kEPL; ++j) z[j] = lane + 32 * j < E ? expf(z[j] - mx) : 0.f;
    float y[kEPL];
#pragma unroll
    for (int j = 0; j < kEPL; ++j) y[j] = 0.f;
#pragma unroll
    for (int l = 0; l < kMaxK; ++l) {
      if (l < k) {
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < kEPL; ++j) { w[l][j] = 1.f - y[j]; s += w[l][j] * z[j]; }
        s = warp_sum(s);
        sl[l] = s;
        const float inv = 1.f / s;
#pragma unroll
        for (int j = 0; j < kEPL; ++j) y[j] = fmaf(w[l][j] * z[j], inv, y[j]);
      }
    }
    float* o = out + (size_t)tok * E;
    if (!kBackward) {
#pragma unroll
      for (int j = 0; j < kEPL; ++j) { const int e = lane + 32 * j; if (e < E) o[e] = y[j]; }
    } else {
      float yb[kEPL], zb[kEPL];
#pragma unroll
      for (int j = 0; j < kEPL; ++j) {
        const int e = lane + 32 * j;
        yb[j] = (e < E && dscores_col) ? __ldg(dscores_col + e) : 0.f; zb[j] = 0.f;
      }
      for (int c = 0; c < k; ++c) {
        const int e = __ldg(expert_idx + (size_t)tok * k + c);
        const float gv = __ldg(dgate_w + (size_t)tok * k + c);
#pragma unroll
        for (int j = 0; j < kEPL; ++j) if (lane + 32 * j == e) yb[j] += gv;
      }
#pragma unroll
      for (int l = kMaxK - 1; l >= 0; --l) {
        if (l < k) {
          const float inv = 1.f / sl[l];
          float dot = 0.f;
#pragma unroll
          for (int j = 0; j < kEPL; ++j) dot += yb[j] * (w[l][j] * z[j] * inv);
          dot = warp_sum(dot);
#pragma unroll
          for (int j = 0; j < kEPL; ++j) {
            const float ub = (yb[j] - dot) * inv;
            zb[j] = fmaf(ub, w[l][j], zb[j]);
            yb[j] = fmaf(-ub, z[j], yb[j]);
          }
        }
      }
#pragma unroll
      for (int j = 0; j < kEPL; ++j) { const int e = lane + 32 * j; if (e < E) o[e] = zb[j] * z[j]; }
    }
  }
}

// Auxiliary load-balance loss, Eq. 9: L = lambda / (E T^2) * sum_j (sum_i A_ij) * load_j, and its
// gradient with respect to A (P is a constant): dL/dA_ij = lambda * load_j / (E T^2) for every token i.
// Column sums are taken by warps over rows (lane l owns columns l, l+32, ...) in double precision and
// merged with one atomic per column and CTA; the last CTA to finish forms the loss and clears the scratch.
__global__ void __launch_bounds__(256)
aux_loss_kernel(const float* __restrict__ scores, const int32_t* __restrict__ expert_load, double* colsum,
                unsigned* ticket, double* __restrict__ loss, float* __restrict__ dscores_col, int T, int E,
                float lambda) {
  __shared__ double ssum[kMaxE];
  __shared__ bool is_last;
  for (int e = threadIdx.x; e < E; e += blockDim.x) ssum[e] = 0.0;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  double acc[kEPL];
#pragma unroll
  for (int j = 0; j < kEPL; ++j) acc[j] = 0.0;
  for (int tok = blockIdx.x * warps_per_block + (threadIdx.x >> 5); tok < T; tok += gridDim.x * warps_per_block) {
    const float* row = scores + (size_t)tok * E;
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      const int e = lane + 32 * j;
      if (e < E) acc[j] += (double)__ldg(row + e);
    }
  }
#pragma unroll
  for (int j = 0; j < kEPL; ++j) {
    const int e = lane + 32 * j;
    if (e < E) atomicAdd(&ssum[e], acc[j]);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) atomicAdd(&colsum[e], ssum[e]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const double coef = (double)lambda / ((double)E * (double)T * (double)T);
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const double load = (double)__ldg(expert_load + e);
    ssum[e] = __ldcg(&colsum[e]) * load;
    dscores_col[e] = (float)(coef * load);
    colsum[e] = 0.0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int e = 0; e < E; ++e) tot += ssum[e];      // fixed order
    *loss = coef * tot;
    *ticket = 0;
  }
}

}  // namespace msr
