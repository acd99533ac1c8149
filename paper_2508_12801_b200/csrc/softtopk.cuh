// SoftTopk forward and backward (Eq. 6 and its derivative), its variants, and the auxiliary loss.
//
// Level j (1-based) of Eq. 6 adds a softmax with temperature t over the entries that are not among
// the j-1 largest (ties: lowest expert index).
#pragma once
#include <cuda_pipeline.h>
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

// ---------------------------------------------------------------------------------------------
// SoftTopk of Eq. 6 and its derivative, two lanes per token.
//
// With the token's k largest logits top[0] >= ... >= top[k-1] known (ties: lowest index first), level j is a
// softmax over everything but top[0..j-1], and its largest entry is top[j].  Taking each level relative to
// its own maximum r_j = top[j] keeps every exponential in (0, 1]:
//   tail entry e (never masked):  w_e(j) = z_e * c_j,   z_e = exp((a_e - top[k-1]) / t),  c_j = exp((top[k-1] - r_j) / t)
//   top entry i >= j:             w_i(j) = exp((top[i] - r_j) / t)
//   Z_j = c_j * sum_tail z + sum_{i >= j} w_i(j)
// so the row is read for one pass that finds the k largest, one pass of exponentials for the tail (whose sum
// is formed once), k(k+1)/2 exponentials among the top entries, and one pass that scales the tail by
// S = sum_j c_j / Z_j: no per-level pass over the row and no per-level reduction, about a third of the
// instructions of the level-by-level warp-per-token form.  Lane q of a token's two owns experts q, q+2, ...: it
// keeps the k largest of those in a sorted list (a new entry's place follows from comparisons with the old list
// alone, so the updates do not wait for one another), the two lists are merged with one exchange, and the sums
// over the tail are added up across the two lanes.  (One lane per token needs the fewest instructions but leaves
// an SM with 14 warps, as many as the rows it can hold in shared memory; four lanes per token double the
// instruction count; two keep it and give 24 warps.)  A CTA of 128 threads stages 64 rows in shared memory
// (coalesced both ways; the row stride is 2 mod 32 words so that a warp's 32 lanes hit 32 banks) and works on
// them in place.
constexpr int kStTok = 64;            // tokens per tile
constexpr int kStSplit = 2;           // lanes per token
constexpr int kStThreads = kStTok * kStSplit;

__host__ __device__ constexpr int st_stride(int E) { return (E + 31) / 32 * 32 + kStSplit; }

// With an even expert count every row starts on an 8-byte boundary in global and in shared memory (the stride is
// even), and the whole tile goes through asynchronous 8-byte copies: all of a warp's rows are in flight at once and no
// register holds them.  Otherwise eight rows at a time per warp through registers (up to 32 loads per lane in flight).
__device__ __forceinline__ void st_load_tile(const float* __restrict__ g, float* sm, int rows, int E, int stride) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kStThreads / 32, kBatch = 8;
  if ((E & 1) == 0) {
    const int pairs = E >> 1;
    for (int r = warp; r < rows; r += kWarps)
      for (int c = lane; c < pairs; c += 32)
        __pipeline_memcpy_async(sm + r * stride + 2 * c, g + (size_t)r * E + 2 * c, 8);
    __pipeline_commit();
    __pipeline_wait_prior(0);
    return;
  }
  for (int r0 = warp; r0 < rows; r0 += kWarps * kBatch) {
    float v[kBatch][kEPL];
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int r = r0 + b * kWarps;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) {
        const int c = lane + 32 * j;
        v[b][j] = (r < rows && c < E) ? __ldg(g + (size_t)r * E + c) : 0.f;
      }
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int r = r0 + b * kWarps;
#pragma unroll
      for (int j = 0; j < kEPL; ++j) {
        const int c = lane + 32 * j;
        if (r < rows && c < E) sm[r * stride + c] = v[b][j];
      }
    }
  }
}
__device__ __forceinline__ void st_store_tile(float* __restrict__ g, const float* sm, int rows, int E, int stride) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int r = warp; r < rows; r += kStThreads / 32) {
#pragma unroll
    for (int j = 0; j < kEPL; ++j) {
      const int c = lane + 32 * j;
      if (c < E) g[(size_t)r * E + c] = sm[r * stride + c];
    }
  }
}

// One more entry into a list of the K largest so far (descending; equal values by ascending index).  With kLex
// false the caller feeds indices in ascending order, so "below every entry that is not strictly smaller" is the
// tie rule; with kLex true (merging another lane's list) the index decides among equal values.
template <int K, bool kLex>
__device__ __forceinline__ void st_insert(float (&tv)[K], int (&ti)[K], float v, int e) {
  bool above[K];
#pragma unroll
  for (int i = 0; i < K; ++i)
    above[i] = kLex ? (v > tv[i] || (v == tv[i] && (unsigned)e < (unsigned)ti[i])) : (v > tv[i]);
#pragma unroll
  for (int i = K - 1; i > 0; --i) {
    tv[i] = above[i - 1] ? tv[i - 1] : (above[i] ? v : tv[i]);
    ti[i] = above[i - 1] ? ti[i - 1] : (above[i] ? e : ti[i]);
  }
  tv[0] = above[0] ? v : tv[0];
  ti[0] = above[0] ? e : ti[0];
}

// The rows of a tile as two bf16 halves, value = hi + lo (what the tensor-core gate backward reads): row t of `split`
// holds hi in columns [0, Kpad) and lo in [Kpad, 2 Kpad), zeros from column E on.  Two columns per lane and step.
__device__ __forceinline__ void st_store_split(__nv_bfloat16* __restrict__ split, const float* sm, int rows, int E,
                                               int stride, int Kpad) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int r = warp; r < rows; r += kStThreads / 32) {
    __nv_bfloat16* out = split + (size_t)r * 2 * Kpad;
    for (int c = 2 * lane; c < Kpad; c += 64) {
      const float x0 = c < E ? sm[r * stride + c] : 0.f, x1 = c + 1 < E ? sm[r * stride + c + 1] : 0.f;
      const __nv_bfloat16 h0 = __float2bfloat16(x0), h1 = __float2bfloat16(x1);
      const __nv_bfloat16 l0 = __float2bfloat16(x0 - __bfloat162float(h0)), l1 = __float2bfloat16(x1 - __bfloat162float(h1));
      *reinterpret_cast<__nv_bfloat162*>(out + c) = __halves2bfloat162(h0, h1);
      *reinterpret_cast<__nv_bfloat162*>(out + Kpad + c) = __halves2bfloat162(l0, l1);
    }
  }
}

// The K largest entries of a row (lane q scans experts q, q + 2, ...; then the lanes' lists are merged), the same
// in every lane of the token.  Slots that no entry reached keep index -1.
template <int K>
__device__ __forceinline__ void st_topk(const float* row, int E, int q, float (&tv)[K], int (&ti)[K]) {
#pragma unroll
  for (int i = 0; i < K; ++i) { tv[i] = -INFINITY; ti[i] = -1; }
#pragma unroll 4
  for (int e = q; e < E; e += kStSplit) st_insert<K, false>(tv, ti, row[e], e);
#pragma unroll
  for (int step = 1; step < kStSplit; step <<= 1) {
    float pv[K]; int pi[K];
#pragma unroll
    for (int i = 0; i < K; ++i) {
      pv[i] = __shfl_xor_sync(0xffffffffu, tv[i], step);
      pi[i] = __shfl_xor_sync(0xffffffffu, ti[i], step);
    }
#pragma unroll
    for (int i = 0; i < K; ++i) if (pi[i] >= 0) st_insert<K, true>(tv, ti, pv[i], pi[i]);
  }
}

__device__ __forceinline__ float st_group_sum(float x) {       // over the lanes of one token, the same in all of them
#pragma unroll
  for (int step = 1; step < kStSplit; step <<= 1) x += __shfl_xor_sync(0xffffffffu, x, step);
  return x;
}

// Levels 0..k-1 over the top entries: S = sum_j c_j / Z_j and, per top entry, y = sum_{j <= i} w_i(j) / Z_j.
// With kGrad, also Hs = sum_j c_j * gq_j / Z_j and, per top entry, sum_{j <= i} (w_i(j) / Z_j) * (g_i - gq_j),
// where gq_j = (c_j * gz_tail + sum_{i >= j} g_i w_i(j)) / Z_j.
template <int K, bool kGrad>
__device__ __forceinline__ void st_levels(const float (&tv)[K], int k, float inv_t, float z_tail, float gz_tail,
                                          const float (&gt)[K], float& S, float& Hs, float (&out)[K]) {
  float vk = tv[0];
#pragma unroll
  for (int i = 0; i < K; ++i) if (i == k - 1) vk = tv[i];
  S = 0.f; Hs = 0.f;
#pragma unroll
  for (int i = 0; i < K; ++i) out[i] = 0.f;
#pragma unroll
  for (int j = 0; j < K; ++j) {
    if (j >= k) break;
    const float rj = tv[j];
    const float cj = expf((vk - rj) * inv_t);
    float w[K];
    float Z = cj * z_tail, GZ = cj * gz_tail;
#pragma unroll
    for (int i = K - 1; i >= j; --i) {                  // smallest first
      w[i] = i < k ? expf((tv[i] - rj) * inv_t) : 0.f;
      Z += w[i];
      if (kGrad) GZ = fmaf(gt[i], w[i], GZ);
    }
    const float inv = 1.f / Z;
    S = fmaf(cj, inv, S);
    const float gq = GZ * inv;
    if (kGrad) Hs = fmaf(cj * inv, gq, Hs);
#pragma unroll
    for (int i = j; i < K; ++i) out[i] = kGrad ? fmaf(w[i] * inv, gt[i] - gq, out[i]) : fmaf(w[i], inv, out[i]);
  }
}

template <int K>
__global__ void __launch_bounds__(kStThreads, 6)
softtopk_fwd_kernel(const float* __restrict__ logits, float* __restrict__ scores, int T, int E, int k, float t) {
  extern __shared__ float st_sm[];
  const int stride = st_stride(E);
  const float inv_t = 1.f / t;
  const int r = threadIdx.x / kStSplit, q = threadIdx.x % kStSplit;
  for (int row0 = blockIdx.x * kStTok; row0 < T; row0 += gridDim.x * kStTok) {
    const int rows = min(kStTok, T - row0);
    st_load_tile(logits + (size_t)row0 * E, st_sm, rows, E, stride);
    __syncthreads();
    {   // every thread works, also on rows past the end of a ragged last tile (whatever the buffer holds there: nothing
        // of it is stored), so that the warp-wide exchanges below always have all 32 lanes
      float* row = st_sm + r * stride;
      float tv[K]; int ti[K];
      st_topk<K>(row, E, q, tv, ti);
      float vk = tv[0];
#pragma unroll
      for (int i = 0; i < K; ++i) {
        if (i == k - 1) vk = tv[i];
        if (q == 0 && i < k && ti[i] >= 0) row[ti[i]] = -INFINITY;   // out of the tail pass
      }
      __syncwarp();
      float acc0 = 0.f, acc1 = 0.f;
      int e = q;
      for (; e + kStSplit < E; e += 2 * kStSplit) {
        const float z0 = expf((row[e] - vk) * inv_t), z1 = expf((row[e + kStSplit] - vk) * inv_t);
        row[e] = z0; row[e + kStSplit] = z1; acc0 += z0; acc1 += z1;
      }
      if (e < E) { const float z0 = expf((row[e] - vk) * inv_t); row[e] = z0; acc0 += z0; }
      const float z_tail = st_group_sum(acc0 + acc1);
      float S, Hs, ytop[K];
      st_levels<K, false>(tv, k, inv_t, z_tail, 0.f, tv, S, Hs, ytop);      // (no gradients: the sixth argument is not read)
      for (e = q; e < E; e += kStSplit) row[e] *= S;
      __syncwarp();
#pragma unroll
      for (int i = 0; i < K; ++i) if (q == 0 && i < k && ti[i] >= 0) row[ti[i]] = ytop[i];
    }
    __syncthreads();
    st_store_tile(scores + (size_t)row0 * E, st_sm, rows, E, stride);
    __syncthreads();
  }
}

// dlogits = J^T g with g = the k gradients of the token's assigned experts plus, if given, a per-expert
// term shared by all tokens (the gradient of the auxiliary loss, Eq. 9).  The masks are constants.
//   da_l = (1/t) * sum_{levels j with l unmasked} q_l(j) * (g_l - gq_j),   q(j) = w(j) / Z_j,  gq_j = sum_i g_i q_i(j)
// which for a tail entry is (z_l / t) * (g_l * S - Hs).
template <int K>
__global__ void __launch_bounds__(kStThreads, 5)
softtopk_bwd_kernel(const float* __restrict__ logits, const int32_t* __restrict__ expert_idx,
                    const float* __restrict__ dgate_w, const float* __restrict__ dscores_col,
                    float* __restrict__ dlogits, __nv_bfloat16* __restrict__ dl_split, int Kpad, int T, int E, int k, float t) {
  extern __shared__ float st_sm[];
  const int stride = st_stride(E);
  float* col = st_sm + kStTok * stride;                  // the shared per-expert term (zeros if none)
  const float inv_t = 1.f / t;
  const int r = threadIdx.x / kStSplit, q = threadIdx.x % kStSplit;
  for (int e = threadIdx.x; e < E; e += kStThreads) col[e] = dscores_col ? __ldg(dscores_col + e) : 0.f;
  for (int row0 = blockIdx.x * kStTok; row0 < T; row0 += gridDim.x * kStTok) {
    const int rows = min(kStTok, T - row0);
    st_load_tile(logits + (size_t)row0 * E, st_sm, rows, E, stride);
    __syncthreads();
    {   // every thread works (see the forward kernel); rows past the end take no gradients
      const int tok = row0 + r;
      const bool live = r < rows;
      float* row = st_sm + r * stride;
      float tv[K]; int ti[K];
      st_topk<K>(row, E, q, tv, ti);
      float vk = tv[0];
      float gt[K];
#pragma unroll
      for (int i = 0; i < K; ++i) {
        if (i == k - 1) vk = tv[i];
        gt[i] = (i < k && ti[i] >= 0) ? col[ti[i]] : 0.f;
        if (q == 0 && i < k && ti[i] >= 0) row[ti[i]] = -INFINITY;
      }
      // the token's own gradients: to the top entry they belong to, else kept for the tail
      int se[kMaxK]; float sg[kMaxK];
#pragma unroll
      for (int c = 0; c < kMaxK; ++c) {
        se[c] = -1; sg[c] = 0.f;
        if (c < k && live) {
          const int e = __ldg(expert_idx + (size_t)tok * k + c);
          const float gv = __ldg(dgate_w + (size_t)tok * k + c);
          bool in_top = false;
#pragma unroll
          for (int i = 0; i < K; ++i) if (i < k && e >= 0 && ti[i] == e) { gt[i] += gv; in_top = true; }
          if (!in_top && e >= 0 && e < E) { se[c] = e; sg[c] = gv; }
        }
      }
      __syncwarp();
      float acc0 = 0.f, acc1 = 0.f, g0 = 0.f, g1 = 0.f;
      int e = q;
      for (; e + kStSplit < E; e += 2 * kStSplit) {
        const float z0 = expf((row[e] - vk) * inv_t), z1 = expf((row[e + kStSplit] - vk) * inv_t);
        row[e] = z0; row[e + kStSplit] = z1; acc0 += z0; acc1 += z1;
        g0 = fmaf(col[e], z0, g0); g1 = fmaf(col[e + kStSplit], z1, g1);
      }
      if (e < E) { const float z0 = expf((row[e] - vk) * inv_t); row[e] = z0; acc0 += z0; g0 = fmaf(col[e], z0, g0); }
      const float z_tail = st_group_sum(acc0 + acc1);
      float gz_tail = st_group_sum(g0 + g1);
      __syncwarp();
      float sz[kMaxK];
#pragma unroll
      for (int c = 0; c < kMaxK; ++c) { sz[c] = se[c] >= 0 ? row[se[c]] : 0.f; gz_tail = fmaf(sg[c], sz[c], gz_tail); }
      float S, Hs, dtop[K];
      st_levels<K, true>(tv, k, inv_t, z_tail, gz_tail, gt, S, Hs, dtop);
      __syncwarp();                                       // every lane has read the z it needs
      for (e = q; e < E; e += kStSplit) row[e] = row[e] * inv_t * fmaf(col[e], S, -Hs);
      __syncwarp();
      if (q == 0) {
#pragma unroll
        for (int c = 0; c < kMaxK; ++c) if (se[c] >= 0) row[se[c]] = fmaf(sz[c] * inv_t, sg[c] * S, row[se[c]]);
#pragma unroll
        for (int i = 0; i < K; ++i) if (i < k && ti[i] >= 0) row[ti[i]] = dtop[i] * inv_t;
      }
    }
    __syncthreads();
    st_store_tile(dlogits + (size_t)row0 * E, st_sm, rows, E, stride);
    if (dl_split) st_store_split(dl_split + (size_t)row0 * 2 * Kpad, st_sm, rows, E, stride, Kpad);
    __syncthreads();
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
