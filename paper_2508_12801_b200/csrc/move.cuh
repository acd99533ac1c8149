// Index build, dispatch, combine and combine-backward: the data movement of Eq. 1 through the
// capacity-shaped [E, C, d_model] expert buffers of Sec. 2.3.
#pragma once
#include "common.cuh"

namespace msr {

// ---------------------------------------------------------------------------------------------
// Index build.  slot_idx[i, c] = rank of token i among the tokens of expert expert_idx[i, c], in
// ascending token order; slot_token is the inverse map.  Deterministic: no atomic decides an order.
//   pass 1: per block of kIdxTok tokens, count tokens per expert
//   pass 2: a block's base offset per expert = sum of the counts of the blocks before it; inside the
//           block, warps are ordered by a scan of per-warp counts and lanes by a ballot mask.
constexpr int kIdxTok = 1024;   // tokens per block, one per thread

__global__ void __launch_bounds__(kIdxTok)
index_count_kernel(const int32_t* __restrict__ expert_idx, int32_t* __restrict__ block_counts, int T,
                   int E, int k) {
  __shared__ int cnt[kMaxE];
  for (int e = threadIdx.x; e < E; e += blockDim.x) cnt[e] = 0;
  __syncthreads();
  int tok = blockIdx.x * kIdxTok + threadIdx.x;
  if (tok < T)
    for (int c = 0; c < k; ++c) {
      int e = __ldg(expert_idx + (size_t)tok * k + c);
      if (e >= 0 && e < E) atomicAdd(&cnt[e], 1);
    }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) block_counts[(size_t)blockIdx.x * E + e] = cnt[e];
}

__global__ void __launch_bounds__(kIdxTok)
index_fill_kernel(const int32_t* __restrict__ expert_idx, const int32_t* __restrict__ block_counts,
                  int32_t* __restrict__ slot_idx, int32_t* __restrict__ slot_token,
                  int32_t* __restrict__ expert_load, int T, int E, int k, int C,
                  const float* __restrict__ scores = nullptr, float* __restrict__ gate_w = nullptr) {
  __shared__ int base[kMaxE];                       // first slot of this block per expert
  __shared__ int wcnt[kIdxTok / 32][kMaxE + 1];     // per-warp counts, then exclusive offsets
  __shared__ unsigned bits[kIdxTok / 32][kMaxE];    // lanes of the warp that hold the expert
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // first slot of this block per expert = the counts of all earlier blocks; the sums are split over
  // the threads (part p of an expert takes blocks p, p + parts, ...) so that the loads overlap.  Integer
  // sums: the order of the additions does not matter.
  __shared__ int total[kMaxE];
  for (int e = threadIdx.x; e < E; e += blockDim.x) { base[e] = 0; total[e] = 0; }
  for (int e = lane; e < E; e += 32) bits[warp][e] = 0u;
  __syncthreads();
  {
    const int parts = max(1, (int)blockDim.x / E);
    const int e = threadIdx.x % E, part = threadIdx.x / E;
    if (part < parts) {
      int b = 0, tot = 0;
#pragma unroll 4
      for (int blk = part; blk < (int)gridDim.x; blk += parts) {
        const int v = __ldg(block_counts + (size_t)blk * E + e);
        if (blk < (int)blockIdx.x) b += v;
        tot += v;
      }
      if (b) atomicAdd(&base[e], b);
      if (tot) atomicAdd(&total[e], tot);
    }
  }
  __syncthreads();
  if (blockIdx.x == 0)
    for (int e = threadIdx.x; e < E; e += blockDim.x) expert_load[e] = total[e];
  const int tok = blockIdx.x * kIdxTok + threadIdx.x;
  int mine[kMaxK];
  float gw[kMaxK];
#pragma unroll
  for (int c = 0; c < kMaxK; ++c) {
    mine[c] = -1;
    if (c < k && tok < T) {
      int e = __ldg(expert_idx + (size_t)tok * k + c);
      if (e >= 0 && e < E) { mine[c] = e; atomicOr(&bits[warp][e], 1u << lane); }
      // on the way, if asked for: the combine weight of the pair, i.e. the token's score for that expert (Eq. 1);
      // all k loads are issued before the first is stored
      if (gate_w) gw[c] = (e >= 0 && e < E) ? __ldg(scores + (size_t)tok * E + e) : 0.f;
    }
  }
  __syncthreads();
  for (int e = lane; e < E; e += 32) wcnt[warp][e] = __popc(bits[warp][e]);
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {   // exclusive scan over the warps of the block
    int run = 0;
    for (int w = 0; w < kIdxTok / 32; ++w) { int v = wcnt[w][e]; wcnt[w][e] = run; run += v; }
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < kMaxK; ++c) {
    if (mine[c] >= 0) {
      int e = mine[c];
      int slot = base[e] + wcnt[warp][e] + __popc(bits[warp][e] & ((1u << lane) - 1u));
      slot_idx[(size_t)tok * k + c] = slot;
      if (slot < C) slot_token[(size_t)e * C + slot] = tok;
    }
  }
  if (gate_w && tok < T) {
#pragma unroll
    for (int c = 0; c < kMaxK; ++c) if (c < k) gate_w[(size_t)tok * k + c] = gw[c];
  }
}

// ---------------------------------------------------------------------------------------------
// Dispatch: xdisp[e, slot, :] = H[token, :] for the token's k (expert, slot) pairs.  Token-major, so
// every row is read once and written k times.  (dispatch_tma_kernel below does the same through the copy
// engine, every warp driving its own ring of bulk copies; it measures 0.86 of the HBM copy peak on the
// write-heavy stress shape, this one 0.91, so this one is the default.)
// One warp per token, a lane owns 16-byte column groups, kDispatchBatch groups are loaded (streaming
// loads) before their copies are stored (streaming stores).
constexpr int kDispatchBatch = 4;     // 16-byte groups a lane loads before it stores their copies
__global__ void __launch_bounds__(256)
dispatch_kernel(const char* __restrict__ src, const int32_t* __restrict__ expert_idx,
                     const int32_t* __restrict__ slot_idx, char* __restrict__ dst, int Tn, uint32_t row_bytes,
                     int k, int C) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const uint32_t nvec = row_bytes / 16;
  for (int tok = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; tok < Tn; tok += warps) {
    long long my_off = -1;
    if (lane < k) {
      const int e = __ldg(expert_idx + (size_t)tok * k + lane), sl = __ldg(slot_idx + (size_t)tok * k + lane);
      if (e >= 0 && sl >= 0 && sl < C) my_off = ((long long)e * C + sl) * (long long)row_bytes;
    }
    long long off[kMaxK];
#pragma unroll
    for (int c = 0; c < kMaxK; ++c) off[c] = __shfl_sync(0xffffffffu, my_off, c);
    const uint4* srow = reinterpret_cast<const uint4*>(src + (size_t)tok * row_bytes);
    for (uint32_t v0 = lane; v0 < nvec; v0 += 32 * kDispatchBatch) {
      uint4 x[kDispatchBatch];
#pragma unroll
      for (int u = 0; u < kDispatchBatch; ++u) if (v0 + 32 * u < nvec) x[u] = __ldcs(srow + v0 + 32 * u);
#pragma unroll
      for (int c = 0; c < kMaxK; ++c) {
        if (c >= k || off[c] < 0) continue;
        uint4* drow = reinterpret_cast<uint4*>(dst + off[c]);
#pragma unroll
        for (int u = 0; u < kDispatchBatch; ++u) if (v0 + 32 * u < nvec) __stcs(drow + v0 + 32 * u, x[u]);
      }
    }
  }
}

// Dispatch through the copy engine: every warp keeps a ring of kTmaStages row buffers in shared memory.  Lane 0
// brings a token's row (or a piece of it, at most kTmaChunk bytes) in with one bulk copy global -> shared that
// completes on an mbarrier; lanes 0..k-1 then each send it to one of the token's k slots with one bulk copy
// shared -> global.  A buffer is reused once the copies out of it have finished reading it
// (cp.async.bulk.wait_group.read).  No register or LSU traffic for the data: the load/store units only carry
// the indices.  Every mbarrier wait is bounded; a wait that runs out raises the error flag and the warp stops.
constexpr int kTmaStages = 4, kTmaWarps = 4, kTmaChunk = 8192;
__global__ void __launch_bounds__(kTmaWarps * 32)
dispatch_tma_kernel(const char* __restrict__ src, const int32_t* __restrict__ expert_idx,
                    const int32_t* __restrict__ slot_idx, char* __restrict__ dst, int Tn, uint32_t row_bytes,
                    uint32_t chunk, int k, int C, unsigned* error_flag) {
  extern __shared__ __align__(128) unsigned char tma_smem[];
  __shared__ __align__(8) uint64_t bars[kTmaWarps][kTmaStages];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned char* ring = tma_smem + (size_t)warp * kTmaStages * chunk;
  if (lane == 0)
    for (int s = 0; s < kTmaStages; ++s) mbar_init(&bars[warp][s], 1);
  fence_barrier_init();
  __syncwarp();
  const uint32_t pieces = (row_bytes + chunk - 1) / chunk;
  const long long units = (long long)Tn * pieces;
  const long long first = (long long)blockIdx.x * kTmaWarps + warp, stride = (long long)gridDim.x * kTmaWarps;
  auto issue_load = [&](long long u, int s) {            // lane 0 only
    const long long tok = u / pieces; const uint32_t pc = (uint32_t)(u - tok * pieces);
    const uint32_t off = pc * chunk, bytes = min(chunk, row_bytes - off);
    mbar_expect_tx(&bars[warp][s], bytes);
    bulk_g2s(ring + (size_t)s * chunk, src + (size_t)tok * row_bytes + off, bytes, &bars[warp][s]);
  };
  // Two loads run ahead of the unit being sent out.  With four buffers that leaves one for the unit in hand and
  // one whose outgoing copies (committed one iteration ago) may still be reading it.
  constexpr int kAhead = kTmaStages - 2;
  if (lane == 0)
    for (int s = 0; s < kAhead; ++s)
      if (first + s * stride < units) issue_load(first + s * stride, s);
  int it = 0; bool failed = false;
  for (long long u = first; u < units; u += stride, ++it) {
    const int s = it % kTmaStages;
    const long long tok = u / pieces; const uint32_t pc = (uint32_t)(u - tok * pieces);
    const uint32_t off = pc * chunk, bytes = min(chunk, row_bytes - off);
    long long my_off = -1;
    if (lane < k) {
      const int e = __ldg(expert_idx + (size_t)tok * k + lane), sl = __ldg(slot_idx + (size_t)tok * k + lane);
      if (e >= 0 && sl >= 0 && sl < C) my_off = ((long long)e * C + sl) * (long long)row_bytes + off;
    }
    // the buffer the next load lands in was last read by the copies committed two iterations ago: every lane
    // waits until at most its latest group is still reading, then the warp agrees before lane 0 overwrites it
    bulk_wait_read<1>();
    __syncwarp();
    if (lane == 0 && u + kAhead * stride < units) issue_load(u + kAhead * stride, (it + kAhead) % kTmaStages);
    int ok = 1;
    if (lane == 0) ok = mbar_wait_bounded(&bars[warp][s], (it / kTmaStages) & 1) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncwarp();
    if (!ok) { failed = true; break; }
    if (my_off >= 0) bulk_s2g(dst + my_off, ring + (size_t)s * chunk, bytes);
    bulk_commit();
  }
  if (failed) {
    // a load never arrived: report it, give the loads still in flight a bounded chance to land, and leave
    if (lane == 0) {
      atomicExch(error_flag, 1u);
      for (int a = 1; a <= kAhead; ++a) mbar_wait_bounded(&bars[warp][(it + a) % kTmaStages], ((it + a) / kTmaStages) & 1, 1u << 16);
    }
  }
  bulk_wait_all<0>();
}

// Zero the rows of padding slots (slot_token < 0) of an [E*C, row] buffer.
__global__ void __launch_bounds__(256)
zero_padding_kernel(const int32_t* __restrict__ slot_token, char* __restrict__ dst, long long n_slots,
                    uint32_t row_bytes) {
  // a warp looks at 32 slots per step and then zeroes, all lanes together, the rows that are padding
  const int warps = blockDim.x >> 5, lane = threadIdx.x & 31;
  for (long long base = ((long long)blockIdx.x * warps + (threadIdx.x >> 5)) * 32; base < n_slots;
       base += (long long)gridDim.x * warps * 32) {
    const long long s = base + lane;
    unsigned mask = __ballot_sync(0xffffffffu, s < n_slots && __ldg(slot_token + s) < 0);
    while (mask) {
      const int b = __ffs(mask) - 1; mask &= mask - 1;
      uint4* row = reinterpret_cast<uint4*>(dst + (base + b) * (long long)row_bytes);
      for (uint32_t v = lane; v < row_bytes / 16; v += 32) row[v] = make_uint4(0, 0, 0, 0);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Combine: dst[i, :] = sum_c w[i, c] * src[e_c, slot_c, :] in fp32, ascending c, rounded once.
// One warp per token: lanes < k fetch the token's slots and weights and share them by shuffle, so no
// block barrier sits between a token's index loads and its row loads; a lane owns 16-byte column
// groups and keeps the k row loads of a group in flight together.
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(const T* __restrict__ src, const int32_t* __restrict__ expert_idx,
               const int32_t* __restrict__ slot_idx, const float* __restrict__ gate_w,
               T* __restrict__ dst, int Tn, int d, int k, int C, int accumulate) {
  constexpr int N = Vec16<T>::N;
  const int nvec = d / N;
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  for (int tok = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; tok < Tn; tok += warps) {
    long long my_off = -1; float my_w = 0.f;
    if (lane < k) {
      const int e = __ldg(expert_idx + (size_t)tok * k + lane);
      const int sl = __ldg(slot_idx + (size_t)tok * k + lane);
      const bool valid = e >= 0 && sl >= 0 && sl < C;   // a malformed or surplus entry contributes nothing:
      my_off = valid ? ((long long)e * C + sl) * (long long)d : -1;   // its row is neither read nor added
      my_w = !valid ? 0.f : gate_w ? __ldg(gate_w + (size_t)tok * k + lane) : 1.f;
    }
    long long rowoff[kMaxK]; float wgt[kMaxK];
#pragma unroll
    for (int c = 0; c < kMaxK; ++c) {
      rowoff[c] = __shfl_sync(0xffffffffu, my_off, c);
      wgt[c] = __shfl_sync(0xffffffffu, my_w, c);
    }
    for (int v = lane; v < nvec; v += 32) {
      float acc[N];
#pragma unroll
      for (int j = 0; j < N; ++j) acc[j] = 0.f;
      if (accumulate) Vec16<T>::load(dst + (size_t)tok * d + (size_t)v * N, acc);
      // all k row loads are issued before any is used; they stay packed (4 registers each) until then
      uint4 raw[kMaxK];
#pragma unroll
      for (int c = 0; c < kMaxK; ++c)
        if (c < k && rowoff[c] >= 0) raw[c] = ldg16(src + rowoff[c] + (size_t)v * N);
#pragma unroll
      for (int c = 0; c < kMaxK; ++c)
        if (c < k && rowoff[c] >= 0) {
          float x[N];
          Vec16<T>::unpack(raw[c], x);
          const float w = wgt[c];
#pragma unroll
          for (int j = 0; j < N; ++j) acc[j] = fmaf(w, x[j], acc[j]);
        }
      Vec16<T>::store(dst + (size_t)tok * d + (size_t)v * N, acc);
    }
  }
}

// Combine backward: dyexp[e_c, slot_c, :] = w[i, c] * dY[i, :],  dgate_w[i, c] = <dY[i, :], yexp[e_c, slot_c, :]>.
// One CTA per token; the dY chunk of a thread is read once and reused for the k experts.
template <typename T>
__global__ void __launch_bounds__(256)
combine_bwd_kernel(const T* __restrict__ dY, const T* __restrict__ yexp,
                   const int32_t* __restrict__ expert_idx, const int32_t* __restrict__ slot_idx,
                   const float* __restrict__ gate_w, T* __restrict__ dyexp, float* __restrict__ dgate_w,
                   int Tn, int d, int k, int C) {
  constexpr int N = Vec16<T>::N;
  __shared__ long long rowoff[kMaxK];
  __shared__ float wgt[kMaxK];
  __shared__ float red[8][kMaxK];
  const int nvec = d / N;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int tok = blockIdx.x; tok < Tn; tok += gridDim.x) {
    __syncthreads();
    if (threadIdx.x < k) {
      int e = __ldg(expert_idx + (size_t)tok * k + threadIdx.x);
      int sl = __ldg(slot_idx + (size_t)tok * k + threadIdx.x);
      const bool valid = e >= 0 && sl >= 0 && sl < C;   // a malformed entry is skipped
      rowoff[threadIdx.x] = valid ? ((long long)e * C + sl) * (long long)d : -1;
      wgt[threadIdx.x] = __ldg(gate_w + (size_t)tok * k + threadIdx.x);
    }
    __syncthreads();
    float dot[kMaxK];
#pragma unroll
    for (int c = 0; c < kMaxK; ++c) dot[c] = 0.f;
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
      float g[N];
      Vec16<T>::load(dY + (size_t)tok * d + (size_t)v * N, g);
      uint4 raw[kMaxK];                                  // the k row loads stay packed until they are used
#pragma unroll
      for (int c = 0; c < kMaxK; ++c)
        if (c < k && rowoff[c] >= 0) raw[c] = ldg16(yexp + rowoff[c] + (size_t)v * N);
#pragma unroll
      for (int c = 0; c < kMaxK; ++c)
        if (c < k && rowoff[c] >= 0) {
          float y[N], o[N];
          Vec16<T>::unpack(raw[c], y);
          const float w = wgt[c];
#pragma unroll
          for (int j = 0; j < N; ++j) { dot[c] = fmaf(g[j], y[j], dot[c]); o[j] = w * g[j]; }
          Vec16<T>::store(dyexp + rowoff[c] + (size_t)v * N, o);
        }
    }
#pragma unroll
    for (int c = 0; c < kMaxK; ++c) {
      float s = warp_sum(dot[c]);
      if (lane == 0) red[warp][c] = s;
    }
    __syncthreads();
    if (threadIdx.x < k) {
      float s = 0.f;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w][threadIdx.x];
      dgate_w[(size_t)tok * k + threadIdx.x] = s;
    }
  }
}

}  // namespace msr
