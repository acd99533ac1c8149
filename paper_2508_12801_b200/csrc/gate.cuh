// Gate logits L = H . W_g (+ bias), Eq. 2, and the derivative GEMMs.
//
// bf16 path: tcgen05 tensor cores.  One CTA owns a 128-token tile; H streams through a ring of
// 128x64 bf16 tiles loaded by TMA (128-byte swizzle), W_g (transposed and padded to [Npad, d] once
// per call) rides along, the fp32 accumulator [128 x Npad] lives in tensor memory and is read back
// by the four warps of the CTA, one TMEM lane quarter each, so that every thread ends up with one
// token's full row of logits.  The contraction is HBM-bound (intensity ~ E flop per byte of H), so
// the design goal is to keep as many H tiles in flight as shared memory allows: two CTAs per SM.
//
// fp32 path: plain FMA tiles (tensor cores would round the inputs to tf32).
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace msr {

// ---- tcgen05 / TMA wrappers ------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* tmap, int x, int y,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
// 2-D tile store shared -> global (clipped at the tensor's bounds), tracked by bulk async-groups
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, int x, int y, const void* smem_src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tmap),
               "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&r)[16]) {
  uint32_t u[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
        "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) r[i] = __uint_as_float(u[i]);
}

// Issue only: the registers may be read after tmem_ld_wait().  Several loads can be in flight.
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&u)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
        "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements) and
// were written by TMA with the 128-byte swizzle: groups of 8 rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc_bf16_m128(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

constexpr int kGateBM = 128, kGateBK = 64, kGateStages = 3;
constexpr int kGateATile = kGateBM * kGateBK * 2;   // 16 KiB
constexpr int kGateStageBytes = kGateATile + 16384; // the W_g tile is padded to 16 KiB to stay 1024-aligned
constexpr int kGateSmemBytes = kGateStages * kGateStageBytes + 1024;

struct GateSmem {
  uint64_t full[kGateStages], empty[kGateStages], accum;
  uint32_t tmem_base;
  int failed;
};

__global__ void __launch_bounds__(128)
gate_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW,
                    const float* __restrict__ bias, float* __restrict__ logits, int T, int E, int Npad,
                    int num_kb, unsigned* error_flag) {
  extern __shared__ unsigned char gsm_raw[];
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(gsm_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ GateSmem sm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * kGateBM;
  const uint32_t b_bytes = (uint32_t)Npad * kGateBK * 2;
  uint32_t tmem_cols = 32; while ((int)tmem_cols < Npad) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGateStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
    mbar_init(&sm.accum, 1);
    sm.failed = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sm.tmem_base, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = sm.tmem_base;

  if (warp == 0 && lane == 0) {
    // ---- producer: TMA loads of the H tile and the matching W_g columns ---------------------------
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % kGateStages;
      const uint32_t ph = (uint32_t)((kb / kGateStages) & 1);
      if (kb >= kGateStages && !mbar_wait_bounded(&sm.empty[s], ph ^ 1)) { sm.failed = 1; break; }
      unsigned char* a = tiles + (size_t)s * kGateStageBytes;
      mbar_expect_tx(&sm.full[s], kGateATile + b_bytes);
      tma_load_2d(a, &tmH, kb * kGateBK, m0, &sm.full[s]);
      tma_load_2d(a + kGateATile, &tmW, kb * kGateBK, 0, &sm.full[s]);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer: four K=16 instructions per 64-wide stage ------------------------------------
    const uint32_t idesc = idesc_bf16_m128(Npad);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % kGateStages;
      const uint32_t ph = (uint32_t)((kb / kGateStages) & 1);
      ok = mbar_wait_bounded(&sm.full[s], ph);
      if (!ok) break;
      tc_fence_after();
      const uint32_t a_addr = smem_u32(tiles + (size_t)s * kGateStageBytes);
      const uint64_t adesc = smem_desc_k128(a_addr), bdesc = smem_desc_k128(a_addr + kGateATile);
#pragma unroll
      for (int kk = 0; kk < kGateBK / 16; ++kk)      // +32 bytes along K inside the swizzle atom
        umma_bf16(tmem_acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
      umma_commit(&sm.empty[s]);                      // frees the stage when these MMAs retire
    }
    if (!ok) sm.failed = 1;
    umma_commit(&sm.accum);                           // accumulator complete
  }
  __syncwarp();
  // ---- epilogue: warp w reads TMEM lanes [32w, 32w+32), i.e. tokens m0 + 32w + lane ------------------
  const bool got = mbar_wait_bounded(&sm.accum, 0);
  tc_fence_after();
  if (got && !sm.failed) {
    const int row = m0 + warp * 32 + lane;
    for (int c0 = 0; c0 < Npad; c0 += 16) {
      float r[16];
      tmem_ld16(tmem_acc + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
      if (row < T) {
#pragma unroll
        for (int j = 0; j < 16; j += 4) {
          const int c = c0 + j;
          if (c + 3 < E && (E & 3) == 0) {
            float4 o = make_float4(r[j], r[j + 1], r[j + 2], r[j + 3]);
            if (bias) { o.x += __ldg(bias + c); o.y += __ldg(bias + c + 1); o.z += __ldg(bias + c + 2); o.w += __ldg(bias + c + 3); }
            *reinterpret_cast<float4*>(logits + (size_t)row * E + c) = o;
          } else {
            for (int jj = 0; jj < 4; ++jj)
              if (c + jj < E) logits[(size_t)row * E + c + jj] = r[j + jj] + (bias ? __ldg(bias + c + jj) : 0.f);
          }
        }
      }
    }
  } else if (threadIdx.x == 0) {
    atomicOr(error_flag, 4u);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, tmem_cols);
}

// W_g -> bf16 [Npad, d] with the contraction index contiguous; rows >= E are zero.
__global__ void wgate_prepare_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, int d,
                                     int E, int Npad, int layout) {
  const long long n = (long long)Npad * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(i / d), col = (int)(i % d);
    __nv_bfloat16 v = __float2bfloat16(0.f);
    if (row < E) v = layout == 0 ? w[(size_t)col * E + row] : w[(size_t)row * d + col];
    wt[i] = v;
  }
}

// ---- fp32 path and the derivative GEMMs: plain FMA tiles ------------------------------------------
template <typename T>
__device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// logits[i][j] = sum_m H[i][m] * W(m, j) + bias[j]; one thread per output, 16 x 16 thread tiles.
template <typename T>
__global__ void __launch_bounds__(256)
gate_gemm_simt_kernel(const T* __restrict__ H, const T* __restrict__ W, const float* __restrict__ bias,
                      float* __restrict__ logits, int Tn, int d, int E, int layout) {
  __shared__ float sh[16][17], sw[16][17];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int row = blockIdx.x * 16 + ty, col = blockIdx.y * 16 + tx;
  float acc = 0.f;
  for (int m0 = 0; m0 < d; m0 += 16) {
    const int hr = blockIdx.x * 16 + ty, hm = m0 + tx;
    sh[ty][tx] = (hr < Tn && hm < d) ? to_f(H[(size_t)hr * d + hm]) : 0.f;
    const int wm = m0 + ty, wc = blockIdx.y * 16 + tx;
    sw[ty][tx] = (wm < d && wc < E) ? to_f(layout == 0 ? W[(size_t)wm * E + wc] : W[(size_t)wc * d + wm]) : 0.f;
    __syncthreads();
#pragma unroll
    for (int m = 0; m < 16; ++m) acc = fmaf(sh[ty][m], sw[m][tx], acc);
    __syncthreads();
  }
  if (row < Tn && col < E) logits[(size_t)row * E + col] = acc + (bias ? bias[col] : 0.f);
}

// dH[i][m] = sum_j dL[i][j] * W(m, j); a CTA caches its 16 rows of dL in shared memory.
template <typename T>
__global__ void __launch_bounds__(256)
gate_bwd_dh_kernel(const float* __restrict__ dL, const T* __restrict__ W, T* __restrict__ dH, int Tn, int d,
                   int E, int layout) {
  __shared__ float sdl[16][kMaxE];
  const int r0 = blockIdx.x * 16;
  for (int i = threadIdx.x; i < 16 * E; i += blockDim.x) {
    const int r = i / E, j = i - r * E;
    sdl[r][j] = (r0 + r < Tn) ? dL[(size_t)(r0 + r) * E + j] : 0.f;
  }
  __syncthreads();
  for (int m = threadIdx.x; m < d; m += blockDim.x) {
    float acc[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) acc[r] = 0.f;
    for (int j = 0; j < E; ++j) {
      const float w = to_f(layout == 0 ? W[(size_t)m * E + j] : W[(size_t)j * d + m]);
#pragma unroll
      for (int r = 0; r < 16; ++r) acc[r] = fmaf(sdl[r][j], w, acc[r]);
    }
#pragma unroll
    for (int r = 0; r < 16; ++r)
      if (r0 + r < Tn) {
        if constexpr (sizeof(T) == 4) dH[(size_t)(r0 + r) * d + m] = acc[r];
        else dH[(size_t)(r0 + r) * d + m] = __float2bfloat16(acc[r]);
      }
  }
}

// dW[m][j] = sum_i H[i][m] * dL[i][j].  A CTA owns a 64-wide slice of m and a chunk of tokens and adds
// its partial sums to dW (fp32 atomics; dW is zeroed first).
constexpr int kDwTok = 256;
template <typename T>
__global__ void __launch_bounds__(256)
gate_bwd_dw_kernel(const T* __restrict__ H, const float* __restrict__ dL, float* __restrict__ dW, int Tn, int d,
                   int E) {
  __shared__ float sh[32][65];
  __shared__ float sdl[32][kMaxE];
  const int m0 = blockIdx.x * 64, i0 = blockIdx.y * kDwTok;
  const int tm = threadIdx.x & 63, tj = threadIdx.x >> 6;    // thread: column m0+tm, experts tj, tj+4, ...
  float acc[kMaxE / 4];
#pragma unroll
  for (int q = 0; q < kMaxE / 4; ++q) acc[q] = 0.f;
  for (int ib = 0; ib < kDwTok; ib += 32) {
    for (int x = threadIdx.x; x < 32 * 64; x += blockDim.x) {
      const int r = x >> 6, c = x & 63, i = i0 + ib + r;
      sh[r][c] = (i < Tn && m0 + c < d) ? to_f(H[(size_t)i * d + m0 + c]) : 0.f;
    }
    for (int x = threadIdx.x; x < 32 * E; x += blockDim.x) {
      const int r = x / E, j = x - r * E, i = i0 + ib + r;
      sdl[r][j] = (i < Tn) ? dL[(size_t)i * E + j] : 0.f;
    }
    __syncthreads();
    for (int r = 0; r < 32; ++r) {
      const float h = sh[r][tm];
#pragma unroll
      for (int q = 0; q < kMaxE / 4; ++q) {
        const int j = tj + 4 * q;
        if (j < E) acc[q] = fmaf(h, sdl[r][j], acc[q]);
      }
    }
    __syncthreads();
  }
  if (m0 + tm < d) {
#pragma unroll
    for (int q = 0; q < kMaxE / 4; ++q) {
      const int j = tj + 4 * q;
      if (j < E) atomicAdd(dW + (size_t)(m0 + tm) * E + j, acc[q]);
    }
  }
}

}  // namespace msr

// =================================================================================================
// Tensor-core derivative GEMMs (bf16 I/O).
//
// dlogits is fp32.  It is split into bf16 hi + lo parts (dL = hi + lo up to 2^-17 relative), laid
// out as dLs[T][2*Kpad] = [hi | lo] with Kpad = E rounded up to 64, so that the products against the
// exact bf16 H and W_g keep close to fp32 accuracy while running on the bf16 tensor pipe.
namespace msr {

__global__ void split_dlogits_kernel(const float* __restrict__ dL, __nv_bfloat16* __restrict__ dLs, int T, int E,
                                     int Kpad) {
  if ((E & 7) == 0) {
    // eight columns per thread: two 16-byte loads, one 16-byte store each for the hi and the lo part
    const int g8 = Kpad >> 3;
    const long long n = (long long)T * g8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
      const long long t = i / g8; const int j = (int)(i - t * g8) << 3;
      float x[8];
      if (j < E) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(dL + t * E + j));
        const float4 b = __ldg(reinterpret_cast<const float4*>(dL + t * E + j) + 1);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
      } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) x[q] = 0.f;
      }
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const __nv_bfloat16 h0 = __float2bfloat16(x[2 * q]), h1 = __float2bfloat16(x[2 * q + 1]);
        const __nv_bfloat16 l0 = __float2bfloat16(x[2 * q] - __bfloat162float(h0));
        const __nv_bfloat16 l1 = __float2bfloat16(x[2 * q + 1] - __bfloat162float(h1));
        hi[q] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
        lo[q] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
      }
      *reinterpret_cast<uint4*>(dLs + t * 2 * Kpad + j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *reinterpret_cast<uint4*>(dLs + t * 2 * Kpad + Kpad + j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
    return;
  }
  const long long n = (long long)T * Kpad;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / Kpad; const int j = (int)(i - t * Kpad);
    float x = j < E ? dL[t * E + j] : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16(x);
    const __nv_bfloat16 lo = __float2bfloat16(x - __bfloat162float(hi));
    dLs[t * 2 * Kpad + j] = hi;
    dLs[t * 2 * Kpad + Kpad + j] = lo;
  }
}

// W_g as bf16 [d][Kpad] (expert index contiguous, zero padded): the K-major B operand of dH = dL . W_g^T
__global__ void wgate_kmajor_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wk, int d, int E,
                                    int Kpad, int layout) {
  const long long n = (long long)d * Kpad;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / Kpad), j = (int)(i % Kpad);
    __nv_bfloat16 v = __float2bfloat16(0.f);
    if (j < E) v = layout == 0 ? w[(size_t)m * E + j] : w[(size_t)j * d + m];
    wk[i] = v;
  }
}

// Descriptor of an MN-major bf16 operand tile written by TMA boxes of 64 (M or N) x rows (K) with the
// 128-byte swizzle: a K row is 128 bytes, groups of 8 K rows are 1024 bytes apart, and the next
// 64-wide chunk along M/N starts `chunk_bytes` further.
__device__ __forceinline__ uint64_t smem_desc_mn128(uint32_t saddr, uint32_t chunk_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((chunk_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__host__ __device__ constexpr uint32_t idesc_bf16_m128_mn(int n) {   // both operands MN-major
  return idesc_bf16_m128(n) | (1u << 15) | (1u << 16);
}

// ---- dH[T, d] = dL[T, E] . W_g^T -------------------------------------------------------------------
// One CTA per 128-token tile.  The dL tile (hi and lo) is loaded once; 128-column tiles of W_g stream
// through a 2-stage ring; two TMEM accumulators alternate so that the four epilogue warps convert and
// stage tile n in shared memory (two TMA tile stores per warp) while the MMA warp works on tile n+1.
constexpr int kDhBN = 128, kDhStages = 2;
constexpr int kDhOutBytes = 2 * 4 * 2 * 4096;     // output staging: [2 buffers][4 warps][2 column halves][32 rows x 128 B]
struct DhSmem {
  uint64_t a_full, b_full[kDhStages], b_empty[kDhStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int failed;
};

__global__ void __launch_bounds__(192)
gate_bwd_dh_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmOut, int T, int d, int Kpad, unsigned* error_flag) {
  extern __shared__ unsigned char dsm_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(dsm_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ DhSmem sm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * 128;
  const int kboxes = Kpad / 64;                       // 64-wide K boxes per part
  const uint32_t a_bytes = 2u * kboxes * 16384u;      // hi and lo
  const uint32_t b_bytes = kboxes * 16384u;
  unsigned char* a_tile = base;                       // [2*kboxes][128 rows][128 B]
  unsigned char* b_ring = base + a_bytes;             // [stage][kboxes][128 rows][128 B]
  unsigned char* out_stage = b_ring + (size_t)kDhStages * b_bytes;   // kDhOutBytes, 1024-byte aligned pieces
  const int n_tiles = (d + kDhBN - 1) / kDhBN;

  if (threadIdx.x == 0) {
    mbar_init(&sm.a_full, 1);
    for (int s = 0; s < kDhStages; ++s) { mbar_init(&sm.b_full[s], 1); mbar_init(&sm.b_empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm.acc_full[b], 1); mbar_init(&sm.acc_empty[b], 4); }
    sm.failed = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sm.tmem_base, 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 0 && lane == 0) {
    mbar_expect_tx(&sm.a_full, a_bytes);
    for (int kb = 0; kb < kboxes; ++kb) {
      tma_load_2d(a_tile + (size_t)kb * 16384, &tmA, kb * 64, m0, &sm.a_full);                      // hi
      tma_load_2d(a_tile + (size_t)(kboxes + kb) * 16384, &tmA, Kpad + kb * 64, m0, &sm.a_full);    // lo
    }
    for (int nt = 0; nt < n_tiles; ++nt) {
      const int s = nt % kDhStages;
      const uint32_t ph = (uint32_t)((nt / kDhStages) & 1);
      if (nt >= kDhStages && !mbar_wait_bounded(&sm.b_empty[s], ph ^ 1)) { sm.failed = 1; break; }
      mbar_expect_tx(&sm.b_full[s], b_bytes);
      for (int kb = 0; kb < kboxes; ++kb)
        tma_load_2d(b_ring + (size_t)s * b_bytes + (size_t)kb * 16384, &tmB, kb * 64, nt * kDhBN, &sm.b_full[s]);
    }
  } else if (warp == 1 && lane == 0) {
    const uint32_t idesc = idesc_bf16_m128(kDhBN);
    bool ok = mbar_wait_bounded(&sm.a_full, 0);
    for (int nt = 0; nt < n_tiles && ok; ++nt) {
      const int s = nt % kDhStages, buf = nt & 1;
      if (nt >= 2) ok = mbar_wait_bounded(&sm.acc_empty[buf], (uint32_t)(((nt >> 1) & 1) ^ 1));
      if (ok) ok = mbar_wait_bounded(&sm.b_full[s], (uint32_t)((nt / kDhStages) & 1));
      if (!ok) break;
      tc_fence_after();
      const uint32_t acc = tmem + (uint32_t)(buf * kDhBN);
      uint32_t first = 0;
      for (int kb = 0; kb < kboxes; ++kb) {
        const uint64_t bd = smem_desc_k128(smem_u32(b_ring + (size_t)s * b_bytes + (size_t)kb * 16384));
        const uint64_t ah = smem_desc_k128(smem_u32(a_tile + (size_t)kb * 16384));
        const uint64_t al = smem_desc_k128(smem_u32(a_tile + (size_t)(kboxes + kb) * 16384));
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          umma_bf16(acc, ah + 2 * kk, bd + 2 * kk, idesc, first); first = 1;
          umma_bf16(acc, al + 2 * kk, bd + 2 * kk, idesc, 1u);
        }
      }
      umma_commit(&sm.b_empty[s]);
      umma_commit(&sm.acc_full[buf]);
    }
    if (!ok) sm.failed = 1;
  } else if (warp >= 2) {
    const int quarter = warp & 3;                      // TMEM lanes this warp may read
    bool ok = true;
    for (int nt = 0; nt < n_tiles && ok; ++nt) {
      const int buf = nt & 1;
      ok = mbar_wait_bounded(&sm.acc_full[buf], (uint32_t)((nt >> 1) & 1));
      if (!ok) break;
      tc_fence_after();
      // Staging for the TMA tile store: per warp and column half a 32-row x 128-byte box in the 128-byte
      // swizzle (16-byte chunk c of row r sits at chunk c ^ (r & 7)), which also spreads the lanes' writes
      // over the banks.  The buffer used two tiles ago must have been read by its store first.
      if (lane == 0 && nt >= 2) bulk_wait_read<1>();
      __syncwarp();
      unsigned char* my_box = out_stage + ((size_t)buf * 4 + quarter) * 8192;
      for (int c0 = 0; c0 < kDhBN; c0 += 64) {          // four TMEM loads in flight, one wait
        uint32_t u[4][16];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          tmem_ld16_issue(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kDhBN + c0 + 16 * q), u[q]);
        tmem_ld_wait();
        unsigned char* my_row = my_box + (c0 >> 6) * 4096 + lane * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(u[q][2 * j]), __uint_as_float(u[q][2 * j + 1]));
            w[j] = *reinterpret_cast<uint32_t*>(&h);
          }
          *reinterpret_cast<uint4*>(my_row + (((2 * q) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(my_row + (((2 * q + 1) ^ (lane & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) {
        // two tile stores per warp and tile (rows beyond T and columns beyond d are clipped by the copy)
        const int y = m0 + quarter * 32;
        if (y < T) {
          const int col0 = nt * kDhBN;
          tma_store_2d(&tmOut, col0, y, my_box);
          if (col0 + 64 < d) tma_store_2d(&tmOut, col0 + 64, y, my_box + 4096);
        }
        bulk_commit();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.acc_empty[buf]);
    }
    if (lane == 0) bulk_wait_all<0>();
    if (!ok && lane == 0) sm.failed = 1;
  }
  __syncthreads();
  if (threadIdx.x == 0 && sm.failed) atomicOr(error_flag, 4u);
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem, 256);
}

// ---- dW[d, E] = H^T . dL ---------------------------------------------------------------------------
// The contraction runs over tokens while both operands are stored with tokens as rows, so both are
// MN-major for the tensor core: a TMA box of 64 columns x 64 tokens lands in exactly the layout the
// MN-major descriptor names.  A CTA owns 128 columns of H (rows of dW) and one chunk of tokens
// (split-K); partial results go to a workspace and are summed in a fixed order by a second kernel.
constexpr int kDwStages = 4, kDwBK = 64;
struct DwSmem {
  uint64_t full[kDwStages], empty[kDwStages], accum;
  uint32_t tmem_base;
  int failed;
};

__global__ void __launch_bounds__(128)
gate_bwd_dw_tc_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmL,
                      float* __restrict__ partial, int T, int d, int E, int Kpad, int tokens_per_split,
                      unsigned* error_flag) {
  extern __shared__ unsigned char wsm_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(wsm_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ DwSmem sm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * 128;
  const int t_begin = blockIdx.y * tokens_per_split;
  const int t_end = min(T, t_begin + tokens_per_split);
  const int num_kb = (t_end - t_begin + kDwBK - 1) / kDwBK;
  const int nboxes = Kpad / 64;                                   // 64-wide N chunks
  const uint32_t a_bytes = 2u * 8192u, b_bytes = 2u * nboxes * 8192u;   // B: hi and lo
  const uint32_t stage_bytes = a_bytes + b_bytes;
  uint32_t tmem_cols = 32; while ((int)tmem_cols < Kpad) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kDwStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
    mbar_init(&sm.accum, 1);
    sm.failed = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sm.tmem_base, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 0 && lane == 0) {
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % kDwStages;
      const uint32_t ph = (uint32_t)((kb / kDwStages) & 1);
      if (kb >= kDwStages && !mbar_wait_bounded(&sm.empty[s], ph ^ 1)) { sm.failed = 1; break; }
      unsigned char* st = base + (size_t)s * stage_bytes;
      const int t0 = t_begin + kb * kDwBK;
      mbar_expect_tx(&sm.full[s], stage_bytes);
      tma_load_2d(st, &tmH, m0, t0, &sm.full[s]);
      tma_load_2d(st + 8192, &tmH, m0 + 64, t0, &sm.full[s]);
      for (int nb = 0; nb < nboxes; ++nb) {
        tma_load_2d(st + a_bytes + (size_t)nb * 8192, &tmL, nb * 64, t0, &sm.full[s]);                          // hi
        tma_load_2d(st + a_bytes + (size_t)(nboxes + nb) * 8192, &tmL, Kpad + nb * 64, t0, &sm.full[s]);        // lo
      }
    }
  } else if (warp == 1 && lane == 0) {
    const uint32_t idesc = idesc_bf16_m128_mn(Kpad);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % kDwStages;
      ok = mbar_wait_bounded(&sm.full[s], (uint32_t)((kb / kDwStages) & 1));
      if (!ok) break;
      tc_fence_after();
      const uint32_t sa = smem_u32(base + (size_t)s * stage_bytes);
      const uint32_t sbh = sa + a_bytes, sbl = sbh + nboxes * 8192u;
#pragma unroll
      for (int kk = 0; kk < kDwBK / 16; ++kk) {           // 16 tokens = 2048 bytes further down each box
        const uint64_t ad = smem_desc_mn128(sa + kk * 2048u, 8192u);
        umma_bf16(tmem, ad, smem_desc_mn128(sbh + kk * 2048u, 8192u), idesc, (kb > 0 || kk > 0) ? 1u : 0u);
        umma_bf16(tmem, ad, smem_desc_mn128(sbl + kk * 2048u, 8192u), idesc, 1u);
      }
      umma_commit(&sm.empty[s]);
    }
    if (!ok) sm.failed = 1;
    umma_commit(&sm.accum);
  }
  __syncwarp();
  const bool got = mbar_wait_bounded(&sm.accum, 0);
  tc_fence_after();
  if (got && !sm.failed && num_kb > 0) {
    const int row = m0 + warp * 32 + lane;              // row of dW = column of H
    float* out = partial + ((size_t)blockIdx.y * d + row) * E;
    for (int c0 = 0; c0 < Kpad; c0 += 16) {
      float r[16];
      tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
      if (row < d)
        for (int j = 0; j < 16; ++j)
          if (c0 + j < E) out[c0 + j] = r[j];
    }
  } else if (num_kb <= 0) {
    const int row = m0 + warp * 32 + lane;
    if (row < d) for (int j = 0; j < E; ++j) partial[((size_t)blockIdx.y * d + row) * E + j] = 0.f;
  } else if (threadIdx.x == 0) {
    atomicOr(error_flag, 4u);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

__global__ void reduce_dw_kernel(const float* __restrict__ partial, float* __restrict__ dW, long long n, int nsplit) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < nsplit; ++s) acc += partial[(size_t)s * n + i];   // fixed order: reproducible
    dW[i] = acc;
  }
}

}  // namespace msr
