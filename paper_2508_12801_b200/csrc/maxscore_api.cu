// C ABI of the MaxScore router (see include/maxscore.h): argument checks, workspace carving and
// kernel launches on the caller's stream.  No device memory is allocated here.
#include "../../include/maxscore.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "common.cuh"
#include "flow.cuh"
#include "gate.cuh"
#include "move.cuh"
#include "softtopk.cuh"
#include "reroute.cuh"
#include "alg1.cuh"

using namespace msr;

namespace {

thread_local char g_last_error[256] = "";

maxscore_status cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
  return MAXSCORE_ERR_CUDA;
}
#define MS_CUDA(call)                                              \
  do {                                                             \
    cudaError_t e_ = (call);                                       \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);            \
  } while (0)
#define MS_LAUNCH_CHECK(name)                                      \
  do {                                                             \
    cudaError_t e_ = cudaGetLastError();                           \
    if (e_ != cudaSuccess) return cuda_fail(e_, name);             \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int32_t capacity_of(const maxscore_params& p) {
  if (p.capacity > 0) return p.capacity;
  // ceil(cf * T * k / E) with cf read as a multiple of 2^-20 (exact for 1.0, 1.25, 1.5, ...)
  const long long cfq = llround((double)p.capacity_factor * 1048576.0);
  const __int128 num = (__int128)cfq * p.T * p.k;
  const __int128 den = (__int128)1048576 * p.E;
  return (int32_t)((num + den - 1) / den);
}

struct Layout {          // byte offsets inside the workspace
  size_t state, aux, cand, rec_val, rec_meta, rec_pos, rec_bxc, rec_ndv, rec_off, rec_cnt, rec_aarg, rr_choice, rr_rank, rr_cnt, rr_base, rr_held, rr_dropped, rr_bc, rr_blk, rr_dtok, rr_order, rr_dnum, a1_v, a1_partial, a1_ticket, cache_x, cache_id, cache_bound, cache_raw, block_counts, wt, error_flag, dls, wk, dwpart, total;
  int Npad, n_idx_blocks;
  int rec_cap;                                // entries of the exact phase's candidate records
  int Kpad, dw_splits, dw_tokens_per_split;   // tensor-core backward GEMMs (bf16 I/O)
};

Layout layout_of(const maxscore_params& p) {
  Layout l{};
  l.Npad = (int)align_up((size_t)p.E, 16);
  l.n_idx_blocks = (p.T + kIdxTok - 1) / kIdxTok;
  size_t off = 0;
  l.state = off; off = align_up(off + sizeof(FlowState), 256);
  l.error_flag = off; off = align_up(off + 16, 256);
  l.aux = off; off = align_up(off + sizeof(double) * kMaxE + 16, 256);     // column sums + ticket of the auxiliary loss
  l.cand = off; off = align_up(off + sizeof(int32_t) * (size_t)p.T, 256);
  {   // candidate records of the exact phase: room for every (token, expert) pair, which the last, unbounded round
      // of a heavily tied problem can need (26 bytes each); beyond 2^21 entries the list is cut short
    long long cap = (long long)p.T * p.E;
    if (cap > (1LL << 21)) cap = 1LL << 21;
    l.rec_cap = (int)cap;
  }
  l.rec_val = off; off = align_up(off + sizeof(long long) * (size_t)l.rec_cap, 256);
  l.rec_meta = off; off = align_up(off + sizeof(unsigned short) * (size_t)l.rec_cap, 256);
  l.rec_pos = off; off = align_up(off + sizeof(int32_t) * (size_t)l.rec_cap, 256);
  l.rec_bxc = off; off = align_up(off + sizeof(int32_t) * (size_t)l.rec_cap, 256);
  l.rec_ndv = off; off = align_up(off + sizeof(long long) * (size_t)l.rec_cap, 256);
  l.rec_off = off; off = align_up(off + sizeof(int32_t) * (size_t)p.T, 256);
  l.rec_cnt = off; off = align_up(off + sizeof(int32_t) * (size_t)p.T, 256);
  l.rec_aarg = off; off = align_up(off + sizeof(int32_t) * (size_t)p.T, 256);
  // iterative rerouting (maxscore_assign_iterative)
  l.rr_choice = off; off = align_up(off + sizeof(int32_t) * (size_t)p.k * p.T, 256);
  l.rr_rank = off; off = align_up(off + sizeof(int32_t) * (size_t)p.k * p.T, 256);
  l.rr_cnt = off; off = align_up(off + sizeof(int32_t) * (size_t)p.k * p.E, 256);
  l.rr_base = off; off = align_up(off + sizeof(int32_t) * (size_t)(p.k + 1) * p.E, 256);
  l.rr_held = off; off = align_up(off + sizeof(uint4) * (size_t)p.T, 256);
  l.rr_dropped = off; off = align_up(off + (size_t)p.T, 256);
  l.rr_bc = off; off = align_up(off + sizeof(int32_t) * (((size_t)p.k * p.T + kIdxTok - 1) / kIdxTok) * p.E, 256);
  l.rr_blk = off; off = align_up(off + sizeof(int32_t) * (2 * (((size_t)p.T + kRrTokBlock - 1) / kRrTokBlock) + 1), 256);
  l.rr_dtok = off; off = align_up(off + sizeof(int32_t) * (size_t)p.T, 256);
  l.rr_order = off; off = align_up(off + (size_t)kRrRow * p.T, 256);
  l.rr_dnum = off; off = align_up(off + (size_t)p.T, 256);
  // Algorithm 1 (maxscore_assign_top2_sinkhorn); its per-token and per-expert integers reuse the rerouting arrays
  l.a1_v = off; off = align_up(off + sizeof(double) * kMaxE, 256);
  l.a1_partial = off; off = align_up(off + sizeof(double) * (size_t)kAlg1Blocks * kMaxE, 256);
  l.a1_ticket = off; off = align_up(off + 16, 256);
  l.cache_x = off; off = align_up(off + sizeof(float) * (size_t)kCacheN * p.T, 256);
  l.cache_id = off; off = align_up(off + (size_t)kCacheN * p.T, 256);
  l.cache_bound = off; off = align_up(off + sizeof(long long) * (size_t)p.T, 256);
  l.cache_raw = off; off = align_up(off + (size_t)p.T, 256);
  l.block_counts = off; off = align_up(off + sizeof(int32_t) * (size_t)l.n_idx_blocks * p.E, 1024);
  l.wt = off;
  off = align_up(off + (p.io_dtype == MAXSCORE_BF16 ? sizeof(__nv_bfloat16) * (size_t)l.Npad * p.d_model : 0), 1024);
  l.Kpad = (int)align_up((size_t)p.E, 64);
  {   // split the token dimension of dW so that about two CTAs per SM are busy
    const int mtiles = (p.d_model + 127) / 128;
    int splits = 296 / mtiles;     // one CTA per SM (192 KB of shared memory): at most two full waves on 148 SMs
    const int max_splits = (p.T + 255) / 256;
    if (splits > max_splits) splits = max_splits;
    if (splits > 64) splits = 64;
    if (splits < 1) splits = 1;
    l.dw_tokens_per_split = (int)align_up((size_t)((p.T + splits - 1) / splits), 64);
    l.dw_splits = (p.T + l.dw_tokens_per_split - 1) / l.dw_tokens_per_split;
  }
  const bool bf = p.io_dtype == MAXSCORE_BF16;
  l.dls = off; off = align_up(off + (bf ? sizeof(__nv_bfloat16) * (size_t)p.T * 2 * l.Kpad : 0), 1024);
  l.wk = off; off = align_up(off + (bf ? sizeof(__nv_bfloat16) * (size_t)p.d_model * l.Kpad : 0), 1024);
  l.dwpart = off; off = align_up(off + (bf ? sizeof(float) * (size_t)l.dw_splits * p.d_model * p.E : 0), 1024);
  l.total = off;
  return l;
}

maxscore_status check_params(const maxscore_params* p) {
  if (!p) return MAXSCORE_ERR_INVALID_ARG;
  if (p->T <= 0 || p->d_model <= 0 || p->E <= 0 || p->k <= 0) return MAXSCORE_ERR_INVALID_ARG;
  if (!(p->t > 0.f) || !isfinite(p->t)) return MAXSCORE_ERR_INVALID_ARG;
  if (p->io_dtype != MAXSCORE_F32 && p->io_dtype != MAXSCORE_BF16) return MAXSCORE_ERR_INVALID_ARG;
  if (p->score_mode != 0 && p->score_mode != 1) return MAXSCORE_ERR_INVALID_ARG;
  if (p->w_gate_layout != 0 && p->w_gate_layout != 1) return MAXSCORE_ERR_INVALID_ARG;
  if (p->capacity <= 0 && !(p->capacity_factor > 0.f)) return MAXSCORE_ERR_INVALID_ARG;
  if (p->score_mode == 1 && (p->quant_shift < 0 || p->quant_shift > 14)) return MAXSCORE_ERR_INVALID_ARG;
  if (p->max_sweeps < 0) return MAXSCORE_ERR_INVALID_ARG;
  if (p->softtopk_mode < 0 || p->softtopk_mode > 2) return MAXSCORE_ERR_INVALID_ARG;
  if (p->softtopk_mode == 1 && (p->rankscale_delta < 0 || p->rankscale_delta > 1 || !isfinite(p->rankscale_beta)))
    return MAXSCORE_ERR_INVALID_ARG;
  if (p->k > p->E) return MAXSCORE_ERR_INFEASIBLE;
  if (p->E > kMaxE || p->k > kMaxK) return MAXSCORE_ERR_UNSUPPORTED;
  if ((long long)p->T * p->k >= (1LL << 31)) return MAXSCORE_ERR_UNSUPPORTED;
  if (p->io_dtype == MAXSCORE_BF16 && p->d_model % 8) return MAXSCORE_ERR_UNSUPPORTED;
  if (p->io_dtype == MAXSCORE_F32 && p->d_model % 4) return MAXSCORE_ERR_UNSUPPORTED;
  const long long C = capacity_of(*p);
  if (C <= 0 || C > (1LL << 30)) return MAXSCORE_ERR_INVALID_ARG;
  const long long cap = C < p->T ? C : p->T;
  if ((long long)p->E * cap < (long long)p->T * p->k) return MAXSCORE_ERR_INFEASIBLE;
  return MAXSCORE_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kDhSmemMax = 2 * 2 * 16384 + kDhStages * 2 * 16384 + kDhOutBytes + 1024;     // Kpad = 128
constexpr int kDwSmemMax = kDwStages * (16384 + 2 * 2 * 8192) + 1024;

}  // namespace

struct maxscore_ctx {
  maxscore_params p;
  int32_t C;
  Layout lay;
  char* ws;
  EncodeTiledFn encode;
  int sm_count;
  int sweep_grid_max;   // CTAs of the sweeps kernel that are resident at once
  long long launches;   // kernels launched through this context so far
  // host path (maxscore_route_dispatch_host): a copy stream and its events, made on the first call
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_start = nullptr, ev_routed = nullptr, ev_copied = nullptr, ev_chunk[8] = {};
};

namespace {

KeyGen keygen_of(const maxscore_ctx* c) {
  KeyGen g{};
  g.mode = c->p.score_mode;
  g.quant_shift = c->p.quant_shift;
  g.seed_mul = c->p.tiebreak_seed * 0x9E3779B9u;
  int s = 0;
  const long long n = (long long)c->p.T * c->p.k;
  while ((1LL << s) < n) ++s;
  g.S = 20 + s;
  g.fshift = ldexpf(1.f, g.quant_shift);
  g.fS = ldexpf(1.f, g.S);
  return g;
}

maxscore_status make_tmap_bf16(const maxscore_ctx* c, CUtensorMap* tm, const void* base, uint64_t inner,
                               uint64_t outer, uint32_t box_inner, uint32_t box_outer) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = c->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(g_last_error, sizeof(g_last_error), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return MAXSCORE_ERR_CUDA;
  }
  return MAXSCORE_OK;
}

unsigned* error_flag_of(const maxscore_ctx* c) { return reinterpret_cast<unsigned*>(c->ws + c->lay.error_flag); }
size_t elem_bytes(const maxscore_ctx* c) { return c->p.io_dtype == MAXSCORE_BF16 ? 2 : 4; }

// The gate GEMM of Eq. 2 in two steps, so that the host path can run it over row blocks as they arrive:
// the weight in the tile layout of the tensor-core kernel (bf16 only), then the rows [row0, row0 + rows).
maxscore_status launch_gate_prepare(maxscore_ctx* c, const void* w_gate, cudaStream_t st) {
  const maxscore_params& p = c->p;
  if (p.io_dtype == MAXSCORE_F32) return MAXSCORE_OK;
  __nv_bfloat16* wt = reinterpret_cast<__nv_bfloat16*>(c->ws + c->lay.wt);
  const int Npad = c->lay.Npad;
  const long long n = (long long)Npad * p.d_model;
  int blocks = (int)((n + 255) / 256); if (blocks > 1184) blocks = 1184;
  wgate_prepare_kernel<<<blocks, 256, 0, st>>>((const __nv_bfloat16*)w_gate, wt, p.d_model, p.E, Npad, p.w_gate_layout);
  MS_LAUNCH_CHECK("wgate_prepare_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status launch_gate_rows(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* bias, float* logits,
                                 int row0, int rows, cudaStream_t st) {
  const maxscore_params& p = c->p;
  float* out = logits + (size_t)row0 * p.E;
  if (p.io_dtype == MAXSCORE_F32) {
    dim3 grid((rows + 15) / 16, (p.E + 15) / 16);
    gate_gemm_simt_kernel<float><<<grid, 256, 0, st>>>((const float*)hidden + (size_t)row0 * p.d_model, (const float*)w_gate,
                                                        bias, out, rows, p.d_model, p.E, p.w_gate_layout);
    MS_LAUNCH_CHECK("gate_gemm_simt_kernel");
    c->launches += 1;
    return MAXSCORE_OK;
  }
  __nv_bfloat16* wt = reinterpret_cast<__nv_bfloat16*>(c->ws + c->lay.wt);
  const int Npad = c->lay.Npad;
  CUtensorMap tmH, tmW;
  maxscore_status s = make_tmap_bf16(c, &tmH, (const __nv_bfloat16*)hidden + (size_t)row0 * p.d_model, (uint64_t)p.d_model,
                                     (uint64_t)rows, kGateBK, kGateBM);
  if (s) return s;
  s = make_tmap_bf16(c, &tmW, wt, (uint64_t)p.d_model, (uint64_t)Npad, kGateBK, (uint32_t)Npad);
  if (s) return s;
  const int num_kb = (p.d_model + kGateBK - 1) / kGateBK;
  gate_gemm_tc_kernel<<<(rows + kGateBM - 1) / kGateBM, 128, kGateSmemBytes, st>>>(tmH, tmW, bias, out, rows, p.E, Npad, num_kb,
                                                                                  error_flag_of(c));
  MS_LAUNCH_CHECK("gate_gemm_tc_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status launch_gate(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* bias,
                            float* logits, cudaStream_t st) {
  maxscore_status s = launch_gate_prepare(c, w_gate, st);
  if (s) return s;
  return launch_gate_rows(c, hidden, w_gate, bias, logits, 0, c->p.T, st);
}

// SoftTopk (Eq. 6) or one of its variants over `rows` rows (every row is on its own).
maxscore_status launch_softtopk_rows(maxscore_ctx* c, const float* logits, float* scores, int rows, cudaStream_t st) {
  const maxscore_params& p = c->p;
  int blocks = (rows + 7) / 8; if (blocks > c->sm_count * 8) blocks = c->sm_count * 8;
  if (p.softtopk_mode == 2)
    itertopk_kernel<false><<<blocks, 256, 0, st>>>(logits, nullptr, nullptr, nullptr, scores, rows, p.E, p.k);
  else if (p.softtopk_mode == 1)
    softtopk_rankscale_kernel<false><<<blocks, 256, 0, st>>>(logits, nullptr, nullptr, nullptr, scores, rows, p.E, p.k, p.t,
                                                             p.rankscale_beta, p.rankscale_delta);
  else {
    const int tiles = (rows + kStTok - 1) / kStTok;
    const int grid = tiles < c->sm_count * 6 ? tiles : c->sm_count * 6;
    const size_t smem = sizeof(float) * (size_t)kStTok * st_stride(p.E);
    if (p.k <= 2) softtopk_fwd_kernel<2><<<grid, kStThreads, smem, st>>>(logits, scores, rows, p.E, p.k, p.t);
    else if (p.k <= 4) softtopk_fwd_kernel<4><<<grid, kStThreads, smem, st>>>(logits, scores, rows, p.E, p.k, p.t);
    else softtopk_fwd_kernel<8><<<grid, kStThreads, smem, st>>>(logits, scores, rows, p.E, p.k, p.t);
  }
  MS_LAUNCH_CHECK("softtopk_fwd_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status launch_softtopk_fwd(maxscore_ctx* c, const float* logits, float* scores, cudaStream_t st) {
  return launch_softtopk_rows(c, logits, scores, c->p.T, st);
}

// dl_split (may be null): the gradient also as hi + lo bf16 halves, in the layout the tensor-core gate backward reads
void launch_softtopk_bwd_tiles(maxscore_ctx* c, const float* logits, const int32_t* expert_idx, const float* dgate_w,
                               const float* dscores_col, float* dlogits, cudaStream_t st, __nv_bfloat16* dl_split = nullptr) {
  const maxscore_params& p = c->p;
  const int tiles = (p.T + kStTok - 1) / kStTok;
  const int grid = tiles < c->sm_count * 6 ? tiles : c->sm_count * 6;
  const size_t smem = sizeof(float) * ((size_t)kStTok * st_stride(p.E) + p.E);
  if (p.k <= 2)
    softtopk_bwd_kernel<2><<<grid, kStThreads, smem, st>>>(logits, expert_idx, dgate_w, dscores_col, dlogits, dl_split, c->lay.Kpad, p.T, p.E, p.k, p.t);
  else if (p.k <= 4)
    softtopk_bwd_kernel<4><<<grid, kStThreads, smem, st>>>(logits, expert_idx, dgate_w, dscores_col, dlogits, dl_split, c->lay.Kpad, p.T, p.E, p.k, p.t);
  else
    softtopk_bwd_kernel<8><<<grid, kStThreads, smem, st>>>(logits, expert_idx, dgate_w, dscores_col, dlogits, dl_split, c->lay.Kpad, p.T, p.E, p.k, p.t);
}

// rounds of (records, exact phase, check): candidate thresholds theta0, then two wider ones (four times the last, or twice
// the price spread that stopped the exact phase), then every token.  The documented workloads need one to three.
constexpr int kSweeps = 24, kRounds = 4, kDefaultAug = 4096;
// Dispatch through registers (dispatch_kernel, 0.91 of the copy peak on the stress shape) or through bulk copies
// (dispatch_tma_kernel, 0.86: the 8-to-1 write-heavy stream is bound by the memory system's write path either way).
// The bulk-copy variant is built with -DMAXSCORE_DISPATCH_TMA so that both can be profiled.
#ifdef MAXSCORE_DISPATCH_TMA
constexpr bool kDispatchByTma = true;
#else
constexpr bool kDispatchByTma = false;
#endif

maxscore_status launch_assign(maxscore_ctx* c, const float* M, int32_t* expert_idx, int32_t* expert_load,
                              maxscore_stats* stats, cudaStream_t st) {
  const maxscore_params& p = c->p;
  FlowState* fs = reinterpret_cast<FlowState*>(c->ws + c->lay.state);
  int32_t* cand = reinterpret_cast<int32_t*>(c->ws + c->lay.cand);
  KeyGen g = keygen_of(c);
  const int scale_bits = p.score_mode == 0 ? 40 : g.S + p.quant_shift;   // log2 of one unit of score
  const int budget = p.max_sweeps > 0 ? p.max_sweeps : kSweeps + kDefaultAug;
  SweepArgs a{};
  a.T = p.T; a.E = p.E; a.k = p.k; a.C = c->C;
  a.n_sweeps = budget < kSweeps ? budget : kSweeps;
  a.balanced = ((long long)p.E * c->C == (long long)p.T * p.k) ? 1 : 0;
  {   // a few units of spare room per expert at most: the sweeps hide them at first (see SweepArgs::slack).  With more
      // spare room than that the guess of who keeps it costs more repairs than the slow start it avoids.
    const long long spare = (long long)p.E * c->C - (long long)p.T * p.k;
    a.slack = (spare > 0 && spare <= 4LL * p.E) ? (int)spare : 0;
  }
  a.eps0 = 1LL << (scale_bits - 10);
  a.eps_min = p.score_mode == 0 ? (1LL << 20) : (1LL << 12);
  // first candidate threshold: 2^-14 of a unit of score.  Half of it lists fewer tokens but on the stress workload
  // often needs a second round (records, exact phase and check pass again); twice as much makes every search
  // round of the exact phase walk over twice as many records
  // (integer keys are logits, whose k-th and (k+1)-th values lie some twenty times further apart than those of the
  // scores, and whose ties the fp32 sweeps cannot tell apart: 2^-11 of a unit lists about as many tokens there)
  a.theta0 = 1LL << (scale_bits - (p.score_mode == 0 ? 14 : 11));
  int max_aug = budget - a.n_sweeps;

  flow_init_kernel<<<32, 256, 0, st>>>(fs, kCapLogMax, a.theta0, a.balanced, p.E);
  MS_LAUNCH_CHECK("flow_init_kernel");
  SweepCache cache{reinterpret_cast<float*>(c->ws + c->lay.cache_x), reinterpret_cast<unsigned char*>(c->ws + c->lay.cache_id),
                   reinterpret_cast<long long*>(c->ws + c->lay.cache_bound), reinterpret_cast<unsigned char*>(c->ws + c->lay.cache_raw)};
  const int warp_blocks = std::min((p.T + 7) / 8, c->sm_count * 8);       // kernels that give a warp to each token
  flow_scan_kernel<<<warp_blocks, 256, 0, st>>>(M, fs, cache, p.T, p.E, g);
  MS_LAUNCH_CHECK("flow_scan_kernel");
  {
    // cooperative launch: every CTA of the grid is resident, which the grid-wide barriers rely on
    int grid = std::min((p.T + kSwThreads - 1) / kSwThreads, c->sweep_grid_max);
    if (grid < 1) grid = 1;
    void* args[] = {(void*)&M, (void*)&fs, (void*)&cache, (void*)&expert_idx, (void*)&cand, (void*)&a, (void*)&g};
    MS_CUDA(cudaLaunchCooperativeKernel((const void*)flow_sweeps_kernel, dim3(grid), dim3(kSwThreads), args, 0, st));
  }
  Records rec{reinterpret_cast<long long*>(c->ws + c->lay.rec_val), reinterpret_cast<unsigned short*>(c->ws + c->lay.rec_meta),
              reinterpret_cast<int*>(c->ws + c->lay.rec_off), reinterpret_cast<int*>(c->ws + c->lay.rec_cnt),
              reinterpret_cast<int*>(c->ws + c->lay.rec_pos), reinterpret_cast<int*>(c->ws + c->lay.rec_bxc),
              reinterpret_cast<long long*>(c->ws + c->lay.rec_ndv), reinterpret_cast<int*>(c->ws + c->lay.rec_aarg), c->lay.rec_cap};
  const int build_blocks = c->sm_count * 4;
  const int check_blocks = std::min((p.T + 255) / 256, c->sm_count * 8);
  for (int r = 0; r < kRounds; ++r) {
    flow_records_kernel<<<build_blocks, 256, 0, st>>>(M, fs, expert_idx, cand, rec, p.T, p.E, p.k, g);
    MS_LAUNCH_CHECK("flow_records_kernel");
    flow_exact_kernel<true><<<1, kP2Threads, kRecSmemBytes, st>>>(fs, expert_idx, cand, rec, p.T, p.E, p.k, c->C, max_aug);
    flow_exact_kernel<false><<<1, kP2Threads, 0, st>>>(fs, expert_idx, cand, rec, p.T, p.E, p.k, c->C, max_aug);
    MS_LAUNCH_CHECK("flow_exact_kernel");
    flow_check_kernel<<<check_blocks, 256, 0, st>>>(M, fs, cache, expert_idx, cand, p.T, p.E, p.k, c->C, g, r == kRounds - 1,
                                                   r == kRounds - 2, expert_load, stats, error_flag_of(c));
    MS_LAUNCH_CHECK("flow_check_kernel");
  }
  // the last check pass has folded the internal-error flag into stats.status: start the next call clean
  MS_CUDA(cudaMemsetAsync(error_flag_of(c), 0, sizeof(unsigned), st));
  c->launches += 3 + 4 * kRounds;
  return MAXSCORE_OK;
}

maxscore_status launch_index_build(maxscore_ctx* c, const int32_t* expert_idx, int32_t* slot_idx, int32_t* slot_token,
                                   int32_t* expert_load, cudaStream_t st, const float* scores = nullptr,
                                   float* gate_w = nullptr) {
  const maxscore_params& p = c->p;
  int32_t* bc = reinterpret_cast<int32_t*>(c->ws + c->lay.block_counts);
  MS_CUDA(cudaMemsetAsync(slot_token, 0xFF, sizeof(int32_t) * (size_t)p.E * c->C, st));
  index_count_kernel<<<c->lay.n_idx_blocks, kIdxTok, 0, st>>>(expert_idx, bc, p.T, p.E, p.k);
  MS_LAUNCH_CHECK("index_count_kernel");
  index_fill_kernel<<<c->lay.n_idx_blocks, kIdxTok, 0, st>>>(expert_idx, bc, slot_idx, slot_token, expert_load, p.T,
                                                            p.E, p.k, c->C, scores, gate_w);
  MS_LAUNCH_CHECK("index_fill_kernel");
  c->launches += 2;
  return MAXSCORE_OK;
}

constexpr int kHostChunks = 8, kHostChunkMinRows = 1024;     // row blocks of the host path, and the smallest worth a copy
maxscore_status host_path_streams(maxscore_ctx* c) {
  static_assert(sizeof(c->ev_chunk) / sizeof(c->ev_chunk[0]) == kHostChunks, "one event per row block");
  if (c->copy_stream) return MAXSCORE_OK;
  MS_CUDA(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
  MS_CUDA(cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming));
  MS_CUDA(cudaEventCreateWithFlags(&c->ev_routed, cudaEventDisableTiming));
  MS_CUDA(cudaEventCreateWithFlags(&c->ev_copied, cudaEventDisableTiming));
  for (int i = 0; i < kHostChunks; ++i) MS_CUDA(cudaEventCreateWithFlags(&c->ev_chunk[i], cudaEventDisableTiming));
  return MAXSCORE_OK;
}

// The part of the forward route that needs every token's scores: assignment, slots, gate weights.
maxscore_status route_after_scores(maxscore_ctx* c, const float* logits, const float* scores, int32_t* expert_idx,
                                   int32_t* slot_idx, float* gate_w, int32_t* slot_token, int32_t* expert_load,
                                   maxscore_stats* stats, cudaStream_t st) {
  maxscore_status s = launch_assign(c, c->p.score_mode == 0 ? scores : logits, expert_idx, expert_load, stats, st);
  if (s) return s;
  // slots and, in the same pass over expert_idx, the combine weights gate_w[i, c] = scores[i, expert_idx[i, c]]
  s = launch_index_build(c, expert_idx, slot_idx, slot_token, expert_load, st, scores, gate_w);
  if (s) return s;
  return MAXSCORE_OK;
}

maxscore_status launch_zero_padding(maxscore_ctx* c, const int32_t* slot_token, void* dst, cudaStream_t st) {
  const long long n_slots = (long long)c->p.E * c->C;
  int blocks = (int)((n_slots + 7) / 8); if (blocks > c->sm_count * 8) blocks = c->sm_count * 8;
  zero_padding_kernel<<<blocks, 256, 0, st>>>(slot_token, (char*)dst, n_slots, (uint32_t)(c->p.d_model * elem_bytes(c)));
  MS_LAUNCH_CHECK("zero_padding_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

}  // namespace

// ==================================================================================================
extern "C" {

int32_t maxscore_capacity(const maxscore_params* params) {
  if (!params || params->E <= 0) return -1;
  return capacity_of(*params);
}

const char* maxscore_last_cuda_error(void) { return g_last_error; }

maxscore_status maxscore_workspace_bytes(const maxscore_params* params, size_t* bytes) {
  if (!bytes) return MAXSCORE_ERR_INVALID_ARG;
  maxscore_status s = check_params(params);
  if (s) return s;
  *bytes = layout_of(*params).total;
  return MAXSCORE_OK;
}

maxscore_status maxscore_create(maxscore_ctx** out, const maxscore_params* params, void* workspace,
                                size_t workspace_bytes) {
  if (!out) return MAXSCORE_ERR_INVALID_ARG;
  *out = nullptr;
  maxscore_status s = check_params(params);
  if (s) return s;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MAXSCORE_ERR_INVALID_ARG;
  const Layout lay = layout_of(*params);
  if (workspace_bytes < lay.total) return MAXSCORE_ERR_WORKSPACE;
  int dev = 0, sms = 0;
  MS_CUDA(cudaGetDevice(&dev));
  MS_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  MS_CUDA(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) {
    snprintf(g_last_error, sizeof(g_last_error), "cuTensorMapEncodeTiled not available from the driver");
    return MAXSCORE_ERR_CUDA;
  }
  MS_CUDA(cudaFuncSetAttribute(gate_gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGateSmemBytes));
  {
    const int st_smem = (int)(sizeof(float) * ((size_t)kStTok * st_stride(kMaxE) + kMaxE));
    MS_CUDA(cudaFuncSetAttribute(softtopk_fwd_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, st_smem));
    MS_CUDA(cudaFuncSetAttribute(softtopk_fwd_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, st_smem));
    MS_CUDA(cudaFuncSetAttribute(softtopk_fwd_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, st_smem));
    MS_CUDA(cudaFuncSetAttribute(softtopk_bwd_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, st_smem));
    MS_CUDA(cudaFuncSetAttribute(softtopk_bwd_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, st_smem));
    MS_CUDA(cudaFuncSetAttribute(softtopk_bwd_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, st_smem));
  }
  MS_CUDA(cudaFuncSetAttribute(flow_exact_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRecSmemBytes));
  MS_CUDA(cudaFuncSetAttribute(gate_bwd_dh_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDhSmemMax));
  MS_CUDA(cudaFuncSetAttribute(gate_bwd_dw_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDwSmemMax));
  MS_CUDA(cudaFuncSetAttribute(dispatch_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTmaWarps * kTmaStages * kTmaChunk));
  int coop = 0, sweep_occ = 0;
  MS_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
  MS_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&sweep_occ, flow_sweeps_kernel, kSwThreads, 0));
  if (!coop || sweep_occ < 1) {
    snprintf(g_last_error, sizeof(g_last_error), "the device cannot launch the cooperative sweeps kernel");
    return MAXSCORE_ERR_CUDA;
  }
  MS_CUDA(cudaMemsetAsync(workspace, 0, lay.cand, 0));
  MS_CUDA(cudaStreamSynchronize(0));
  maxscore_ctx* c = new (std::nothrow) maxscore_ctx();
  if (!c) return MAXSCORE_ERR_INVALID_ARG;
  c->p = *params; c->C = capacity_of(*params); c->lay = lay; c->ws = static_cast<char*>(workspace);
  c->encode = reinterpret_cast<EncodeTiledFn>(fn); c->sm_count = sms;
  c->sweep_grid_max = sms * sweep_occ;
  c->launches = 0;
  *out = c;
  return MAXSCORE_OK;
}

void maxscore_destroy(maxscore_ctx* ctx) {
  if (!ctx) return;
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
  if (ctx->ev_routed) cudaEventDestroy(ctx->ev_routed);
  if (ctx->ev_copied) cudaEventDestroy(ctx->ev_copied);
  for (cudaEvent_t e : ctx->ev_chunk) if (e) cudaEventDestroy(e);
  delete ctx;
}

maxscore_status maxscore_gate(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* bias,
                              float* logits, void* stream) {
  if (!c || !hidden || !w_gate || !logits) return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(w_gate) || !aligned16(logits)) return MAXSCORE_ERR_INVALID_ARG;
  return launch_gate(c, hidden, w_gate, bias, logits, (cudaStream_t)stream);
}

maxscore_status maxscore_softtopk_fwd(maxscore_ctx* c, const float* logits, float* scores, void* stream) {
  if (!c || !logits || !scores) return MAXSCORE_ERR_INVALID_ARG;
  return launch_softtopk_fwd(c, logits, scores, (cudaStream_t)stream);
}

maxscore_status maxscore_softtopk_bwd(maxscore_ctx* c, const float* logits, const int32_t* expert_idx,
                                      const float* dgate_w, float* dlogits, void* stream) {
  if (!c || !logits || !expert_idx || !dgate_w || !dlogits) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  int blocks = (p.T + 7) / 8; if (blocks > c->sm_count * 8) blocks = c->sm_count * 8;
  if (p.softtopk_mode == 2)
    itertopk_kernel<true><<<blocks, 256, 0, (cudaStream_t)stream>>>(logits, expert_idx, dgate_w, nullptr, dlogits, p.T, p.E, p.k);
  else if (p.softtopk_mode == 1)
    softtopk_rankscale_kernel<true><<<blocks, 256, 0, (cudaStream_t)stream>>>(logits, expert_idx, dgate_w, nullptr, dlogits, p.T,
                                                                             p.E, p.k, p.t, p.rankscale_beta, p.rankscale_delta);
  else
    launch_softtopk_bwd_tiles(c, logits, expert_idx, dgate_w, nullptr, dlogits, (cudaStream_t)stream);
  MS_LAUNCH_CHECK("softtopk_bwd_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status maxscore_softtopk_bwd_aux(maxscore_ctx* c, const float* logits, const int32_t* expert_idx,
                                          const float* dgate_w, const float* dscores_col, float* dlogits, void* stream) {
  if (!c || !logits || !expert_idx || !dgate_w || !dscores_col || !dlogits) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  int blocks = (p.T + 7) / 8; if (blocks > c->sm_count * 8) blocks = c->sm_count * 8;
  if (p.softtopk_mode == 2)
    itertopk_kernel<true><<<blocks, 256, 0, (cudaStream_t)stream>>>(logits, expert_idx, dgate_w, dscores_col, dlogits, p.T, p.E, p.k);
  else if (p.softtopk_mode == 1)
    softtopk_rankscale_kernel<true><<<blocks, 256, 0, (cudaStream_t)stream>>>(logits, expert_idx, dgate_w, dscores_col, dlogits,
                                                                             p.T, p.E, p.k, p.t, p.rankscale_beta, p.rankscale_delta);
  else
    launch_softtopk_bwd_tiles(c, logits, expert_idx, dgate_w, dscores_col, dlogits, (cudaStream_t)stream);
  MS_LAUNCH_CHECK("softtopk_bwd_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status maxscore_aux_loss(maxscore_ctx* c, const float* scores, const int32_t* expert_load, float lambda,
                                  double* loss, float* dscores_col, void* stream) {
  if (!c || !scores || !expert_load || !loss || !dscores_col) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  double* colsum = reinterpret_cast<double*>(c->ws + c->lay.aux);
  unsigned* ticket = reinterpret_cast<unsigned*>(c->ws + c->lay.aux + sizeof(double) * kMaxE);
  int blocks = (p.T + 7) / 8; if (blocks > c->sm_count * 4) blocks = c->sm_count * 4;
  aux_loss_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(scores, expert_load, colsum, ticket, loss, dscores_col, p.T, p.E, lambda);
  MS_LAUNCH_CHECK("aux_loss_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status maxscore_assign(maxscore_ctx* c, const float* matrix, int32_t* expert_idx, int32_t* expert_load,
                                maxscore_stats* stats, void* stream) {
  if (!c || !matrix || !expert_idx || !expert_load || !stats) return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(matrix)) return MAXSCORE_ERR_INVALID_ARG;
  return launch_assign(c, matrix, expert_idx, expert_load, stats, (cudaStream_t)stream);
}

maxscore_status maxscore_index_build(maxscore_ctx* c, const int32_t* expert_idx, int32_t* slot_idx,
                                     int32_t* slot_token, int32_t* expert_load, void* stream) {
  if (!c || !expert_idx || !slot_idx || !slot_token || !expert_load) return MAXSCORE_ERR_INVALID_ARG;
  return launch_index_build(c, expert_idx, slot_idx, slot_token, expert_load, (cudaStream_t)stream);
}

maxscore_status maxscore_route_fwd(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* bias,
                                   float* logits, float* scores, int32_t* expert_idx, int32_t* slot_idx,
                                   float* gate_w, int32_t* slot_token, int32_t* expert_load, maxscore_stats* stats,
                                   void* stream) {
  if (!c || !hidden || !w_gate || !logits || !scores || !expert_idx || !slot_idx || !gate_w || !slot_token ||
      !expert_load || !stats)
    return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(w_gate) || !aligned16(logits) || !aligned16(scores))
    return MAXSCORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  maxscore_status s = launch_gate(c, hidden, w_gate, bias, logits, st);
  if (s) return s;
  s = launch_softtopk_fwd(c, logits, scores, st);
  if (s) return s;
  return route_after_scores(c, logits, scores, expert_idx, slot_idx, gate_w, slot_token, expert_load, stats, st);
}

maxscore_status maxscore_dispatch(maxscore_ctx* c, const void* src, const int32_t* expert_idx,
                                  const int32_t* slot_idx, const int32_t* slot_token, void* dst, void* stream) {
  if (!c || !src || !expert_idx || !slot_idx || !slot_token || !dst) return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(src) || !aligned16(dst)) return MAXSCORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const maxscore_params& p = c->p;
  const uint32_t row_bytes = (uint32_t)(p.d_model * elem_bytes(c));
  if (kDispatchByTma) {
    const uint32_t chunk = row_bytes < (uint32_t)kTmaChunk ? row_bytes : (uint32_t)kTmaChunk;      // multiples of 16 bytes
    const size_t smem = (size_t)kTmaWarps * kTmaStages * chunk;
    dispatch_tma_kernel<<<c->sm_count, kTmaWarps * 32, smem, st>>>((const char*)src, expert_idx, slot_idx, (char*)dst, p.T,
                                                                  row_bytes, chunk, p.k, c->C, error_flag_of(c));
  } else {
    dispatch_kernel<<<c->sm_count * 8, 256, 0, st>>>((const char*)src, expert_idx, slot_idx, (char*)dst, p.T, row_bytes, p.k, c->C);
  }
  MS_LAUNCH_CHECK("dispatch_kernel");
  c->launches += 1;
  return launch_zero_padding(c, slot_token, dst, st);
}

maxscore_status maxscore_combine(maxscore_ctx* c, const void* src, const int32_t* expert_idx,
                                 const int32_t* slot_idx, const float* gate_w, void* dst, int accumulate,
                                 void* stream) {
  if (!c || !src || !expert_idx || !slot_idx || !dst) return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(src) || !aligned16(dst)) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  int blocks = (p.T + 7) / 8 < c->sm_count * 8 ? (p.T + 7) / 8 : c->sm_count * 8;   // a warp per token
  if (p.io_dtype == MAXSCORE_BF16)
    combine_kernel<__nv_bfloat16><<<blocks, 256, 0, (cudaStream_t)stream>>>(
        (const __nv_bfloat16*)src, expert_idx, slot_idx, gate_w, (__nv_bfloat16*)dst, p.T, p.d_model, p.k, c->C, accumulate);
  else
    combine_kernel<float><<<blocks, 256, 0, (cudaStream_t)stream>>>((const float*)src, expert_idx, slot_idx, gate_w,
                                                                     (float*)dst, p.T, p.d_model, p.k, c->C, accumulate);
  MS_LAUNCH_CHECK("combine_kernel");
  c->launches += 1;
  return MAXSCORE_OK;
}

maxscore_status maxscore_combine_bwd(maxscore_ctx* c, const void* dY, const void* yexp, const int32_t* expert_idx,
                                     const int32_t* slot_idx, const float* gate_w, const int32_t* slot_token,
                                     void* dyexp, float* dgate_w, void* stream) {
  if (!c || !dY || !yexp || !expert_idx || !slot_idx || !gate_w || !slot_token || !dyexp || !dgate_w)
    return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(yexp) || !aligned16(dyexp)) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  cudaStream_t st = (cudaStream_t)stream;
  int blocks = p.T < c->sm_count * 8 ? p.T : c->sm_count * 8;
  if (p.io_dtype == MAXSCORE_BF16)
    combine_bwd_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dY, (const __nv_bfloat16*)yexp,
                                                              expert_idx, slot_idx, gate_w, (__nv_bfloat16*)dyexp,
                                                              dgate_w, p.T, p.d_model, p.k, c->C);
  else
    combine_bwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)dY, (const float*)yexp, expert_idx, slot_idx, gate_w,
                                                      (float*)dyexp, dgate_w, p.T, p.d_model, p.k, c->C);
  MS_LAUNCH_CHECK("combine_bwd_kernel");
  c->launches += 1;
  return launch_zero_padding(c, slot_token, dyexp, st);
}

static maxscore_status gate_bwd_impl(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* dlogits,
                                     float* dw_gate, void* dH, void* stream, bool split_ready);

maxscore_status maxscore_gate_bwd(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* dlogits,
                                  float* dw_gate, void* dH, void* stream) {
  return gate_bwd_impl(c, hidden, w_gate, dlogits, dw_gate, dH, stream, false);
}

// split_ready: the hi/lo bf16 halves of dlogits are already in the workspace (written by the SoftTopk backward)
static maxscore_status gate_bwd_impl(maxscore_ctx* c, const void* hidden, const void* w_gate, const float* dlogits,
                                     float* dw_gate, void* dH, void* stream, bool split_ready) {
  if (!c || !hidden || !w_gate || !dlogits || !dw_gate || !dH) return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(w_gate) || !aligned16(dlogits) || !aligned16(dw_gate) || !aligned16(dH))
    return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  cudaStream_t st = (cudaStream_t)stream;
  if (p.io_dtype != MAXSCORE_BF16) MS_CUDA(cudaMemsetAsync(dw_gate, 0, sizeof(float) * (size_t)p.d_model * p.E, st));
  dim3 gw((p.d_model + 63) / 64, (p.T + kDwTok - 1) / kDwTok);
  const int gh = (p.T + 15) / 16;
  if (p.io_dtype == MAXSCORE_BF16) {
    const Layout& l = c->lay;
    __nv_bfloat16* dls = reinterpret_cast<__nv_bfloat16*>(c->ws + l.dls);
    __nv_bfloat16* wk = reinterpret_cast<__nv_bfloat16*>(c->ws + l.wk);
    float* part = reinterpret_cast<float*>(c->ws + l.dwpart);
    const int Kpad = l.Kpad;
    {
      long long n = (long long)p.T * Kpad;
      int blocks = (int)((n + 255) / 256); if (blocks > c->sm_count * 16) blocks = c->sm_count * 16;
      if (!split_ready) {
        split_dlogits_kernel<<<blocks, 256, 0, st>>>(dlogits, dls, p.T, p.E, Kpad);
        MS_LAUNCH_CHECK("split_dlogits_kernel");
        c->launches += 1;
      }
      n = (long long)p.d_model * Kpad;
      blocks = (int)((n + 255) / 256); if (blocks > c->sm_count * 16) blocks = c->sm_count * 16;
      wgate_kmajor_kernel<<<blocks, 256, 0, st>>>((const __nv_bfloat16*)w_gate, wk, p.d_model, p.E, Kpad, p.w_gate_layout);
      MS_LAUNCH_CHECK("wgate_kmajor_kernel");
    }
    CUtensorMap tmA, tmB, tmH2, tmL2;
    maxscore_status s2 = make_tmap_bf16(c, &tmA, dls, (uint64_t)2 * Kpad, (uint64_t)p.T, 64, 128);
    if (!s2) s2 = make_tmap_bf16(c, &tmB, wk, (uint64_t)Kpad, (uint64_t)p.d_model, 64, 128);
    if (!s2) s2 = make_tmap_bf16(c, &tmH2, hidden, (uint64_t)p.d_model, (uint64_t)p.T, 64, 64);
    if (!s2) s2 = make_tmap_bf16(c, &tmL2, dls, (uint64_t)2 * Kpad, (uint64_t)p.T, 64, 64);
    if (s2) return s2;
    const int kboxes = Kpad / 64;
    const size_t dh_smem = (size_t)2 * kboxes * 16384 + (size_t)kDhStages * kboxes * 16384 + (size_t)kDhOutBytes + 1024;
    CUtensorMap tmOut;
    s2 = make_tmap_bf16(c, &tmOut, dH, (uint64_t)p.d_model, (uint64_t)p.T, 64, 32);
    if (s2) return s2;
    gate_bwd_dh_tc_kernel<<<(p.T + 127) / 128, 192, dh_smem, st>>>(tmA, tmB, tmOut, p.T, p.d_model, Kpad, error_flag_of(c));
    MS_LAUNCH_CHECK("gate_bwd_dh_tc_kernel");
    const size_t dw_smem = (size_t)kDwStages * (16384 + (size_t)2 * kboxes * 8192) + 1024;
    dim3 gdw((p.d_model + 127) / 128, l.dw_splits);
    gate_bwd_dw_tc_kernel<<<gdw, 128, dw_smem, st>>>(tmH2, tmL2, part, p.T, p.d_model, p.E, Kpad, l.dw_tokens_per_split,
                                                    error_flag_of(c));
    MS_LAUNCH_CHECK("gate_bwd_dw_tc_kernel");
    const long long nw = (long long)p.d_model * p.E;
    int rblocks = (int)((nw + 255) / 256); if (rblocks > c->sm_count * 8) rblocks = c->sm_count * 8;
    reduce_dw_kernel<<<rblocks, 256, 0, st>>>(part, dw_gate, nw, l.dw_splits);
    c->launches += 4;
  } else {
    gate_bwd_dw_kernel<float><<<gw, 256, 0, st>>>((const float*)hidden, dlogits, dw_gate, p.T, p.d_model, p.E);
    MS_LAUNCH_CHECK("gate_bwd_dw_kernel");
    gate_bwd_dh_kernel<float><<<gh, 256, 0, st>>>(dlogits, (const float*)w_gate, (float*)dH, p.T, p.d_model, p.E,
                                                  p.w_gate_layout);
    c->launches += 2;
  }
  MS_LAUNCH_CHECK("gate_bwd_dh_kernel");
  return MAXSCORE_OK;
}

maxscore_status maxscore_route_bwd(maxscore_ctx* c, const void* dY, const void* yexp, const void* hidden,
                                   const void* w_gate, const float* logits, const int32_t* expert_idx,
                                   const int32_t* slot_idx, const float* gate_w, const int32_t* slot_token,
                                   void* dyexp, float* dgate_w, float* dlogits, float* dw_gate, void* dH,
                                   void* stream) {
  if (!logits || !dlogits) return MAXSCORE_ERR_INVALID_ARG;
  maxscore_status s = maxscore_combine_bwd(c, dY, yexp, expert_idx, slot_idx, gate_w, slot_token, dyexp, dgate_w, stream);
  if (s) return s;
  if (c->p.io_dtype == MAXSCORE_BF16 && c->p.softtopk_mode == 0) {
    // the SoftTopk backward also leaves its result as the hi/lo bf16 halves that the tensor-core gate backward reads
    if (!expert_idx || !dgate_w) return MAXSCORE_ERR_INVALID_ARG;
    launch_softtopk_bwd_tiles(c, logits, expert_idx, dgate_w, nullptr, dlogits, (cudaStream_t)stream,
                              reinterpret_cast<__nv_bfloat16*>(c->ws + c->lay.dls));
    MS_LAUNCH_CHECK("softtopk_bwd_kernel");
    c->launches += 1;
    return gate_bwd_impl(c, hidden, w_gate, dlogits, dw_gate, dH, stream, true);
  }
  s = maxscore_softtopk_bwd(c, logits, expert_idx, dgate_w, dlogits, stream);
  if (s) return s;
  return maxscore_gate_bwd(c, hidden, w_gate, dlogits, dw_gate, dH, stream);
}

maxscore_status maxscore_assign_iterative(maxscore_ctx* c, const float* scores, int32_t* expert_idx, int32_t* expert_load,
                                          int32_t* counts, void* stream) {
  if (!c || !scores || !expert_idx || !expert_load || !counts) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t* choice = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_choice);      // [k][T], level-major
  int32_t* rank = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_rank);          // [k][T]
  int32_t* total = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_cnt);          // [E] pairs that chose the expert
  uint4* held = reinterpret_cast<uint4*>(c->ws + c->lay.rr_held);
  unsigned char* dropped = reinterpret_cast<unsigned char*>(c->ws + c->lay.rr_dropped);
  int32_t* bc = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_bc);
  const int nblk = (p.T + kRrTokBlock - 1) / kRrTokBlock;
  int32_t* blk_cnt = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_blk);        // [nblk]
  int32_t* blk_off = blk_cnt + nblk;                                           // [nblk + 1]
  int32_t* dtok = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_dtok);
  unsigned char* order = reinterpret_cast<unsigned char*>(c->ws + c->lay.rr_order);     // [T][kRrRow]
  unsigned char* dnum = reinterpret_cast<unsigned char*>(c->ws + c->lay.rr_dnum);
  MS_CUDA(cudaMemsetAsync(counts, 0, 2 * sizeof(int32_t), st));
  const int warp_blocks = std::min((p.T + 7) / 8, c->sm_count * 8);
  reroute_choices_kernel<<<warp_blocks, 256, 0, st>>>(scores, choice, p.T, p.E, p.k);
  MS_LAUNCH_CHECK("reroute_choices_kernel");
  // rank of every pair among the pairs of its expert in level-major order: the choice array as k*T tokens of one expert each
  const int flat = p.T * p.k;
  const int flat_blocks = (flat + kIdxTok - 1) / kIdxTok;
  index_count_kernel<<<flat_blocks, kIdxTok, 0, st>>>(choice, bc, flat, p.E, 1);
  index_fill_kernel<<<flat_blocks, kIdxTok, 0, st>>>(choice, bc, rank, choice, total, flat, p.E, 1, 0);
  MS_LAUNCH_CHECK("index_fill_kernel(levels)");
  reroute_accept_kernel<<<nblk, kRrTokBlock, 0, st>>>(choice, rank, held, dropped, blk_cnt, counts, p.T, p.E, p.k, c->C);
  reroute_scan_kernel<<<1, 1024, 0, st>>>(blk_cnt, blk_off, nblk);
  reroute_compact_kernel<<<nblk, kRrTokBlock, 0, st>>>(dropped, blk_off, dtok, dnum, p.T);
  reroute_order_kernel<<<c->sm_count * 4, 256, 0, st>>>(scores, total, held, blk_off + nblk, dtok, order, p.E, c->C);
  reroute_place_kernel<<<1, kRrThreads, 0, st>>>(total, held, blk_off + nblk, dtok, dnum, order, expert_load, counts, p.E, c->C);
  const int tok_blocks = std::min((p.T + 255) / 256, c->sm_count * 8);
  reroute_write_kernel<<<tok_blocks, 256, 0, st>>>(held, expert_idx, p.T, p.k);
  MS_LAUNCH_CHECK("reroute kernels");
  c->launches += 9;
  return MAXSCORE_OK;
}

maxscore_status maxscore_assign_top2_sinkhorn(maxscore_ctx* c, const float* scores, float sinkhorn_eps, int32_t sinkhorn_iters,
                                              int32_t* expert_idx, int32_t* expert_load, double* plan, int32_t* counts,
                                              void* stream) {
  if (!c || !scores || !expert_idx || !expert_load || !counts) return MAXSCORE_ERR_INVALID_ARG;
  if (!(sinkhorn_eps > 0.f) || !isfinite(sinkhorn_eps) || sinkhorn_iters < 0) return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  if (p.k != 2) return MAXSCORE_ERR_UNSUPPORTED;            // Algorithm 1 is stated for top-2
  cudaStream_t st = (cudaStream_t)stream;
  int32_t* first = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_choice);           // [T]
  int32_t* second = first + p.T;                                                   // [T]
  int32_t* rank = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_rank);              // [T]
  int32_t* cnt = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_cnt);                // [E]
  int32_t* resid = reinterpret_cast<int32_t*>(c->ws + c->lay.rr_base);             // [E]
  int32_t* cnt2 = resid + p.E;                                                     // [E]
  double* v = reinterpret_cast<double*>(c->ws + c->lay.a1_v);
  double* partial = reinterpret_cast<double*>(c->ws + c->lay.a1_partial);
  unsigned* ticket = reinterpret_cast<unsigned*>(c->ws + c->lay.a1_ticket);
  int32_t* bc = reinterpret_cast<int32_t*>(c->ws + c->lay.block_counts);
  MS_CUDA(cudaMemsetAsync(counts, 0, 2 * sizeof(int32_t), st));
  MS_CUDA(cudaMemsetAsync(cnt, 0, sizeof(int32_t) * p.E, st));
  MS_CUDA(cudaMemsetAsync(expert_load, 0, sizeof(int32_t) * p.E, st));
  MS_CUDA(cudaMemsetAsync(ticket, 0, sizeof(unsigned), st));
  const int warp_blocks = std::min((p.T + 7) / 8, c->sm_count * 8);
  alg1_top1_kernel<<<warp_blocks, 256, 0, st>>>(scores, first, cnt, p.T, p.E);
  alg1_resid_kernel<<<1, 128, 0, st>>>(cnt, resid, v, counts, p.E, c->C);
  MS_LAUNCH_CHECK("alg1_top1_kernel");
  const double inv_eps = 1.0 / (double)sinkhorn_eps;
  const int sk_blocks = std::min(kAlg1Blocks, (p.T + kAlg1Threads / 32 - 1) / (kAlg1Threads / 32));
  for (int it = 0; it < sinkhorn_iters; ++it)
    alg1_sinkhorn_kernel<<<sk_blocks, kAlg1Threads, 0, st>>>(scores, first, resid, v, partial, ticket, p.T, p.E, inv_eps);
  MS_LAUNCH_CHECK("alg1_sinkhorn_kernel");
  alg1_round_kernel<<<warp_blocks, 256, 0, st>>>(scores, first, v, second, plan, p.T, p.E, inv_eps);
  index_count_kernel<<<c->lay.n_idx_blocks, kIdxTok, 0, st>>>(second, bc, p.T, p.E, 1);
  index_fill_kernel<<<c->lay.n_idx_blocks, kIdxTok, 0, st>>>(second, bc, rank, first, cnt2, p.T, p.E, 1, 0);
  const int tok_blocks = std::min((p.T + 255) / 256, c->sm_count * 8);
  alg1_finish_kernel<<<tok_blocks, 256, 0, st>>>(first, second, rank, resid, expert_idx, expert_load, counts, p.T, p.E);
  MS_LAUNCH_CHECK("alg1_finish_kernel");
  c->launches += 6 + sinkhorn_iters;
  return MAXSCORE_OK;
}

long long maxscore_launch_count(const maxscore_ctx* c) { return c ? c->launches : -1; }

maxscore_status maxscore_check_internal(maxscore_ctx* c, uint32_t* flag_out, void* stream) {
  if (!c || !flag_out) return MAXSCORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned v = 0;
  MS_CUDA(cudaMemcpyAsync(&v, error_flag_of(c), sizeof(unsigned), cudaMemcpyDeviceToHost, st));
  MS_CUDA(cudaMemsetAsync(error_flag_of(c), 0, sizeof(unsigned), st));
  MS_CUDA(cudaStreamSynchronize(st));
  *flag_out = v;
  return MAXSCORE_OK;
}

maxscore_status maxscore_test_raise_internal(maxscore_ctx* c, void* stream) {
  if (!c) return MAXSCORE_ERR_INVALID_ARG;
  // every byte 1: any non-zero word reads as "a bounded wait gave up"
  MS_CUDA(cudaMemsetAsync(error_flag_of(c), 1, sizeof(unsigned), (cudaStream_t)stream));
  return MAXSCORE_OK;
}

maxscore_status maxscore_route_dispatch_host(maxscore_ctx* c, const void* hidden_host, const void* w_gate_host,
                                             const float* bias_host, const maxscore_device_buffers* dev,
                                             int32_t* expert_idx_host, int32_t* slot_idx_host, float* gate_w_host,
                                             maxscore_stats* stats_host, void* stream) {
  if (!c || !hidden_host || !w_gate_host || !dev || !expert_idx_host || !slot_idx_host || !gate_w_host || !stats_host)
    return MAXSCORE_ERR_INVALID_ARG;
  if (!dev->hidden || !dev->w_gate || !dev->xdisp || (bias_host && !dev->expert_bias)) return MAXSCORE_ERR_INVALID_ARG;
  if (!aligned16(dev->hidden) || !aligned16(dev->w_gate) || !aligned16(dev->logits) || !aligned16(dev->scores) ||
      !aligned16(dev->xdisp))
    return MAXSCORE_ERR_INVALID_ARG;
  const maxscore_params& p = c->p;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t eb = elem_bytes(c);
  maxscore_status s = host_path_streams(c);
  if (s) return s;
  cudaStream_t cs = c->copy_stream;
  // The token rows go up in blocks on a second stream; the gate GEMM and SoftTopk of a block start when it has
  // landed, so only the last block's share of them is left when the copy ends.  The assignment needs every row.
  MS_CUDA(cudaMemcpyAsync(dev->w_gate, w_gate_host, eb * (size_t)p.d_model * p.E, cudaMemcpyHostToDevice, st));
  if (bias_host) MS_CUDA(cudaMemcpyAsync(dev->expert_bias, bias_host, sizeof(float) * p.E, cudaMemcpyHostToDevice, st));
  s = launch_gate_prepare(c, dev->w_gate, st);
  if (s) return s;
  MS_CUDA(cudaEventRecord(c->ev_start, st));          // what ran before on the caller's stream may still read dev->hidden
  MS_CUDA(cudaStreamWaitEvent(cs, c->ev_start, 0));
  int nchunks = p.T / kHostChunkMinRows < kHostChunks ? p.T / kHostChunkMinRows : kHostChunks;
  if (nchunks < 1) nchunks = 1;
  const int rows_per = (int)align_up((size_t)((p.T + nchunks - 1) / nchunks), 128);
  const float* bias_dev = bias_host ? dev->expert_bias : nullptr;
  for (int i = 0, row0 = 0; row0 < p.T; ++i, row0 += rows_per) {
    const int rows = p.T - row0 < rows_per ? p.T - row0 : rows_per;
    const size_t off = eb * (size_t)row0 * p.d_model;
    MS_CUDA(cudaMemcpyAsync((char*)dev->hidden + off, (const char*)hidden_host + off, eb * (size_t)rows * p.d_model,
                            cudaMemcpyHostToDevice, cs));
    MS_CUDA(cudaEventRecord(c->ev_chunk[i], cs));
    MS_CUDA(cudaStreamWaitEvent(st, c->ev_chunk[i], 0));
    s = launch_gate_rows(c, dev->hidden, dev->w_gate, bias_dev, dev->logits, row0, rows, st);
    if (s) return s;
    s = launch_softtopk_rows(c, dev->logits + (size_t)row0 * p.E, dev->scores + (size_t)row0 * p.E, rows, st);
    if (s) return s;
  }
  s = route_after_scores(c, dev->logits, dev->scores, dev->expert_idx, dev->slot_idx, dev->gate_w, dev->slot_token,
                         dev->expert_load, dev->stats, st);
  if (s) return s;
  // the indices go back on the copy stream while the rows are dispatched
  MS_CUDA(cudaEventRecord(c->ev_routed, st));
  MS_CUDA(cudaStreamWaitEvent(cs, c->ev_routed, 0));
  const size_t nk = (size_t)p.T * p.k;
  MS_CUDA(cudaMemcpyAsync(expert_idx_host, dev->expert_idx, sizeof(int32_t) * nk, cudaMemcpyDeviceToHost, cs));
  MS_CUDA(cudaMemcpyAsync(slot_idx_host, dev->slot_idx, sizeof(int32_t) * nk, cudaMemcpyDeviceToHost, cs));
  MS_CUDA(cudaMemcpyAsync(gate_w_host, dev->gate_w, sizeof(float) * nk, cudaMemcpyDeviceToHost, cs));
  MS_CUDA(cudaMemcpyAsync(stats_host, dev->stats, sizeof(maxscore_stats), cudaMemcpyDeviceToHost, cs));
  MS_CUDA(cudaEventRecord(c->ev_copied, cs));
  s = maxscore_dispatch(c, dev->hidden, dev->expert_idx, dev->slot_idx, dev->slot_token, dev->xdisp, stream);
  if (s) return s;
  MS_CUDA(cudaStreamWaitEvent(st, c->ev_copied, 0));   // later work on the caller's stream may overwrite the indices
  MS_CUDA(cudaStreamSynchronize(st));
  return MAXSCORE_OK;
}

}  // extern "C"

// ==================================================================================================
// Index build without a context or a workspace, for callers that cannot allocate device memory.
// The scratch of the two-pass index build (expert counts per block of kIdxTok tokens) is a fixed array
// in the device image.  In host code the array's name is only a handle: the device address each GPU
// gave it is fetched once per device with cudaGetSymbolAddress and handed to the kernels.
namespace {

constexpr int kNoAllocMaxBlocks = MAXSCORE_NOALLOC_MAX_T / kIdxTok;          // 1024 blocks
static __device__ __align__(256) int32_t g_noalloc_block_counts[kNoAllocMaxBlocks * kMaxE];   // 512 KiB

constexpr int kMaxDevices = 64;
int32_t* g_noalloc_scratch_ptr[kMaxDevices] = {};      // per device, filled on the first call there

maxscore_status noalloc_scratch(int32_t** out) {
  int dev = 0;
  MS_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return MAXSCORE_ERR_UNSUPPORTED;
  int32_t* p = __atomic_load_n(&g_noalloc_scratch_ptr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    void* addr = nullptr;
    MS_CUDA(cudaGetSymbolAddress(&addr, g_noalloc_block_counts));   // address on the current device
    p = static_cast<int32_t*>(addr);
    __atomic_store_n(&g_noalloc_scratch_ptr[dev], p, __ATOMIC_RELEASE);   // racing first calls store the same value
  }
  *out = p;
  return MAXSCORE_OK;
}

}  // namespace

extern "C" maxscore_status maxscore_index_build_noalloc(int32_t T, int32_t E, int32_t k, int32_t C,
                                                        const int32_t* expert_idx, int32_t* slot_idx,
                                                        int32_t* slot_token, int32_t* expert_load,
                                                        void* cuda_stream) {
  if (!expert_idx || !slot_idx || !slot_token || !expert_load) return MAXSCORE_ERR_INVALID_ARG;
  if (T <= 0 || E <= 0 || k <= 0 || C <= 0) return MAXSCORE_ERR_INVALID_ARG;
  if (k > E) return MAXSCORE_ERR_INFEASIBLE;
  if (T > MAXSCORE_NOALLOC_MAX_T || E > kMaxE || k > kMaxK) {
    snprintf(g_last_error, sizeof(g_last_error),
             "maxscore_index_build_noalloc: T=%d E=%d k=%d exceeds the fixed scratch (T <= %d, E <= %d, k <= %d)",
             T, E, k, MAXSCORE_NOALLOC_MAX_T, kMaxE, kMaxK);
    return MAXSCORE_ERR_UNSUPPORTED;
  }
  int32_t* scratch = nullptr;
  maxscore_status s = noalloc_scratch(&scratch);
  if (s) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int blocks = (T + kIdxTok - 1) / kIdxTok;
  // every scratch entry the fill pass reads (blocks x E counts) is written by the count pass first,
  // so what an earlier call left in the array does not matter
  MS_CUDA(cudaMemsetAsync(slot_token, 0xFF, sizeof(int32_t) * (size_t)E * C, st));
  index_count_kernel<<<blocks, kIdxTok, 0, st>>>(expert_idx, scratch, T, E, k);
  MS_LAUNCH_CHECK("index_count_kernel");
  index_fill_kernel<<<blocks, kIdxTok, 0, st>>>(expert_idx, scratch, slot_idx, slot_token, expert_load, T, E, k, C);
  MS_LAUNCH_CHECK("index_fill_kernel");
  return MAXSCORE_OK;
}
