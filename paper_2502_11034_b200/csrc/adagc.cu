// Fused AdaGC + AdamW optimizer step for B200 (sm_100a): kernels and the C ABI of include/adagc.h.
//
// One step of Algorithm 1 of the paper is three phases on the caller's stream:
//   1. norm      every fixed-size chunk of every gradient tensor -> one float64 partial sum of
//                squares (Eq. 3 needs ||g_t,i||, Eq. 2 needs ||g_t||);
//   2. finalize  per tensor: fixed-order sum of its partials -> norm -> clip factor h, flag and the
//                gamma update (warm-up branch: global norm first, then min-seeding).  On AdaGC steps
//                this phase runs in the tail of the norm kernel, so a step is two launches;
//   3. update    every chunk again: g, theta, m, v read once, hat(g) = h * g kept on chip,
//                AdamW lines of Algorithm 1 (or Lion's rule, or momentum SGD), theta, m, v written
//                once; m and v are fp32 or bfloat16 arenas.  Two kernels: a bulk-async one
//                (cp.async.bulk + mbarrier ring through shared memory, the default) and a
//                register-streaming one.
// This is pure streaming work (18..28 bytes per parameter, ~20 flops): the bound is HBM bandwidth,
// so the kernels are built around large coalesced transfers, a measured amount of loads in flight
// per SM and streaming cache hints; there is no contraction here and tensor cores are not used.
//
// One translation unit in parts: adagc_common.cuh (constants, chunk-table entry, device helpers), adagc_norm.cuh
// (phase 1), adagc_decide.cuh (phase 2 and the norm kernel that carries it in its tail), adagc_update.cuh and
// adagc_update_bulk.cuh (phase 3), adagc_scale.cuh (clip-only), adagc_fused_small.cuh (the one-kernel step),
// adagc_tables.h (host: descriptor validation and the balanced per-block chunk tables built once at adagc_create);
// this file holds the context, the launch sequences, the entry points of include/adagc.h, and adagc_step_host,
// which pipelines groups of tensors behind the host-to-device copies.
//
// Reductions are deterministic: fixed element->thread mapping, fixed shuffle tree, fixed-order sums
// of partials; no floating-point atomics.  Sums of squares are accumulated in float64 so that the
// clip decision ||g|| > lambda_rel * gamma agrees with a float64 evaluation of the same predicate.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <cmath>
#include <functional>
#include <mutex>
#include <new>
#include <queue>
#include <type_traits>
#include <utility>
#include <vector>

#include "../../include/adagc.h"

#include "adagc_common.cuh"
#include "adagc_norm.cuh"
#include "adagc_decide.cuh"
#include "adagc_update.cuh"
#include "adagc_update_bulk.cuh"
#include "adagc_scale.cuh"
#include "adagc_fused_small.cuh"
#include "adagc_tables.h"

struct adagc_ctx {
  int32_t T = 0;
  int32_t n_chunks = 0;
  int64_t arena_elems = 0;
  bool bf16 = false;        // gradient arena is bfloat16
  bool state_bf16 = false;  // m and v arenas are bfloat16
  double lambda_abs = 1.0;
  int device = 0;
  int grid_wide = 1, grid_update = 1;  // norm and scale kernels: SMs x resident blocks; update: SMs x 2 or x 1
  bool update_bulk = false;            // update phase through the bulk-async (TMA) kernel
  bool sr_stochastic = false;          // adagc_set_state_rounding: bfloat16 moments rounded stochastically
  uint64_t sr_seed = 0;
  int64_t sr_step = 0;                 // step number of the launches being enqueued (part of the generator's counter)
  StateRounding rounding() const {
    StateRounding r;
    r.seed_lo = static_cast<uint32_t>(sr_seed);
    r.seed_hi = static_cast<uint32_t>(sr_seed >> 32);
    r.step_lo = static_cast<uint32_t>(sr_step);
    r.step_hi = static_cast<uint32_t>(static_cast<uint64_t>(sr_step) >> 32);
    r.stochastic = sr_stochastic ? 1 : 0;
    return r;
  }
  bool fold_finalize = true;           // AdaGC steps decide in the norm kernel's tail (needs every tensor to have a chunk)
  bool offsets_mult8 = true;           // every tensor offset is a multiple of 8 elements (bf16 arenas stay 16-byte aligned)
  bool keep_initial = false;           // ADAGC_EMA_KEEP_INITIAL
  bool global_adaptive = false;        // ADAGC_CLIP_GLOBAL_ADAPTIVE
  double ema_cap = 0.0;                // adagc_set_ema_cap: > 0 selects thresholded initialization
  bool fused_small = false;            // ADAGC_FUSED_SMALL: adagc_step runs as one cooperative kernel
  int grid_fused = 1;                  // its grid: every block resident at once
  unsigned long long barriers_done = 0;  // grid barriers executed by earlier fused launches of this context
  bool fused_poisoned = false;           // adagc_get_stats has seen ADAGC_E_TIMEOUT: the barrier counter is out of step
  char* ws = nullptr;
  Layout L{};
  uint64_t launches = 0;
  bool timing = false;
  bool timing_valid = false;
  cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
  struct Group {
    int64_t elem_begin = 0, elem_end = 0;  // arena range holding the group's tensors
    int32_t chunk_base = 0;                // first entry of the group in the grouped chunk tables
    int32_t order_first = 0, n_tensors = 0;
    int grid_wide = 1, grid_update = 1;
  };
  std::vector<Group> groups;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_entry = nullptr;
  std::vector<cudaEvent_t> ev_group;
  const Chunk* d_chunks_wide() const { return reinterpret_cast<const Chunk*>(ws + L.chunks_wide); }
  const Chunk* d_chunks_upd() const { return reinterpret_cast<const Chunk*>(ws + L.chunks_upd); }
  const int32_t* d_begin_wide() const { return reinterpret_cast<const int32_t*>(ws + L.begin_wide); }
  const int32_t* d_begin_upd() const { return reinterpret_cast<const int32_t*>(ws + L.begin_upd); }
  const int32_t* d_mid_upd() const { return reinterpret_cast<const int32_t*>(ws + L.mid_upd); }
  const TensorEntry* d_tensors() const { return reinterpret_cast<const TensorEntry*>(ws + L.tensors); }
  double* d_partials() const { return reinterpret_cast<double*>(ws + L.partials); }
  Guard guard() const {
    Guard g;
    g.arena_elems = arena_elems;
    g.n_chunks = n_chunks;
    g.n_tensors = T;
    g.status = reinterpret_cast<int*>(ws + L.scalars + 8);
    return g;
  }
  StatPtrs stats() const {
    StatPtrs s;
    s.sumsq = reinterpret_cast<double*>(ws + L.sumsq);
    s.norm = reinterpret_cast<float*>(ws + L.norm);
    s.h = reinterpret_cast<float*>(ws + L.h);
    s.flag = reinterpret_cast<uint8_t*>(ws + L.flag);
    s.clip_count = reinterpret_cast<unsigned long long*>(ws + L.clip_count);
    s.steps_done = reinterpret_cast<unsigned long long*>(ws + L.scalars);
    s.status = reinterpret_cast<int*>(ws + L.scalars + 8);
    return s;
  }
};

namespace {

int check_clip_args(adagc_ctx* ctx, const float* d_ema, int64_t step, double lambda_rel, double beta,
                    int64_t warmup) {
  if (!ctx || !d_ema) return ADAGC_E_INVALID_ARG;
  int dev = -1;  // the context's tables live on the device that was current at adagc_create
  if (cudaGetDevice(&dev) != cudaSuccess) return ADAGC_E_CUDA;
  if (dev != ctx->device) return ADAGC_E_INVALID_ARG;
  if (step < 1 || warmup < 0) return ADAGC_E_INVALID_ARG;
  if (!(lambda_rel > 0.0) || !std::isfinite(lambda_rel)) return ADAGC_E_INVALID_ARG;
  if (!(beta >= 0.0 && beta < 1.0)) return ADAGC_E_INVALID_ARG;
  ctx->sr_step = step;  // the launches that follow belong to this step
  return ADAGC_OK;
}

// Largest L1 carve-out for the register kernels (L1 lines hold their loads in flight); opt-in shared
// memory size for the bulk-async kernels.
template <bool kBF16, int kOpt, bool kSB>
bool prepare_update_kernel() {
  return cudaFuncSetAttribute(adagc_update_kernel<kBF16, kOpt, kSB>, cudaFuncAttributePreferredSharedMemoryCarveout,
                              cudaSharedmemCarveoutMaxL1) == cudaSuccess &&
         cudaFuncSetAttribute(adagc_update_tma_kernel<kBF16, kOpt, kSB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              tma_smem_bytes<kSB>(kBF16, kOpt, kOpt == kOptAdamW)) == cudaSuccess;
}
template <bool kBF16, bool kSB>
bool prepare_update_kernels() {
  return prepare_update_kernel<kBF16, kOptAdamW, kSB>() && prepare_update_kernel<kBF16, kOptLion, kSB>() &&
         prepare_update_kernel<kBF16, kOptSgdM, kSB>();
}

// One kernel's view of the chunk tables: the whole layout, or one group of the pipelined host step.
struct TableView {
  const Chunk* chunks;
  const int32_t* begin;
  const int32_t* mid;  // update tables only
  int grid;
};

// Launch with the programmatic-stream-serialization attribute: the kernel may be scheduled while the preceding kernel
// of the stream drains; it calls griddep_wait before it reads what that kernel wrote.
template <typename... Params, typename... Args>
void launch_dependent(void (*kernel)(Params...), int grid, int block, size_t smem, cudaStream_t s, bool programmatic,
                      Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);  // errors surface in finish_launches
}

template <bool kBF16, int kOpt, bool kSB>
void launch_update_t(adagc_ctx* ctx, const TableView& tv, float* p, const void* g, void* m, void* v,
                     const AdamScalars& a, cudaStream_t s, uint16_t* lowp, const AdamScalars* d_a) {
  const StatPtrs st = ctx->stats();
  // Only the bulk-async kernel is launched as a programmatic dependent (and not in the capturable step, which keeps
  // ordinary launches): its shared memory admits one block per SM, so blocks that become resident while the norm
  // kernel drains still end up one per SM.  The register kernel counts on exactly two blocks per SM; launched early,
  // its blocks pile onto the SMs that free up first (measured: 32.9 instead of 29.3 ms on the 7B-shaped layout).
  const bool programmatic = d_a == nullptr;
  if (ctx->update_bulk)
    launch_dependent(adagc_update_tma_kernel<kBF16, kOpt, kSB>, tv.grid, kTmaThreads,
                     tma_smem_bytes<kSB>(kBF16, kOpt, lowp != nullptr), s, programmatic, p, g, m, v, tv.chunks, tv.begin,
                     tv.mid, st.h, a, st.status, lowp, d_a, ctx->guard(), ctx->rounding());
  else
    launch_dependent(adagc_update_kernel<kBF16, kOpt, kSB>, tv.grid, kThreads, 0, s, false, p, g, m, v, tv.chunks,
                     tv.begin, st.h, a, lowp, d_a, ctx->guard(), ctx->rounding());
  ctx->launches++;
}

// The update phase over one table view, in the context's gradient and state dtypes.  m and v are fp32 or bfloat16
// arenas (adagc_desc.state_dtype); v is unused by Lion and momentum SGD.
template <int kOpt>
void launch_update(adagc_ctx* ctx, const TableView& tv, void* p, const void* g, void* m, void* v,
                   const AdamScalars& a, cudaStream_t s, void* lowp = nullptr, const AdamScalars* d_a = nullptr) {
  float* pf = static_cast<float*>(p);
  uint16_t* lp = static_cast<uint16_t*>(lowp);
  if (ctx->bf16) {
    if (ctx->state_bf16) launch_update_t<true, kOpt, true>(ctx, tv, pf, g, m, v, a, s, lp, d_a);
    else launch_update_t<true, kOpt, false>(ctx, tv, pf, g, m, v, a, s, lp, d_a);
  } else {
    if (ctx->state_bf16) launch_update_t<false, kOpt, true>(ctx, tv, pf, g, m, v, a, s, lp, d_a);
    else launch_update_t<false, kOpt, false>(ctx, tv, pf, g, m, v, a, s, lp, d_a);
  }
}

template <int kOpt>
void launch_update(adagc_ctx* ctx, void* p, const void* g, void* m, void* v, const AdamScalars& a,
                   cudaStream_t s, void* lowp = nullptr, const AdamScalars* d_a = nullptr) {
  const TableView tv = {ctx->d_chunks_upd(), ctx->d_begin_upd(), ctx->d_mid_upd(), ctx->grid_update};
  launch_update<kOpt>(ctx, tv, p, g, m, v, a, s, lowp, d_a);
}

void launch_norm(adagc_ctx* ctx, const TableView& tv, const void* d_grads, cudaStream_t s) {
  if (ctx->bf16)
    adagc_norm_kernel<true><<<tv.grid, kThreads, 0, s>>>(d_grads, tv.chunks, tv.begin, ctx->d_partials(), ctx->guard());
  else
    adagc_norm_kernel<false><<<tv.grid, kThreads, 0, s>>>(d_grads, tv.chunks, tv.begin, ctx->d_partials(), ctx->guard());
  ctx->launches++;
}

ClipScalars make_clip_scalars(const adagc_ctx* ctx, int64_t step, double lambda_rel, double beta) {
  ClipScalars cs;
  cs.lambda_rel = lambda_rel;
  cs.beta = beta;
  cs.one_minus_beta = 1.0 - beta;
  cs.lambda_abs = ctx->lambda_abs;
  cs.step = step;
  cs.n_tensors = ctx->T;
  cs.seed = (step == 1 && !ctx->keep_initial) ? 1 : 0;
  cs.ema_cap = ctx->ema_cap;
  return cs;
}

// scalar coefficients of the AdamW lines of Algorithm 1, in double, rounded once to the kernel's fp32
AdamScalars make_adam_scalars(int64_t step, double lr, double beta1, double beta2, double eps, double wd) {
  const double bc1 = 1.0 - std::pow(beta1, static_cast<double>(step));
  const double bc2 = 1.0 - std::pow(beta2, static_cast<double>(step));
  AdamScalars a;
  a.beta1 = static_cast<float>(beta1);
  a.one_minus_beta1 = static_cast<float>(1.0 - beta1);
  a.beta2 = static_cast<float>(beta2);
  a.one_minus_beta2 = static_cast<float>(1.0 - beta2);
  a.inv_bc2 = static_cast<float>(1.0 / bc2);
  a.step_size = static_cast<float>(lr / bc1);
  a.decay = static_cast<float>(1.0 - lr * wd);
  a.eps = static_cast<float>(eps);
  return a;
}

// need_arenas = false: the context holds no element (a rank of a sharded model that owns nothing), so the arena
// pointers are never dereferenced and may be anything, NULL included.
int check_adamw_args(const void* d_params, const void* d_grads, const void* d_m, const void* d_v, double lr,
                     double beta1, double beta2, double eps, double wd, bool need_arenas = true) {
  if (need_arenas && (!d_params || !d_grads || !d_m || !d_v)) return ADAGC_E_INVALID_ARG;
  if (!(beta1 >= 0.0 && beta1 < 1.0) || !(beta2 >= 0.0 && beta2 < 1.0)) return ADAGC_E_INVALID_ARG;
  if (!(eps >= 0.0) || !std::isfinite(eps) || !std::isfinite(lr) || !std::isfinite(wd)) return ADAGC_E_INVALID_ARG;
  if (need_arenas && (!aligned16(d_params) || !aligned16(d_grads) || !aligned16(d_m) || !aligned16(d_v)))
    return ADAGC_E_MISALIGNED;
  return ADAGC_OK;
}

// phases 1 and 2
int enqueue_clip_phases(adagc_ctx* ctx, const void* d_grads, float* d_ema, int64_t step, double lambda_rel,
                        double beta, int64_t warmup, cudaStream_t s) {
  if (ctx->timing) cudaEventRecord(ctx->ev[0], s);
  const TableView wide = {ctx->d_chunks_wide(), ctx->d_begin_wide(), nullptr, ctx->grid_wide};
  const ClipScalars cs = make_clip_scalars(ctx, step, lambda_rel, beta);
  const bool in_warmup = step <= warmup;
  const bool per_tensor = !in_warmup && !ctx->global_adaptive;
  if (per_tensor && ctx->fold_finalize) {
    // AdaGC step: a tensor's decision needs that tensor's partials only, so the block that completes a tensor takes it
    // at once: phases 1 and 2 are one launch
    unsigned int* tickets = reinterpret_cast<unsigned int*>(ctx->ws + ctx->L.tickets);
    const Chunk* in_order = reinterpret_cast<const Chunk*>(ctx->ws + ctx->L.chunks_range);
    const int32_t* ranges = reinterpret_cast<const int32_t*>(ctx->ws + ctx->L.begin_range);
    if (ctx->bf16)
      adagc_norm_decide_kernel<true><<<wide.grid, kThreads, 0, s>>>(d_grads, in_order, ranges, ctx->d_partials(),
                                                                  ctx->d_tensors(), tickets, cs, d_ema, ctx->stats(),
                                                                  ctx->guard());
    else
      adagc_norm_decide_kernel<false><<<wide.grid, kThreads, 0, s>>>(d_grads, in_order, ranges, ctx->d_partials(),
                                                                   ctx->d_tensors(), tickets, cs, d_ema, ctx->stats(),
                                                                   ctx->guard());
    ctx->launches++;
    if (ctx->timing) {
      cudaEventRecord(ctx->ev[1], s);
      cudaEventRecord(ctx->ev[2], s);  // no separate finalize phase
    }
    return ADAGC_OK;
  }
  launch_norm(ctx, wide, d_grads, s);
  if (ctx->timing) cudaEventRecord(ctx->ev[1], s);
  const int blocks = (ctx->T * 32 + kFinalizeThreads - 1) / kFinalizeThreads;
  adagc_tensor_finalize_kernel<<<blocks, kFinalizeThreads, 0, s>>>(ctx->d_partials(), ctx->d_tensors(), cs,
                                                                  per_tensor ? 1 : 0, d_ema, ctx->stats(), nullptr, 0,
                                                                  ctx->T, 1);
  ctx->launches++;
  if (ctx->global_adaptive) {
    adagc_global_finalize_kernel<<<1, kWarmupThreads, 0, s>>>(cs, in_warmup ? 1 : 0, d_ema, ctx->stats());
    ctx->launches++;
  } else if (in_warmup) {
    adagc_warmup_finalize_kernel<<<1, kWarmupThreads, 0, s>>>(cs, d_ema, ctx->stats());
    ctx->launches++;
  }
  if (ctx->timing) cudaEventRecord(ctx->ev[2], s);
  return ADAGC_OK;
}

// Phase 2 from per-tensor sums of squares the caller provides (already summed over the ranks of a sharded model).
void enqueue_presummed_phase(adagc_ctx* ctx, const double* d_sumsq, float* d_ema, int64_t step, double lambda_rel,
                             double beta, int64_t warmup, cudaStream_t s) {
  if (ctx->timing) {
    cudaEventRecord(ctx->ev[0], s);
    cudaEventRecord(ctx->ev[1], s);  // no norm phase in this call
  }
  const ClipScalars cs = make_clip_scalars(ctx, step, lambda_rel, beta);
  const bool in_warmup = step <= warmup;
  const bool per_tensor = !in_warmup && !ctx->global_adaptive;
  const int blocks = (ctx->T + kFinalizeThreads - 1) / kFinalizeThreads;
  adagc_presummed_finalize_kernel<<<blocks, kFinalizeThreads, 0, s>>>(d_sumsq, cs, per_tensor ? 1 : 0, d_ema,
                                                                     ctx->stats());
  ctx->launches++;
  if (ctx->global_adaptive) {
    adagc_global_finalize_kernel<<<1, kWarmupThreads, 0, s>>>(cs, in_warmup ? 1 : 0, d_ema, ctx->stats());
    ctx->launches++;
  } else if (in_warmup) {
    adagc_warmup_finalize_kernel<<<1, kWarmupThreads, 0, s>>>(cs, d_ema, ctx->stats());
    ctx->launches++;
  }
  if (ctx->timing) cudaEventRecord(ctx->ev[2], s);
}

// Clip-only phase 3: hat(g) = h g in the gradient dtype.
void launch_scale(adagc_ctx* ctx, const void* d_grads_in, void* d_grads_out, cudaStream_t s) {
  const int in_place = d_grads_in == d_grads_out ? 1 : 0;
  if (ctx->bf16)
    adagc_scale_kernel<true><<<ctx->grid_wide, kThreads, 0, s>>>(d_grads_in, d_grads_out, ctx->d_chunks_wide(),
                                                                ctx->d_begin_wide(), ctx->stats().h, in_place, ctx->guard());
  else
    adagc_scale_kernel<false><<<ctx->grid_wide, kThreads, 0, s>>>(d_grads_in, d_grads_out, ctx->d_chunks_wide(),
                                                                 ctx->d_begin_wide(), ctx->stats().h, in_place, ctx->guard());
  ctx->launches++;
}

// Norm, finalize and AdamW update of an AdaGC step (step > warmup), one group of tensors after the other.
// With wait_copies, stream s waits for each group's host-to-device copy event first.
int enqueue_grouped_adamw(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v, float* d_ema,
                          const ClipScalars& cs, const AdamScalars& a, bool wait_copies, cudaStream_t s) {
  const Chunk* gcw = reinterpret_cast<const Chunk*>(ctx->ws + ctx->L.g_chunks_wide);
  const Chunk* gcu = reinterpret_cast<const Chunk*>(ctx->ws + ctx->L.g_chunks_upd);
  const int32_t* gbw = reinterpret_cast<const int32_t*>(ctx->ws + ctx->L.g_begin_wide);
  const int32_t* gbu = reinterpret_cast<const int32_t*>(ctx->ws + ctx->L.g_begin_upd);
  const int32_t* gmu = reinterpret_cast<const int32_t*>(ctx->ws + ctx->L.g_mid_upd);
  const int32_t* order = reinterpret_cast<const int32_t*>(ctx->ws + ctx->L.g_order);
  for (size_t k = 0; k < ctx->groups.size(); ++k) {
    const adagc_ctx::Group& gr = ctx->groups[k];
    const size_t slot = k * (kGroupMaxGrid + 1);
    if (wait_copies && cudaStreamWaitEvent(s, ctx->ev_group[k], 0) != cudaSuccess) return ADAGC_E_CUDA;
    const TableView wide = {gcw + gr.chunk_base, gbw + slot, nullptr, gr.grid_wide};
    const TableView upd = {gcu + gr.chunk_base, gbu + slot, gmu + slot, gr.grid_update};
    launch_norm(ctx, wide, d_grads, s);
    const int blocks = (gr.n_tensors * 32 + kFinalizeThreads - 1) / kFinalizeThreads;
    adagc_tensor_finalize_kernel<<<blocks, kFinalizeThreads, 0, s>>>(ctx->d_partials(), ctx->d_tensors(), cs, 1, d_ema,
                                                                    ctx->stats(), order, gr.order_first, gr.n_tensors,
                                                                    k == 0 ? 1 : 0);
    ctx->launches++;
    launch_update<kOptAdamW>(ctx, upd, d_params, d_grads, d_m, d_v, a, s);
  }
  return ADAGC_OK;
}

int finish_launches(adagc_ctx* ctx, cudaStream_t s) {
  if (ctx->timing) {
    cudaEventRecord(ctx->ev[3], s);
    ctx->timing_valid = true;
  }
  return cudaGetLastError() == cudaSuccess ? ADAGC_OK : ADAGC_E_CUDA;
}

const void* fused_small_kernel_of(const adagc_ctx* ctx) {
  if (ctx->bf16)
    return ctx->state_bf16 ? reinterpret_cast<const void*>(adagc_fused_small_kernel<true, true>)
                           : reinterpret_cast<const void*>(adagc_fused_small_kernel<true, false>);
  return ctx->state_bf16 ? reinterpret_cast<const void*>(adagc_fused_small_kernel<false, true>)
                         : reinterpret_cast<const void*>(adagc_fused_small_kernel<false, false>);
}

// adagc_step of a context created with ADAGC_FUSED_SMALL: one cooperative launch.
int launch_fused_small(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v, float* d_ema,
                       ClipScalars cs, bool in_warmup, AdamScalars a, cudaStream_t s) {
  if (ctx->timing) {
    cudaEventRecord(ctx->ev[0], s);
    cudaEventRecord(ctx->ev[1], s);
    cudaEventRecord(ctx->ev[2], s);  // the phases are not separable here: the whole kernel is reported as the third
  }
  float* p = static_cast<float*>(d_params);
  void* m = d_m;
  void* v = d_v;
  const Chunk* chunks = ctx->d_chunks_upd();
  int n_chunks = ctx->n_chunks;
  const TensorEntry* tensors = ctx->d_tensors();
  double* partials = reinterpret_cast<double*>(ctx->ws + ctx->L.slice_partials);
  int warm = in_warmup ? 1 : 0;
  StatPtrs st = ctx->stats();
  unsigned long long* counter = reinterpret_cast<unsigned long long*>(ctx->ws + ctx->L.scalars + 16);
  unsigned long long index = ctx->barriers_done;
  float* gamma_prev = reinterpret_cast<float*>(ctx->ws + ctx->L.gamma_prev);
  Guard guard = ctx->guard();
  StateRounding sr = ctx->rounding();
  void* args[] = {&p,        &d_grads, &m,    &v, &d_ema, &chunks,  &n_chunks, &tensors,
                  &partials, &cs,      &warm, &a, &st,    &counter, &index, &gamma_prev, &guard, &sr};
  const void* fn = fused_small_kernel_of(ctx);
  if (cudaLaunchCooperativeKernel(fn, dim3(ctx->grid_fused), dim3(kThreads), args, 0, s) != cudaSuccess) {
    (void)cudaGetLastError();
    return ADAGC_E_CUDA;
  }
  ctx->barriers_done += in_warmup ? 3 : 1;
  ctx->launches++;
  return finish_launches(ctx, s);
}

// What the host remembers of a status word it has read: after a timed-out grid barrier the device-side arrival counter
// and the host's count of barriers differ for good, so every later one-kernel step would wait its full limit and skip
// its update; the context refuses them instead.
void latch_device_status(adagc_ctx* ctx, int32_t device_status) {
  if (ctx->fused_small && (device_status & ADAGC_E_TIMEOUT)) ctx->fused_poisoned = true;
}

void release_ctx(adagc_ctx* ctx) {
  for (int k = 0; k < 4; ++k)
    if (ctx->ev[k]) cudaEventDestroy(ctx->ev[k]);
  for (cudaEvent_t e : ctx->ev_group)
    if (e) cudaEventDestroy(e);
  if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  delete ctx;
}


}  // namespace

extern "C" {

size_t adagc_workspace_bytes(const adagc_desc* desc) {
  int64_t n_chunks = 0;
  if (validate_desc(desc, &n_chunks, nullptr) != ADAGC_OK) return 0;
  return make_layout(n_chunks, desc->n_tensors, (desc->flags & ADAGC_FUSED_SMALL) != 0).total;
}

int64_t adagc_num_chunks(const adagc_desc* desc) {
  int64_t n_chunks = 0;
  const int rc = validate_desc(desc, &n_chunks, nullptr);
  return rc != ADAGC_OK ? rc : n_chunks;
}

int adagc_create(const adagc_desc* desc, void* d_workspace, size_t workspace_bytes, void* cuda_stream,
                 adagc_ctx** out) {
  if (!out) return ADAGC_E_INVALID_ARG;
  *out = nullptr;
  int64_t n_chunks = 0, extent = 0;
  const int rc = validate_desc(desc, &n_chunks, &extent);
  if (rc != ADAGC_OK) return rc;
  const Layout L = make_layout(n_chunks, desc->n_tensors, (desc->flags & ADAGC_FUSED_SMALL) != 0);
  if (!d_workspace || workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(d_workspace) & 255u))
    return ADAGC_E_WORKSPACE;

  std::vector<Chunk> chunks;
  std::vector<TensorEntry> tensors;
  cut_into_chunks(desc, n_chunks, &chunks, &tensors);

  adagc_ctx* ctx = new (std::nothrow) adagc_ctx();
  if (!ctx) return ADAGC_E_NOMEM;
  ctx->T = desc->n_tensors;
  ctx->n_chunks = static_cast<int32_t>(n_chunks);
  ctx->arena_elems = extent;
  ctx->bf16 = desc->grad_dtype == ADAGC_BF16;
  ctx->state_bf16 = desc->state_dtype == ADAGC_BF16;
  ctx->lambda_abs = desc->lambda_abs;
  bool any_empty = false;
  for (int32_t i = 0; i < desc->n_tensors; ++i) {
    if (desc->tensors[i].numel == 0) any_empty = true;
    else ctx->offsets_mult8 = ctx->offsets_mult8 && desc->tensors[i].offset % 8 == 0;
  }
  ctx->ws = static_cast<char*>(d_workspace);
  ctx->L = L;
  ctx->fold_finalize = !any_empty && !(desc->flags & ADAGC_SEPARATE_FINALIZE);

  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaDeviceProp prop;
  bool ok = cudaGetDevice(&ctx->device) == cudaSuccess &&
            cudaGetDeviceProperties(&prop, ctx->device) == cudaSuccess;
  if (ok) {
    int occ_n = 0, occ_s = 0;
    if (ctx->bf16) {
      ok = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_n, adagc_norm_kernel<true>, kThreads, 0) == cudaSuccess &&
           cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_s, adagc_scale_kernel<true>, kThreads, 0) == cudaSuccess &&
           (ctx->state_bf16 ? prepare_update_kernels<true, true>() : prepare_update_kernels<true, false>());
    } else {
      ok = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_n, adagc_norm_kernel<false>, kThreads, 0) == cudaSuccess &&
           cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_s, adagc_scale_kernel<false>, kThreads, 0) == cudaSuccess &&
           (ctx->state_bf16 ? prepare_update_kernels<false, true>() : prepare_update_kernels<false, false>());
    }
    if (ok) {
      const int64_t sms = prop.multiProcessorCount;
      const int64_t wide = sms * std::max(1, std::min(occ_n, occ_s));
      ctx->grid_wide = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>({n_chunks, wide, kMaxGrid})));
      ctx->update_bulk = (desc->flags & ADAGC_UPDATE_PATH_MASK) != ADAGC_UPDATE_PATH_REGISTERS;
      ctx->keep_initial = (desc->flags & ADAGC_EMA_KEEP_INITIAL) != 0;
      ctx->global_adaptive = (desc->flags & ADAGC_CLIP_GLOBAL_ADAPTIVE) != 0;
      ctx->grid_update = static_cast<int>(std::max<int64_t>(
          1, std::min<int64_t>({n_chunks, sms * (ctx->update_bulk ? 1 : kUpdateBlocksPerSM), kMaxGrid})));
    }
  }
  if (ok && (desc->flags & ADAGC_FUSED_SMALL)) {
    // the one-kernel step needs every block resident at once (cooperative launch) and is meant for small layouts
    int coop = 0, occ_f = 0;
    ok = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device) == cudaSuccess &&
         cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_f, fused_small_kernel_of(ctx), kThreads, 0) == cudaSuccess;
    if (ok && (!coop || n_chunks > kFusedMaxChunks || occ_f < 1)) {
      release_ctx(ctx);
      return ADAGC_E_INVALID_ARG;
    }
    ctx->fused_small = ok;
    ctx->grid_fused = static_cast<int>(std::max<int64_t>(
        1, std::min<int64_t>(n_chunks * 4, static_cast<int64_t>(prop.multiProcessorCount) * std::min(occ_f, 2))));
  }
  std::vector<Chunk> table_wide, table_upd;
  std::vector<int32_t> begin_wide, begin_upd, mid_upd, begin_range;
  if (ok) {
    balance_chunks(chunks, ctx->grid_wide, &table_wide, &begin_wide);
    balance_chunks(chunks, ctx->grid_update, &table_upd, &begin_upd, &mid_upd);
    begin_range = contiguous_ranges(chunks, ctx->grid_wide);
  }
  auto upload = [&](size_t off, const void* src, size_t bytes) {
    if (bytes == 0) return;  // a rank of a sharded model may hold no chunk at all
    ok = ok && cudaMemcpyAsync(ctx->ws + off, src, bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  };
  ok = ok && cudaMemsetAsync(ctx->ws, 0, L.total, s) == cudaSuccess;
  upload(L.chunks_range, chunks.data(), sizeof(Chunk) * chunks.size());
  upload(L.begin_range, begin_range.data(), sizeof(int32_t) * begin_range.size());
  upload(L.chunks_wide, table_wide.data(), sizeof(Chunk) * table_wide.size());
  upload(L.chunks_upd, table_upd.data(), sizeof(Chunk) * table_upd.size());
  upload(L.begin_wide, begin_wide.data(), sizeof(int32_t) * begin_wide.size());
  upload(L.begin_upd, begin_upd.data(), sizeof(int32_t) * begin_upd.size());
  upload(L.mid_upd, mid_upd.data(), sizeof(int32_t) * mid_upd.size());
  upload(L.tensors, tensors.data(), sizeof(TensorEntry) * tensors.size());
  // groups of tensors (arena order) for the pipelined host step, each with its own balanced tables
  std::vector<Chunk> g_table_wide, g_table_upd;
  std::vector<int32_t> g_begin_wide(static_cast<size_t>(kMaxGroups) * (kGroupMaxGrid + 1), 0), g_begin_upd = g_begin_wide,
                       g_mid_upd = g_begin_wide, g_order(desc->n_tensors);
  if (ok && !any_empty) {  // (a shard that lists tensors it holds nothing of takes the unpipelined host step)
    const int64_t esz = ctx->bf16 ? 2 : 4;
    for (int32_t i = 0; i < desc->n_tensors; ++i) g_order[i] = i;
    std::sort(g_order.begin(), g_order.end(),
              [&](int32_t x, int32_t y) { return desc->tensors[x].offset < desc->tensors[y].offset; });
    int64_t total_bytes = 0;
    for (int32_t i = 0; i < desc->n_tensors; ++i) total_bytes += desc->tensors[i].numel * esz;
    const int64_t target = std::max<int64_t>(kGroupMinBytes, (total_bytes + kMaxGroups - 1) / kMaxGroups);
    g_table_wide.reserve(n_chunks);
    g_table_upd.reserve(n_chunks);
    int32_t k = 0;
    while (k < desc->n_tensors) {
      adagc_ctx::Group gr;
      gr.order_first = k;
      gr.chunk_base = static_cast<int32_t>(g_table_wide.size());
      gr.elem_begin = desc->tensors[g_order[k]].offset;
      std::vector<Chunk> mine;
      int64_t bytes = 0;
      const bool last_group = static_cast<int>(ctx->groups.size()) == kMaxGroups - 1;
      while (k < desc->n_tensors && (bytes < target || last_group)) {
        const int32_t i = g_order[k];
        bytes += desc->tensors[i].numel * esz;
        gr.elem_end = desc->tensors[i].offset + desc->tensors[i].numel;
        mine.insert(mine.end(), chunks.begin() + tensors[i].first_chunk,
                    chunks.begin() + tensors[i].first_chunk + tensors[i].n_chunks);
        ++k;
      }
      gr.n_tensors = k - gr.order_first;
      const int64_t nc = static_cast<int64_t>(mine.size());
      gr.grid_wide = static_cast<int>(std::min<int64_t>({nc, ctx->grid_wide, kGroupMaxGrid}));
      gr.grid_update = static_cast<int>(std::min<int64_t>({nc, ctx->grid_update, kGroupMaxGrid}));
      std::vector<Chunk> tw, tu;
      std::vector<int32_t> bw, bu, mu;
      balance_chunks(mine, gr.grid_wide, &tw, &bw);
      balance_chunks(mine, gr.grid_update, &tu, &bu, &mu);
      const size_t slot = ctx->groups.size() * (kGroupMaxGrid + 1);
      std::copy(bw.begin(), bw.end(), g_begin_wide.begin() + slot);
      std::copy(bu.begin(), bu.end(), g_begin_upd.begin() + slot);
      std::copy(mu.begin(), mu.end(), g_mid_upd.begin() + slot);
      g_table_wide.insert(g_table_wide.end(), tw.begin(), tw.end());
      g_table_upd.insert(g_table_upd.end(), tu.begin(), tu.end());
      ctx->groups.push_back(gr);
    }
  }
  upload(L.g_chunks_wide, g_table_wide.data(), sizeof(Chunk) * g_table_wide.size());
  upload(L.g_chunks_upd, g_table_upd.data(), sizeof(Chunk) * g_table_upd.size());
  upload(L.g_begin_wide, g_begin_wide.data(), sizeof(int32_t) * g_begin_wide.size());
  upload(L.g_begin_upd, g_begin_upd.data(), sizeof(int32_t) * g_begin_upd.size());
  upload(L.g_mid_upd, g_mid_upd.data(), sizeof(int32_t) * g_mid_upd.size());
  upload(L.g_order, g_order.data(), sizeof(int32_t) * g_order.size());
  ok = ok && cudaStreamSynchronize(s) == cudaSuccess;  // the host vectors die at return
  for (int k = 0; ok && k < 4; ++k) ok = cudaEventCreate(&ctx->ev[k]) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming) == cudaSuccess;
  ctx->ev_group.assign(ctx->groups.size(), nullptr);
  for (size_t k = 0; ok && k < ctx->ev_group.size(); ++k)
    ok = cudaEventCreateWithFlags(&ctx->ev_group[k], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    (void)cudaGetLastError();
    release_ctx(ctx);
    return ADAGC_E_CUDA;
  }
  *out = ctx;
  return ADAGC_OK;
}

int adagc_destroy(adagc_ctx* ctx) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  release_ctx(ctx);
  return ADAGC_OK;
}

int adagc_step(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v, float* d_ema,
               int64_t step, double lr, double beta1, double beta2, double eps, double wd, double lambda_rel,
               double beta, int64_t warmup, void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  rc = check_adamw_args(d_params, d_grads, d_m, d_v, lr, beta1, beta2, eps, wd);
  if (rc != ADAGC_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (ctx->fused_small && ctx->fused_poisoned) return ADAGC_E_POISONED;
  if (ctx->fused_small)
    return launch_fused_small(ctx, d_params, d_grads, d_m, d_v, d_ema, make_clip_scalars(ctx, step, lambda_rel, beta),
                              step <= warmup, make_adam_scalars(step, lr, beta1, beta2, eps, wd), s);
  rc = enqueue_clip_phases(ctx, d_grads, d_ema, step, lambda_rel, beta, warmup, s);
  if (rc != ADAGC_OK) return rc;
  const AdamScalars a = make_adam_scalars(step, lr, beta1, beta2, eps, wd);
  launch_update<kOptAdamW>(ctx, d_params, d_grads, d_m, d_v, a, s);
  return finish_launches(ctx, s);
}

int adagc_step_emit_bf16(adagc_ctx* ctx, void* d_params, void* d_params_bf16, const void* d_grads, void* d_m,
                         void* d_v, float* d_ema, int64_t step, double lr, double beta1, double beta2, double eps,
                         double wd, double lambda_rel, double beta, int64_t warmup, void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  rc = check_adamw_args(d_params, d_grads, d_m, d_v, lr, beta1, beta2, eps, wd);
  if (rc != ADAGC_OK) return rc;
  if (!d_params_bf16) return ADAGC_E_INVALID_ARG;
  if (!aligned16(d_params_bf16) || !ctx->offsets_mult8) return ADAGC_E_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  rc = enqueue_clip_phases(ctx, d_grads, d_ema, step, lambda_rel, beta, warmup, s);
  if (rc != ADAGC_OK) return rc;
  const AdamScalars a = make_adam_scalars(step, lr, beta1, beta2, eps, wd);
  launch_update<kOptAdamW>(ctx, d_params, d_grads, d_m, d_v, a, s, d_params_bf16);
  return finish_launches(ctx, s);
}

int adagc_step_lion(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, float* d_ema, int64_t step,
                    double lr, double beta1, double beta2, double wd, double lambda_rel, double beta,
                    int64_t warmup, void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  if (!d_params || !d_grads || !d_m) return ADAGC_E_INVALID_ARG;
  if (!(beta1 >= 0.0 && beta1 < 1.0) || !(beta2 >= 0.0 && beta2 < 1.0)) return ADAGC_E_INVALID_ARG;
  if (!std::isfinite(lr) || !std::isfinite(wd)) return ADAGC_E_INVALID_ARG;
  if (!aligned16(d_params) || !aligned16(d_grads) || !aligned16(d_m)) return ADAGC_E_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  rc = enqueue_clip_phases(ctx, d_grads, d_ema, step, lambda_rel, beta, warmup, s);
  if (rc != ADAGC_OK) return rc;
  AdamScalars a;
  a.beta1 = static_cast<float>(beta1);
  a.one_minus_beta1 = static_cast<float>(1.0 - beta1);
  a.beta2 = static_cast<float>(beta2);
  a.one_minus_beta2 = static_cast<float>(1.0 - beta2);
  a.inv_bc2 = 0.0f;
  a.step_size = static_cast<float>(lr);
  a.decay = static_cast<float>(1.0 - lr * wd);
  a.eps = 0.0f;
  launch_update<kOptLion>(ctx, d_params, d_grads, d_m, nullptr, a, s);
  return finish_launches(ctx, s);
}

int adagc_step_sgdm(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, float* d_ema, int64_t step,
                    double lr, double momentum, double wd, double lambda_rel, double beta, int64_t warmup,
                    void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  if (!d_params || !d_grads || !d_m) return ADAGC_E_INVALID_ARG;
  if (!(momentum >= 0.0 && momentum < 1.0) || !std::isfinite(lr) || !std::isfinite(wd)) return ADAGC_E_INVALID_ARG;
  if (!aligned16(d_params) || !aligned16(d_grads) || !aligned16(d_m)) return ADAGC_E_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  rc = enqueue_clip_phases(ctx, d_grads, d_ema, step, lambda_rel, beta, warmup, s);
  if (rc != ADAGC_OK) return rc;
  AdamScalars a = {};
  a.beta1 = static_cast<float>(momentum);
  a.step_size = static_cast<float>(lr);
  a.decay = static_cast<float>(wd);
  launch_update<kOptSgdM>(ctx, d_params, d_grads, d_m, nullptr, a, s);
  return finish_launches(ctx, s);
}

int adagc_clip(adagc_ctx* ctx, const void* d_grads_in, void* d_grads_out, float* d_ema, int64_t step,
               double lambda_rel, double beta, int64_t warmup, void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  if (!d_grads_in || !d_grads_out) return ADAGC_E_INVALID_ARG;
  if (!aligned16(d_grads_in) || !aligned16(d_grads_out)) return ADAGC_E_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  rc = enqueue_clip_phases(ctx, d_grads_in, d_ema, step, lambda_rel, beta, warmup, s);
  if (rc != ADAGC_OK) return rc;
  launch_scale(ctx, d_grads_in, d_grads_out, s);
  return finish_launches(ctx, s);
}

int adagc_step_capturable(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v, float* d_ema,
                          const float* d_lr, double lr, double beta1, double beta2, double eps, double wd,
                          double lambda_rel, double beta, int64_t warmup, void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, 1, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  rc = check_adamw_args(d_params, d_grads, d_m, d_v, lr, beta1, beta2, eps, wd);
  if (rc != ADAGC_OK) return rc;
  if (d_lr && (reinterpret_cast<uintptr_t>(d_lr) & 3u)) return ADAGC_E_MISALIGNED;
  if (ctx->sr_stochastic) return ADAGC_E_INVALID_ARG;  // the generator's counter holds the step number, known on the host only
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  DeviceStep* ds = reinterpret_cast<DeviceStep*>(ctx->ws + ctx->L.dev_step);
  StepHyper hh;
  hh.lr = lr; hh.beta1 = beta1; hh.beta2 = beta2; hh.eps = eps; hh.wd = wd;
  hh.lambda_rel = lambda_rel; hh.beta = beta; hh.lambda_abs = ctx->lambda_abs; hh.ema_cap = ctx->ema_cap;
  hh.warmup = warmup; hh.n_tensors = ctx->T; hh.keep_initial = ctx->keep_initial ? 1 : 0;
  const StatPtrs st = ctx->stats();
  // the same launches every step: what differs between steps is read from device memory
  adagc_step_prologue_kernel<<<1, 32, 0, s>>>(st.steps_done, d_lr, hh, ds);
  ctx->launches++;
  const TableView wide = {ctx->d_chunks_wide(), ctx->d_begin_wide(), nullptr, ctx->grid_wide};
  launch_norm(ctx, wide, d_grads, s);
  const int blocks = (ctx->T * 32 + kFinalizeThreads - 1) / kFinalizeThreads;
  adagc_tensor_finalize_kernel<<<blocks, kFinalizeThreads, 0, s>>>(ctx->d_partials(), ctx->d_tensors(), ClipScalars{},
                                                                  ctx->global_adaptive ? 0 : 1, d_ema, st, nullptr, 0,
                                                                  ctx->T, 1, ds);
  ctx->launches++;
  if (ctx->global_adaptive)
    adagc_global_finalize_kernel<<<1, kWarmupThreads, 0, s>>>(ClipScalars{}, 0, d_ema, st, ds);
  else
    adagc_warmup_finalize_kernel<<<1, kWarmupThreads, 0, s>>>(ClipScalars{}, d_ema, st, ds);
  ctx->launches++;
  launch_update<kOptAdamW>(ctx, d_params, d_grads, d_m, d_v, AdamScalars{}, s, nullptr, &ds->a);
  return cudaGetLastError() == cudaSuccess ? ADAGC_OK : ADAGC_E_CUDA;
}

int adagc_set_step_counter(adagc_ctx* ctx, uint64_t steps_done, void* cuda_stream) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  adagc_set_counter_kernel<<<1, 1, 0, s>>>(ctx->stats().steps_done, static_cast<unsigned long long>(steps_done));
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ADAGC_OK : ADAGC_E_CUDA;
}

int adagc_shard_sumsq(adagc_ctx* ctx, const void* d_grads, double* d_sumsq_out, void* cuda_stream) {
  if (!ctx || !d_sumsq_out) return ADAGC_E_INVALID_ARG;
  const bool holds = ctx->n_chunks > 0;  // a rank that owns nothing may pass any gradient pointer, NULL included
  if (holds && !d_grads) return ADAGC_E_INVALID_ARG;
  if ((holds && !aligned16(d_grads)) || (reinterpret_cast<uintptr_t>(d_sumsq_out) & 7u)) return ADAGC_E_MISALIGNED;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return ADAGC_E_CUDA;
  if (dev != ctx->device) return ADAGC_E_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const TableView wide = {ctx->d_chunks_wide(), ctx->d_begin_wide(), nullptr, ctx->grid_wide};
  launch_norm(ctx, wide, d_grads, s);
  // the same fixed-order per-tensor sum as the unsharded step, written to the caller's vector; no decision
  StatPtrs st = ctx->stats();
  st.sumsq = d_sumsq_out;
  const int blocks = (ctx->T * 32 + kFinalizeThreads - 1) / kFinalizeThreads;
  adagc_tensor_finalize_kernel<<<blocks, kFinalizeThreads, 0, s>>>(ctx->d_partials(), ctx->d_tensors(), ClipScalars{},
                                                                  0, nullptr, st, nullptr, 0, ctx->T, 0);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ADAGC_OK : ADAGC_E_CUDA;
}

int adagc_step_presummed(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v, float* d_ema,
                         const double* d_sumsq, int64_t step, double lr, double beta1, double beta2, double eps,
                         double wd, double lambda_rel, double beta, int64_t warmup, void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  rc = check_adamw_args(d_params, d_grads, d_m, d_v, lr, beta1, beta2, eps, wd, ctx->n_chunks > 0);
  if (rc != ADAGC_OK) return rc;
  if (!d_sumsq) return ADAGC_E_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_sumsq) & 7u) return ADAGC_E_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  enqueue_presummed_phase(ctx, d_sumsq, d_ema, step, lambda_rel, beta, warmup, s);
  const AdamScalars a = make_adam_scalars(step, lr, beta1, beta2, eps, wd);
  launch_update<kOptAdamW>(ctx, d_params, d_grads, d_m, d_v, a, s);
  return finish_launches(ctx, s);
}

int adagc_clip_presummed(adagc_ctx* ctx, const void* d_grads_in, void* d_grads_out, float* d_ema,
                         const double* d_sumsq, int64_t step, double lambda_rel, double beta, int64_t warmup,
                         void* cuda_stream) {
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  const bool holds = ctx->n_chunks > 0;
  if ((holds && (!d_grads_in || !d_grads_out)) || !d_sumsq) return ADAGC_E_INVALID_ARG;
  if ((holds && (!aligned16(d_grads_in) || !aligned16(d_grads_out))) || (reinterpret_cast<uintptr_t>(d_sumsq) & 7u))
    return ADAGC_E_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  enqueue_presummed_phase(ctx, d_sumsq, d_ema, step, lambda_rel, beta, warmup, s);
  launch_scale(ctx, d_grads_in, d_grads_out, s);
  return finish_launches(ctx, s);
}

int adagc_shard_plan(const adagc_desc* full, int32_t rank, int32_t world, adagc_tensor* local, int64_t* elem_begin,
                     int64_t* elem_end) {
  int64_t extent = 0;
  const int rc = validate_desc(full, nullptr, &extent);
  if (rc != ADAGC_OK) return rc;
  if (!local || world < 1 || rank < 0 || rank >= world) return ADAGC_E_INVALID_ARG;
  const int64_t shard = ((extent + world - 1) / world + 7) / 8 * 8;
  int64_t b = std::min<int64_t>(extent, shard * rank), e = std::min<int64_t>(extent, shard * (rank + 1));
  if (b == e) b = e = 0;  // a rank beyond the end of a small arena holds nothing: the empty range at the start
  for (int32_t i = 0; i < full->n_tensors; ++i) {
    const adagc_tensor& t = full->tensors[i];
    const int64_t lo = std::max<int64_t>(t.offset, b), hi = std::min<int64_t>(t.offset + t.numel, e);
    adagc_tensor out = {};
    if (t.numel > 0 && hi > lo) {
      out.numel = hi - lo;
      out.offset = lo - b;
    }
    local[i] = out;
  }
  if (elem_begin) *elem_begin = b;
  if (elem_end) *elem_end = e;
  return ADAGC_OK;
}

int adagc_get_stats(adagc_ctx* ctx, float* h_norm, float* h_clipfactor, uint8_t* h_flag, uint64_t* h_clip_count,
                    uint64_t* h_steps_done, int32_t* h_device_status, void* cuda_stream) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const StatPtrs st = ctx->stats();
  const size_t T = static_cast<size_t>(ctx->T);
  bool ok = true;
  if (h_norm) ok = ok && cudaMemcpyAsync(h_norm, st.norm, 4 * T, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (h_clipfactor) ok = ok && cudaMemcpyAsync(h_clipfactor, st.h, 4 * T, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (h_flag) ok = ok && cudaMemcpyAsync(h_flag, st.flag, T, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (h_clip_count)
    ok = ok && cudaMemcpyAsync(h_clip_count, st.clip_count, 8 * T, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (h_steps_done)
    ok = ok && cudaMemcpyAsync(h_steps_done, st.steps_done, 8, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (h_device_status)
    ok = ok && cudaMemcpyAsync(h_device_status, st.status, 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  int32_t status_now = 0;  // read in any case: a timed-out grid barrier of the one-kernel step must be latched
  ok = ok && cudaMemcpyAsync(&status_now, st.status, 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
  if (ok) latch_device_status(ctx, status_now);
  return ok ? ADAGC_OK : ADAGC_E_CUDA;
}

int adagc_debug_chunk_tables(const adagc_desc* desc, int32_t which, int32_t grid, int64_t* h_start, int32_t* h_count,
                             int32_t* h_tensor, int32_t* h_partial, int32_t* h_block_begin, int32_t* h_block_mid) {
  int64_t n_chunks = 0;
  const int rc = validate_desc(desc, &n_chunks, nullptr);
  if (rc != ADAGC_OK) return rc;
  if (which < 0 || which > 2 || grid < 1 || grid > kMaxGrid || !h_start || !h_count || !h_tensor || !h_partial ||
      !h_block_begin || (which == 2 && !h_block_mid))
    return ADAGC_E_INVALID_ARG;
  std::vector<Chunk> chunks, table;
  std::vector<TensorEntry> tensors;
  cut_into_chunks(desc, n_chunks, &chunks, &tensors);
  std::vector<int32_t> begin, mid;
  if (which == 0) {
    table = chunks;
    begin = contiguous_ranges(chunks, grid);
  } else if (which == 1) {
    balance_chunks(chunks, grid, &table, &begin);
  } else {
    balance_chunks(chunks, grid, &table, &begin, &mid);
  }
  for (size_t k = 0; k < table.size(); ++k) {
    h_start[k] = chunk_start(table[k]);
    h_count[k] = table[k].count;
    h_tensor[k] = table[k].tensor;
    h_partial[k] = table[k].partial;
  }
  std::copy(begin.begin(), begin.end(), h_block_begin);
  if (which == 2) std::copy(mid.begin(), mid.begin() + grid, h_block_mid);
  return ADAGC_OK;
}

int adagc_debug_chunk_entry_ok(int64_t start, int32_t count, int32_t tensor, int32_t partial, int64_t arena_elems,
                               int32_t n_chunks, int32_t n_tensors) {
  if (start < 0 || (start & 3) || (start >> 2) > int64_t(0xffffffff)) return 0;
  Chunk c;
  c.start4 = static_cast<uint32_t>(start >> 2);
  c.count = count;
  c.tensor = tensor;
  c.partial = partial;
  return chunk_entry_ok(c, arena_elems, n_chunks, n_tensors) ? 1 : 0;
}

int adagc_debug_bounds_checked_build(void) {
#ifdef ADAGC_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}

int adagc_debug_latch_status(adagc_ctx* ctx, int32_t device_status) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  latch_device_status(ctx, device_status);
  return ADAGC_OK;
}

int adagc_get_sumsq(adagc_ctx* ctx, double* h_sumsq, void* cuda_stream) {
  if (!ctx || !h_sumsq) return ADAGC_E_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  bool ok = cudaMemcpyAsync(h_sumsq, ctx->stats().sumsq, 8 * static_cast<size_t>(ctx->T),
                            cudaMemcpyDeviceToHost, s) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
  return ok ? ADAGC_OK : ADAGC_E_CUDA;
}

int adagc_step_host(adagc_ctx* ctx, void* d_params, void* d_grads, void* d_m, void* d_v, float* d_ema,
                    const void* h_grads, int64_t step, double lr, double beta1, double beta2, double eps,
                    double wd, double lambda_rel, double beta, int64_t warmup, float* h_norm,
                    float* h_clipfactor, uint8_t* h_flag, void* cuda_stream) {
  if (!ctx || !h_grads || !d_grads) return ADAGC_E_INVALID_ARG;
  int rc = check_clip_args(ctx, d_ema, step, lambda_rel, beta, warmup);
  if (rc != ADAGC_OK) return rc;
  rc = check_adamw_args(d_params, d_grads, d_m, d_v, lr, beta1, beta2, eps, wd);
  if (rc != ADAGC_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t esz = ctx->bf16 ? 2 : 4;
  const char* h_bytes = static_cast<const char*>(h_grads);
  char* d_bytes = static_cast<char*>(d_grads);

  if (step <= warmup || ctx->timing || ctx->global_adaptive || ctx->groups.size() < 2) {
    // warm-up needs the global norm before any update can start: copy everything, then the plain step
    const size_t bytes = static_cast<size_t>(ctx->arena_elems) * esz;
    if (cudaMemcpyAsync(d_grads, h_grads, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return ADAGC_E_CUDA;
    rc = adagc_step(ctx, d_params, d_grads, d_m, d_v, d_ema, step, lr, beta1, beta2, eps, wd, lambda_rel, beta,
                    warmup, cuda_stream);
    if (rc != ADAGC_OK) return rc;
    return adagc_get_stats(ctx, h_norm, h_clipfactor, h_flag, nullptr, nullptr, nullptr, cuda_stream);
  }

  // AdaGC steps decide per tensor, so a group of tensors can go through all three phases as soon as its
  // gradients have arrived: the copies run on a second stream, group by group, and the caller's stream
  // follows one group behind.  The copy engine stays busy from start to end; the kernels hide behind it.
  bool ok = cudaEventRecord(ctx->ev_entry, s) == cudaSuccess &&      // earlier work on s may still read d_grads
            cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_entry, 0) == cudaSuccess;
  for (size_t k = 0; ok && k < ctx->groups.size(); ++k) {
    const adagc_ctx::Group& gr = ctx->groups[k];
    const size_t off = static_cast<size_t>(gr.elem_begin) * esz;
    const size_t bytes = static_cast<size_t>(gr.elem_end - gr.elem_begin) * esz;
    ok = cudaMemcpyAsync(d_bytes + off, h_bytes + off, bytes, cudaMemcpyHostToDevice, ctx->copy_stream) == cudaSuccess &&
         cudaEventRecord(ctx->ev_group[k], ctx->copy_stream) == cudaSuccess;
  }
  if (!ok) return ADAGC_E_CUDA;
  rc = enqueue_grouped_adamw(ctx, d_params, d_grads, d_m, d_v, d_ema, make_clip_scalars(ctx, step, lambda_rel, beta),
                             make_adam_scalars(step, lr, beta1, beta2, eps, wd), true, s);
  if (rc != ADAGC_OK) return rc;
  if (cudaGetLastError() != cudaSuccess) return ADAGC_E_CUDA;
  return adagc_get_stats(ctx, h_norm, h_clipfactor, h_flag, nullptr, nullptr, nullptr, cuda_stream);
}

int adagc_debug_wait_timeout(adagc_ctx* ctx, double limit_ms, void* cuda_stream) {
  if (!ctx || !(limit_ms > 0.0) || limit_ms > 1000.0) return ADAGC_E_INVALID_ARG;
  adagc_debug_wait_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<uint64_t>(limit_ms * 1e6), ctx->stats().status);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ADAGC_OK : ADAGC_E_CUDA;
}

int adagc_set_ema_cap(adagc_ctx* ctx, double cap) {
  if (!ctx || !(cap >= 0.0) || !std::isfinite(cap)) return ADAGC_E_INVALID_ARG;
  ctx->ema_cap = cap;
  return ADAGC_OK;
}

int adagc_set_state_rounding(adagc_ctx* ctx, int32_t mode, uint64_t seed) {
  if (!ctx || (mode != ADAGC_ROUND_NEAREST && mode != ADAGC_ROUND_STOCHASTIC)) return ADAGC_E_INVALID_ARG;
  if (mode == ADAGC_ROUND_STOCHASTIC && !ctx->state_bf16) return ADAGC_E_DTYPE;
  ctx->sr_stochastic = mode == ADAGC_ROUND_STOCHASTIC;
  ctx->sr_seed = seed;
  return ADAGC_OK;
}

int adagc_update_path(const adagc_ctx* ctx) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  return ctx->update_bulk ? ADAGC_UPDATE_PATH_BULK : ADAGC_UPDATE_PATH_REGISTERS;
}

int adagc_launch_grids(const adagc_ctx* ctx, int32_t* norm_grid, int32_t* update_grid) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  if (norm_grid) *norm_grid = ctx->grid_wide;
  if (update_grid) *update_grid = ctx->grid_update;
  return ADAGC_OK;
}

int64_t adagc_arena_elems(const adagc_ctx* ctx) { return ctx ? ctx->arena_elems : ADAGC_E_INVALID_ARG; }

uint64_t adagc_launch_count(const adagc_ctx* ctx) { return ctx ? ctx->launches : 0; }

int adagc_set_phase_timing(adagc_ctx* ctx, int enabled) {
  if (!ctx) return ADAGC_E_INVALID_ARG;
  ctx->timing = enabled != 0;
  ctx->timing_valid = false;
  return ADAGC_OK;
}

int adagc_get_phase_times(adagc_ctx* ctx, float ms[3]) {
  if (!ctx || !ms || !ctx->timing_valid) return ADAGC_E_INVALID_ARG;
  if (cudaEventSynchronize(ctx->ev[3]) != cudaSuccess) return ADAGC_E_CUDA;
  for (int k = 0; k < 3; ++k)
    if (cudaEventElapsedTime(&ms[k], ctx->ev[k], ctx->ev[k + 1]) != cudaSuccess) return ADAGC_E_CUDA;
  return ADAGC_OK;
}

const char* adagc_strerror(int status) {
  switch (status) {
    case ADAGC_OK: return "ok";
    case ADAGC_E_INVALID_ARG: return "invalid argument";
    case ADAGC_E_MISALIGNED: return "tensor offset or arena pointer not 16-byte aligned";
    case ADAGC_E_OVERLAP: return "tensors overlap";
    case ADAGC_E_WORKSPACE: return "workspace too small or misaligned";
    case ADAGC_E_DTYPE: return "unsupported dtype combination";
    case ADAGC_E_CUDA: return "CUDA runtime error";
    case ADAGC_E_NOMEM: return "host allocation failed";
    case ADAGC_E_TOO_LARGE: return "size exceeds the fixed scratch of the no-allocation entry point";
    case ADAGC_E_POISONED: return "a grid barrier of the one-kernel step timed out earlier: create the context anew";
    default: return "unknown status";
  }
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Sum of squares of one contiguous gradient buffer with NO caller- or library-allocated scratch.
//
// Some callers cannot obtain device memory at the moment they need a norm: code running while an
// allocator is locked or exhausted, plug-ins that are handed only their input and output buffers,
// or hosts whose memory budget is fixed up front.  For them the per-chunk partial sums (the scratch
// that the norm phase above keeps in the caller's workspace) live in a fixed array inside this
// library's device image.  Every GPU that loads the library holds that array until the process exits.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxChunks = 65536;  // 512 KiB of scratch; covers 2^30 elements
constexpr int64_t kStaticMaxElems = int64_t(kStaticMaxChunks) * kChunkElems;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) double g_static_partials[kStaticMaxChunks];

// Same per-chunk arithmetic and thread mapping as adagc_norm_kernel (block_chunk_sumsq), chunks taken
// implicitly as consecutive kChunkElems-element slices of one buffer.
template <bool kBF16>
__global__ void __launch_bounds__(kThreads)
adagc_sumsq_static_kernel(const void* __restrict__ grads, int64_t numel, int n_chunks,
                          double* __restrict__ partials) {
  __shared__ double warp_part[kThreads / 32];
  for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
    const int64_t start = int64_t(c) * kChunkElems;
    const int count = static_cast<int>(numel - start < kChunkElems ? numel - start : kChunkElems);
    const uint4* vec = reinterpret_cast<const uint4*>(static_cast<const char*>(grads) + start * (kBF16 ? 2 : 4));
    const double s = block_chunk_sumsq<kBF16>(vec, count, warp_part);
    if (threadIdx.x == 0) partials[c] = s;  // every partial that is read below is rewritten by this launch
  }
}

// One warp sums the partials in the same fixed order as the step's per-tensor sums (tensor_partial_sum).
__global__ void __launch_bounds__(32)
adagc_sumsq_static_reduce_kernel(const double* __restrict__ partials, int n_chunks, double* __restrict__ out) {
  const int lane = threadIdx.x;
  TensorEntry te;
  te.first_chunk = 0;
  te.n_chunks = n_chunks;
  const double acc = tensor_partial_sum(partials, te, lane);
  if (lane == 0) *out = acc;
}

struct StaticScratch {  // host side; one entry per device ordinal, filled once by the first call on that device
  std::once_flag once[kMaxDevices];
  double* ptr[kMaxDevices] = {};
  int sms[kMaxDevices] = {};
};
StaticScratch g_static;

// With `dev` current: look up the array's device address.  In host code the array's name is only a handle; the address
// the kernels need comes from the runtime, once per device.  Leaves ptr[dev] null on failure.
void static_scratch_setup(int dev) {
  double* p = nullptr;
  int sms = 0;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || !p ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
    (void)cudaGetLastError();
    return;
  }
  g_static.sms[dev] = sms;
  g_static.ptr[dev] = p;
}

}  // namespace

extern "C" int adagc_sumsq_noalloc(const void* d_grads, int32_t grad_dtype, int64_t numel, double* d_sumsq_out,
                                   void* cuda_stream) {
  if (!d_grads || !d_sumsq_out || numel <= 0) return ADAGC_E_INVALID_ARG;
  if (grad_dtype != ADAGC_F32 && grad_dtype != ADAGC_BF16) return ADAGC_E_DTYPE;
  if (numel > kStaticMaxElems) return ADAGC_E_TOO_LARGE;
  if (!aligned16(d_grads) || (reinterpret_cast<uintptr_t>(d_sumsq_out) & 7u)) return ADAGC_E_MISALIGNED;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return ADAGC_E_CUDA;
  }
  // several host threads may make the first call on a device at the same time: one of them does the lookup, the others
  // wait for it (std::call_once also orders its writes before their reads)
  std::call_once(g_static.once[dev], static_scratch_setup, dev);
  if (!g_static.ptr[dev]) return ADAGC_E_CUDA;
  (void)cudaGetLastError();  // an error left behind by earlier calls of the process is not this call's
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int n_chunks = static_cast<int>((numel + kChunkElems - 1) / kChunkElems);
  const int grid = std::max(1, std::min(n_chunks, g_static.sms[dev] * 8));
  double* partials = g_static.ptr[dev];
  if (grad_dtype == ADAGC_BF16)
    adagc_sumsq_static_kernel<true><<<grid, kThreads, 0, s>>>(d_grads, numel, n_chunks, partials);
  else
    adagc_sumsq_static_kernel<false><<<grid, kThreads, 0, s>>>(d_grads, numel, n_chunks, partials);
  adagc_sumsq_static_reduce_kernel<<<1, 32, 0, s>>>(partials, n_chunks, d_sumsq_out);
  return cudaGetLastError() == cudaSuccess ? ADAGC_OK : ADAGC_E_CUDA;
}
