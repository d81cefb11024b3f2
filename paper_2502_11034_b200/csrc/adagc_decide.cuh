// Phase 2: per-tensor reduction of the chunk partials, clip decision and gamma update (Algorithm 1, Eq. 2 and Eq. 3):
// the finalize kernels, the norm kernel with the decisions in its tail, the pre-summed (sharded) finalize and the
// prologue of the capturable step.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

// ------------------------------------------------------------------------------------------------
// phase 2: per-tensor reduction, clip decision, gamma update
// ------------------------------------------------------------------------------------------------
struct StatPtrs {
  double* sumsq;         // [T] float64 sum of squares of this step
  float* norm;           // [T]
  float* h;              // [T] clip factor
  uint8_t* flag;         // [T]
  unsigned long long* clip_count;  // [T] cumulative
  unsigned long long* steps_done;  // [1]
  int* status;           // [1] device status word
};

// AdaGC branch of Algorithm 1 for one tensor (Eq. 3 and the gamma update).
struct Decision {
  double n, h, g_new;  // norm, clip factor, gamma after the step
  bool clip;
};

// The arithmetic of the decision alone (no memory touched): the same inputs give the same bits wherever it runs.
__device__ __forceinline__ Decision adagc_decision(double s, float gamma_stored, const ClipScalars& cs) {
  Decision d;
  d.n = sqrt(s);  // ||g_t,i||
  // gamma is fp32 state; with T_start = 0 the first step seeds it with this step's norm
  double g_prev = cs.seed ? (double)(float)d.n : (double)gamma_stored;
  if (cs.seed && cs.ema_cap > 0.0 && !(g_prev < cs.ema_cap)) g_prev = cs.ema_cap;
  const double thr = __dmul_rn(cs.lambda_rel, g_prev);
  d.clip = d.n > thr;  // strict: equality is not a clip
  d.h = d.clip ? __ddiv_rn(thr, d.n) : 1.0;
  const double c = d.clip ? thr : d.n;  // clipped norm: exactly lambda_rel * gamma when active
  d.g_new = __dadd_rn(__dmul_rn(cs.beta, g_prev), __dmul_rn(cs.one_minus_beta, c));
  return d;
}

__device__ __forceinline__ void adagc_commit(int i, double s, const Decision& d, float* __restrict__ ema,
                                             const StatPtrs& st) {
  ema[i] = (float)d.g_new;
  st.norm[i] = (float)d.n;
  st.h[i] = (float)d.h;
  st.flag[i] = d.clip ? 1 : 0;
  if (d.clip) st.clip_count[i] += 1ull;
  if (!isfinite(s)) atomicOr(st.status, ADAGC_W_NONFINITE);
}

__device__ __forceinline__ void adagc_decide(int i, double s, const ClipScalars& cs,
                                             float* __restrict__ ema, const StatPtrs& st) {
  adagc_commit(i, s, adagc_decision(s, ema[i], cs), ema, st);
}

// Fixed-order sum of one tensor's chunk partials.  The order is defined once and implemented twice, with identical
// bits: partial j is added, in increasing j, into slot j mod 256; the 32 slots of each group of 32 consecutive slots
// are combined by the xor-shuffle tree of warp_sum; the 8 group totals are added in order.
//   tensor_partial_sum        one warp: lane l keeps the 8 slots l, l + 32, ..., l + 224 (result in every lane);
//   tensor_partial_sum_block  a block of kThreads = 256 threads: thread t keeps slot t (result in thread 0; ends
//                             with a barrier) -- for tensors with thousands of partials.
__device__ __forceinline__ double tensor_partial_sum(const double* __restrict__ partials, const TensorEntry te, int lane) {
  const double* __restrict__ tp = partials + te.first_chunk;
  const int n = te.n_chunks;
  if (n <= 32) {  // slots 0..31 only: the other groups would add zeros
    return warp_sum(lane < n ? __ldcg(tp + lane) : 0.0);
  }
  double slot[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) slot[k] = 0.0;
  for (int base = 0; base < n; base += 256) {
    double t[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {  // the loads of one round are independent; the additions stay in index order
      const int j = base + k * 32 + lane;
      t[k] = j < n ? __ldcg(tp + j) : 0.0;
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) slot[k] += t[k];
  }
  double total = warp_sum(slot[0]);
#pragma unroll
  for (int k = 1; k < 8; ++k) total += warp_sum(slot[k]);
  return total;
}

__device__ __forceinline__ double tensor_partial_sum_block(const double* __restrict__ partials, const TensorEntry te,
                                                           double* warp_part) {
  static_assert(kThreads == 256, "the summation order is defined over 256 slots");
  const double* __restrict__ tp = partials + te.first_chunk;
  const int tid = threadIdx.x;
  double acc = 0.0;
  int j = tid;
  for (; j + 15 * kThreads < te.n_chunks; j += 16 * kThreads) {  // sixteen loads in flight, additions in index order
    double t[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) t[u] = __ldcg(tp + j + u * kThreads);
#pragma unroll
    for (int u = 0; u < 16; ++u) acc += t[u];
  }
  for (; j < te.n_chunks; j += kThreads) acc += __ldcg(tp + j);
  const double w = warp_sum(acc);
  if ((tid & 31) == 0) warp_part[tid >> 5] = w;
  __syncthreads();
  double s = 0.0;
  if (tid == 0) {
    s = warp_part[0];
#pragma unroll
    for (int k = 1; k < kThreads / 32; ++k) s += warp_part[k];
  }
  __syncthreads();
  return s;
}

constexpr int kBigTensorChunks = 1024;  // from here on the finalize kernel puts a whole block on the tensor's partials

// One warp per tensor (a whole block for tensors with very many chunks): fixed-order sum of the tensor's chunk
// partials; in the AdaGC branch the same warp takes the decision.
__global__ void __launch_bounds__(kFinalizeThreads)
adagc_tensor_finalize_kernel(const double* __restrict__ partials, const TensorEntry* __restrict__ tensors,
                             ClipScalars cs, int decide, float* __restrict__ ema, StatPtrs st,
                             const int32_t* __restrict__ order, int first, int count, int bump_steps,
                             const DeviceStep* __restrict__ ds = nullptr) {
  static_assert(kFinalizeThreads == kThreads, "tensor_partial_sum_block runs in this kernel's blocks");
  __shared__ double warp_part[kFinalizeThreads / 32];
  if (ds) {  // capturable step: scalars and the warm-up switch come from device memory
    cs = ds->cs;
    decide = decide && !ds->in_warmup;
  }
  // the warps of this launch take `count` tensors: order[first..first+count) if an order is given
  // (a group of the pipelined host step), else the tensors first..first+count-1
  const int k = (blockIdx.x * kFinalizeThreads + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (k < count) {
    const int w = order ? order[first + k] : first + k;
    const TensorEntry te = tensors[w];
    if (te.n_chunks < kBigTensorChunks) {
      const double acc = tensor_partial_sum(partials, te, lane);
      if (lane == 0) {
        st.sumsq[w] = acc;
        if (decide) {
          adagc_decide(w, acc, cs, ema, st);
          if (k == 0 && bump_steps) *st.steps_done += 1ull;
        }
      }
    }
  }
  // the big tensors among this block's eight, one after the other, by the whole block (uniform control flow)
  for (int k8 = 0; k8 < kFinalizeThreads / 32; ++k8) {
    const int kk = blockIdx.x * (kFinalizeThreads / 32) + k8;
    if (kk >= count) break;
    const int w = order ? order[first + kk] : first + kk;
    const TensorEntry te = tensors[w];
    if (te.n_chunks < kBigTensorChunks) continue;
    const double acc = tensor_partial_sum_block(partials, te, warp_part);
    if (threadIdx.x == 0) {
      st.sumsq[w] = acc;
      if (decide) {
        adagc_decide(w, acc, cs, ema, st);
        if (kk == 0 && bump_steps) *st.steps_done += 1ull;
      }
    }
  }
}

// AdaGC steps: the norm phase with the per-tensor finalize folded into its tail, so that a step is two launches.
// Here block b owns a contiguous range [range_begin[b], range_begin[b+1]) of the chunks in their original order
// (tensor after tensor), balanced by cost, so a block holds all chunks of most of its tensors and shares at most its
// first and its last tensor with neighbouring blocks.  The streaming loop is that of adagc_norm_kernel.  Afterwards,
// once per block: a tensor whose chunks all lie in this block is complete; for a shared tensor the block adds its
// number of chunks to the tensor's ticket word, and the block whose addition completes the count knows that every
// partial of the tensor is written and visible.  Complete tensors are summed in the fixed order and decided by the
// warps of the block that completed them.  Tickets are integers and nothing waits on them; no floating-point value goes
// through an atomic, and which block completes a tensor does not change any bit of the result.  A ticket word is left
// at zero for the next launch.  Tensors without chunks are not handled here (contexts that list such tensors use the
// separate kernel).
constexpr int kDoneListMax = 1024;  // complete tensors a block collects before it works them off

template <bool kBF16>
__global__ void __launch_bounds__(kThreads, 8)  // as many resident blocks as adagc_norm_kernel: the grid is sized for that
adagc_norm_decide_kernel(const void* __restrict__ grads, const Chunk* __restrict__ chunks,
                         const int32_t* __restrict__ range_begin, double* partials,
                         const TensorEntry* __restrict__ tensors, unsigned int* tickets, ClipScalars cs,
                         float* __restrict__ ema, StatPtrs st, Guard guard) {
  __shared__ double warp_part[2][kThreads / 32];  // alternating from chunk to chunk: one barrier per chunk
  __shared__ int done_list[kDoneListMax];
  __shared__ int n_done;
  griddep_launch_dependents();  // the update kernel may be staged now; it waits for this grid before it needs h
  const int lo = range_begin[blockIdx.x], hi = range_begin[blockIdx.x + 1];
  ADAGC_CHECK_ENTRIES(chunks, lo, hi, guard);
  if (lo >= hi) return;
  Chunk ck = chunks[lo];  // original order: entry c is chunk c, its partial is partials[c]
  int flip = 0;
  bool any_warp_sized = false;
  for (int c = lo; c < hi; ++c) {
    const Chunk ck_next = c + 1 < hi ? chunks[c + 1] : ck;  // one entry ahead, as in adagc_norm_kernel
    if (warp_sized_chunk<kBF16>(ck.count)) {
      any_warp_sized = true;  // left to the warps below
    } else {
      const uint4* vec =
          reinterpret_cast<const uint4*>(static_cast<const char*>(grads) + chunk_start(ck) * (kBF16 ? 2 : 4));
      const double s = block_chunk_sumsq<kBF16, true, false>(vec, ck.count, warp_part[flip]);
      flip ^= 1;
      if (threadIdx.x == 0) partials[c] = s;
    }
    ck = ck_next;
  }
  if (any_warp_sized)
    sum_warp_sized_chunks<kBF16, true>(grads, chunks, lo, hi, partials);
  const int t_first = chunks[lo].tensor, t_last = chunks[hi - 1].tensor;  // tensors with chunks in this block
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) __threadfence();  // this block's partials (written by lane 0 of its warps) are visible device-wide before any ticket is
  for (int t0 = t_first; t0 <= t_last; t0 += kDoneListMax) {  // (one round, unless a block holds over a thousand tensors)
    const int t1 = min(t_last, t0 + kDoneListMax - 1);
    if (threadIdx.x == 0) n_done = 0;
    __syncthreads();
    for (int t = t0 + threadIdx.x; t <= t1; t += kThreads) {
      const TensorEntry te = tensors[t];
      const int mine = min(hi, te.first_chunk + te.n_chunks) - max(lo, te.first_chunk);  // its chunks in this block
      bool complete = mine == te.n_chunks;
      if (!complete) {
        const unsigned int before = atomicAdd(tickets + t, static_cast<unsigned int>(mine));
        complete = before + static_cast<unsigned int>(mine) == static_cast<unsigned int>(te.n_chunks);
        if (complete) tickets[t] = 0u;  // every block that holds a part of the tensor has added its share
      }
      if (complete) done_list[atomicAdd(&n_done, 1)] = t;
    }
    __syncthreads();
    __threadfence();  // (the partials of the other blocks are read below)
    const int n = n_done;
    // tensors of one chunk: a thread each (the fixed-order sum of a single partial is that partial, and a layout of
    // many small tensors would otherwise queue their decisions -- three dependent memory round trips each -- behind one
    // another in eight warps); tensors of a few chunks: one warp each; tensors with very many chunks: the whole block
    for (int k = threadIdx.x; k < n; k += kThreads) {
      const int t = done_list[k];
      const TensorEntry te = tensors[t];
      if (te.n_chunks != 1) continue;
      const double total = __ldcg(partials + te.first_chunk);
      st.sumsq[t] = total;
      adagc_decide(t, total, cs, ema, st);
      if (t == 0) *st.steps_done += 1ull;
    }
    for (int k = warp; k < n; k += kThreads / 32) {
      const int t = done_list[k];
      const TensorEntry te = tensors[t];
      if (te.n_chunks == 1 || te.n_chunks >= kBigTensorChunks) continue;
      const double total = tensor_partial_sum(partials, te, lane);
      if (lane == 0) {
        st.sumsq[t] = total;
        adagc_decide(t, total, cs, ema, st);
        if (t == 0) *st.steps_done += 1ull;
      }
    }
    for (int k = 0; k < n; ++k) {  // uniform over the block
      const int t = done_list[k];
      const TensorEntry te = tensors[t];
      if (te.n_chunks < kBigTensorChunks) continue;
      const double total = tensor_partial_sum_block(partials, te, warp_part[0]);
      if (threadIdx.x == 0) {
        st.sumsq[t] = total;
        adagc_decide(t, total, cs, ema, st);
        if (t == 0) *st.steps_done += 1ull;
      }
    }
    __syncthreads();  // done_list is free again
  }
}

// Sharded use: the per-tensor sums of squares arrive already summed over the ranks that hold parts of each
// tensor (Section 4.3 "Communication": one all-reduce of the partial sums), so phase 2 starts from them.
// One thread per tensor.
__global__ void __launch_bounds__(kFinalizeThreads)
adagc_presummed_finalize_kernel(const double* __restrict__ sumsq_in, ClipScalars cs, int decide,
                                float* __restrict__ ema, StatPtrs st) {
  const int i = blockIdx.x * kFinalizeThreads + threadIdx.x;
  if (i >= cs.n_tensors) return;
  const double s = sumsq_in[i];
  st.sumsq[i] = s;
  if (decide) {
    adagc_decide(i, s, cs, ema, st);
    if (i == 0) *st.steps_done += 1ull;
  }
}

// adagc_set_step_counter: the value travels as a kernel argument, so no host buffer has to outlive the call.
__global__ void adagc_set_counter_kernel(unsigned long long* __restrict__ dst, unsigned long long value) { *dst = value; }

// Capturable step, first launch: derive this step's scalars on the device.  t = steps executed so far + 1, eta_t
// from device memory if the caller keeps it there; the bias corrections 1 - beta^t are formed in float64 like the
// host does for adagc_step and rounded once to the kernels' fp32.
__global__ void adagc_step_prologue_kernel(const unsigned long long* __restrict__ steps_done,
                                           const float* __restrict__ d_lr, StepHyper hh, DeviceStep* __restrict__ out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const long long t = static_cast<long long>(*steps_done) + 1;
  const double lr = d_lr ? (double)*d_lr : hh.lr;
  DeviceStep ds;
  ds.cs.lambda_rel = hh.lambda_rel;
  ds.cs.beta = hh.beta;
  ds.cs.one_minus_beta = 1.0 - hh.beta;
  ds.cs.lambda_abs = hh.lambda_abs;
  ds.cs.step = t;
  ds.cs.n_tensors = hh.n_tensors;
  ds.cs.seed = (t == 1 && !hh.keep_initial) ? 1 : 0;
  ds.cs.ema_cap = hh.ema_cap;
  const double bc1 = 1.0 - pow(hh.beta1, (double)t);
  const double bc2 = 1.0 - pow(hh.beta2, (double)t);
  ds.a.beta1 = (float)hh.beta1;
  ds.a.one_minus_beta1 = (float)(1.0 - hh.beta1);
  ds.a.beta2 = (float)hh.beta2;
  ds.a.one_minus_beta2 = (float)(1.0 - hh.beta2);
  ds.a.inv_bc2 = (float)(1.0 / bc2);
  ds.a.step_size = (float)(lr / bc1);
  ds.a.decay = (float)(1.0 - lr * hh.wd);
  ds.a.eps = (float)hh.eps;
  ds.in_warmup = t <= hh.warmup ? 1 : 0;
  ds.pad = 0;
  *out = ds;
}

// Warm-up branch of Algorithm 1: global norm (Eq. 2), one clip factor for every tensor, and
// gamma_t,i = min{gamma_t-1,i, ||hat(g)_t,i||} with gamma_0,i = ||hat(g)_1,i||.  One block.
// Body for one block of kBlock threads (warp_part: kBlock / 32 doubles of shared memory, total_s: one).
template <int kBlock>
__device__ __forceinline__ void warmup_finalize_block(const ClipScalars& cs, float* __restrict__ ema, const StatPtrs& st,
                                                      double* warp_part, double* total_s_ptr) {
  const int tid = threadIdx.x;
  double acc = 0.0;
  for (int i = tid; i < cs.n_tensors; i += kBlock) acc += st.sumsq[i];
  acc = warp_sum(acc);
  if ((tid & 31) == 0) warp_part[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double s = warp_part[0];
    for (int k = 1; k < kBlock / 32; ++k) s += warp_part[k];
    *total_s_ptr = s;
    *st.steps_done += 1ull;
  }
  __syncthreads();
  const double total_s = *total_s_ptr;
  constexpr int kWarmupThreads = kBlock;  // stride of the per-tensor loop below
  const double G = sqrt(total_s);  // ||g_t||
  const bool clip_all = G > cs.lambda_abs;
  const double h = clip_all ? __ddiv_rn(cs.lambda_abs, G) : 1.0;  // min{lambda_abs / ||g_t||, 1}
  const float hf = (float)h;
  for (int i = tid; i < cs.n_tensors; i += kWarmupThreads) {
    const double s = st.sumsq[i];
    const double n = sqrt(s);
    const double c = __dmul_rn(h, n);  // ||hat(g)_t,i||
    double g_new = c;
    if (cs.ema_cap > 0.0) {  // the constant stands where gamma_t-1,i stands in the default
      g_new = (c < cs.ema_cap) ? c : cs.ema_cap;
    } else if (!cs.seed) {
      const double g_prev = (double)ema[i];
      g_new = (c < g_prev) ? c : g_prev;
    }
    ema[i] = (float)g_new;
    st.norm[i] = (float)n;
    st.h[i] = hf;
    st.flag[i] = clip_all ? 1 : 0;
    if (clip_all) st.clip_count[i] += 1ull;
    if (!isfinite(s)) atomicOr(st.status, ADAGC_W_NONFINITE);
  }
}

__global__ void __launch_bounds__(kWarmupThreads)
adagc_warmup_finalize_kernel(ClipScalars cs, float* __restrict__ ema, StatPtrs st,
                             const DeviceStep* __restrict__ ds = nullptr) {
  if (ds) {  // capturable step: always launched, does nothing outside warm-up
    if (!ds->in_warmup) return;
    cs = ds->cs;
  }
  __shared__ double warp_part[kWarmupThreads / 32];
  __shared__ double total_s;
  warmup_finalize_block<kWarmupThreads>(cs, ema, st, warp_part, &total_s);
}

// "Global AdaGC" (the adaptivity / locality ablation of Section 5): one adaptive threshold for the whole
// model, i.e. Algorithm 1 applied to the single tensor that all gradients form together.  One block;
// every tensor receives the same clip factor, flag and gamma.  `in_warmup` selects Eq. 2 or Eq. 3.
__global__ void __launch_bounds__(kWarmupThreads)
adagc_global_finalize_kernel(ClipScalars cs, int in_warmup, float* __restrict__ ema, StatPtrs st,
                             const DeviceStep* __restrict__ ds = nullptr) {
  if (ds) {
    cs = ds->cs;
    in_warmup = ds->in_warmup;
  }
  __shared__ double warp_part[kWarmupThreads / 32];
  __shared__ double total_s;
  const int tid = threadIdx.x;
  double acc = 0.0;
  for (int i = tid; i < cs.n_tensors; i += kWarmupThreads) acc += st.sumsq[i];
  acc = warp_sum(acc);
  if ((tid & 31) == 0) warp_part[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double s = warp_part[0];
    for (int k = 1; k < kWarmupThreads / 32; ++k) s += warp_part[k];
    total_s = s;
    *st.steps_done += 1ull;
  }
  __syncthreads();
  const double G = sqrt(total_s);        // the norm of the one big tensor
  const double g_in = (double)ema[0];    // read by every thread before anyone overwrites it ...
  __syncthreads();                       // ... which this barrier guarantees
  bool clip;
  double h, g_new;
  if (in_warmup) {
    clip = G > cs.lambda_abs;
    h = clip ? __ddiv_rn(cs.lambda_abs, G) : 1.0;
    const double c = __dmul_rn(h, G);
    if (cs.ema_cap > 0.0) g_new = (c < cs.ema_cap) ? c : cs.ema_cap;
    else g_new = cs.seed ? c : ((c < g_in) ? c : g_in);
  } else {
    double g_prev = cs.seed ? (double)(float)G : g_in;
    if (cs.seed && cs.ema_cap > 0.0 && !(g_prev < cs.ema_cap)) g_prev = cs.ema_cap;
    const double thr = __dmul_rn(cs.lambda_rel, g_prev);
    clip = G > thr;
    h = clip ? __ddiv_rn(thr, G) : 1.0;
    const double c = clip ? thr : G;
    g_new = __dadd_rn(__dmul_rn(cs.beta, g_prev), __dmul_rn(cs.one_minus_beta, c));
  }
  const float hf = (float)h, gf = (float)g_new;
  for (int i = tid; i < cs.n_tensors; i += kWarmupThreads) {
    const double s = st.sumsq[i];
    ema[i] = gf;
    st.norm[i] = (float)sqrt(s);
    st.h[i] = hf;
    st.flag[i] = clip ? 1 : 0;
    if (clip) st.clip_count[i] += 1ull;
    if (!isfinite(s)) atomicOr(st.status, ADAGC_W_NONFINITE);
  }
}

}  // namespace
