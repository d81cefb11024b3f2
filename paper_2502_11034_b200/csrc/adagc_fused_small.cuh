// Small layouts: the whole step as one cooperative kernel.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

// ------------------------------------------------------------------------------------------------
// Small layouts: the whole step in ONE kernel.  When the arenas are a few MB, the three dependent launches of a
// step cost more than the data movement; here every block computes the partial sums of its chunks, the grid
// meets at a barrier, the decisions are taken (one warp per tensor; warm-up: block 0 after one more barrier), the
// grid meets again and every block updates its chunks.  The kernel is launched cooperatively, so all blocks are
// resident and the barriers cannot deadlock; each wait is bounded all the same.
// ------------------------------------------------------------------------------------------------
// Barrier number `index` (counted over all launches of this context) of a grid of gridDim.x blocks on a counter that
// only ever grows.  Returns false if the other blocks did not arrive within the time limit.
__device__ __forceinline__ bool grid_barrier_bounded(unsigned long long* counter, unsigned long long index) {
  __shared__ int arrived_flag;
  __syncthreads();  // this block's work before the barrier is complete ...
  if (threadIdx.x == 0) {
    __threadfence();  // ... and visible to the other blocks before the arrival is
    atomicAdd(counter, 1ull);
    const unsigned long long target = (index + 1ull) * gridDim.x;
    const uint64_t t0 = global_timer_ns();
    int ok = 1;
    for (uint32_t spins = 1; *reinterpret_cast<volatile unsigned long long*>(counter) < target; ++spins) {
      if ((spins & 63u) == 0 && global_timer_ns() - t0 > kWaitLimitNs) {
        ok = 0;
        break;
      }
    }
    __threadfence();
    arrived_flag = ok;
  }
  __syncthreads();
  return arrived_flag != 0;
}

// Work unit of the one-kernel step: a slice of kSlice elements of a chunk, so that a layout of a few dozen chunks
// still spreads over every SM.  Unit u = 4 * (table position of the chunk) + (slice in the chunk); block b takes the
// units b, b + gridDim.x, ...  Each slice has its own partial sum (slot 4 * chunk + slice; slots of slices a short
// chunk does not have stay zero), and a tensor's sum of squares is the fixed-order sum of its slots.
constexpr int kSlice = 4096;
constexpr int kSlicesPerChunk = kChunkElems / kSlice;

template <bool kBF16, bool kSB>
__global__ void __launch_bounds__(kThreads)
adagc_fused_small_kernel(float* __restrict__ params, const void* __restrict__ grads, void* __restrict__ m_arena,
                         void* __restrict__ v_arena, float* ema, const Chunk* __restrict__ chunks, int n_chunks,
                         const TensorEntry* __restrict__ tensors, double* slice_partials, ClipScalars cs, int in_warmup,
                         AdamScalars a, StatPtrs st, unsigned long long* barrier_counter,
                         unsigned long long barrier_index, float* gamma_prev, Guard guard, StateRounding sr) {
  __shared__ double warp_part[kThreads / 32];
  __shared__ double total_s;
  __shared__ float h_shared;
  ADAGC_CHECK_ENTRIES(chunks, 0, n_chunks, guard);  // (every block checks the whole table, so all of them agree)
  const int n_units = n_chunks * kSlicesPerChunk;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  auto slices_of = [](const TensorEntry te) {
    TensorEntry x;
    x.first_chunk = te.first_chunk * kSlicesPerChunk;
    x.n_chunks = te.n_chunks * kSlicesPerChunk;
    return x;
  };
  // phase 1: sums of squares of this block's slices; the block that holds a tensor's very first slice also sets
  // aside the gamma the step starts from, so that after the barrier any block can take that tensor's decision
  for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
    const Chunk ck = chunks[u / kSlicesPerChunk];
    const int k = u % kSlicesPerChunk, begin = k * kSlice;
    if (begin >= ck.count) continue;  // uniform over the block
    const int count = min(kSlice, ck.count - begin);
    const uint4* vec = reinterpret_cast<const uint4*>(static_cast<const char*>(grads) +
                                                      (chunk_start(ck) + begin) * (kBF16 ? 2 : 4));
    const double s = block_chunk_sumsq<kBF16>(vec, count, warp_part);
    if (threadIdx.x == 0) {
      slice_partials[ck.partial * kSlicesPerChunk + k] = s;
      if (!in_warmup && k == 0 && ck.partial == tensors[ck.tensor].first_chunk) gamma_prev[ck.tensor] = ema[ck.tensor];
    }
  }
  bool ok = grid_barrier_bounded(barrier_counter, barrier_index);
  if (ok && in_warmup) {
    // warm-up step: the global norm couples all tensors, so the decisions wait for every tensor's sum
    const int warps = gridDim.x * (kThreads / 32);
    for (int w = blockIdx.x * (kThreads / 32) + warp; w < cs.n_tensors; w += warps) {
      const double acc = tensor_partial_sum(slice_partials, slices_of(tensors[w]), lane);
      if (lane == 0) st.sumsq[w] = acc;
    }
    ok = grid_barrier_bounded(barrier_counter, barrier_index + 1);
    if (ok && blockIdx.x == 0) warmup_finalize_block<kThreads>(cs, ema, st, warp_part, &total_s);
    if (ok) ok = grid_barrier_bounded(barrier_counter, barrier_index + 2);
  }
  if (!ok) {
    if (threadIdx.x == 0) atomicOr(st.status, ADAGC_E_TIMEOUT);
    return;
  }
  if (!in_warmup) {
    // AdaGC step: no further barrier.  Every block takes the decision of the tensors its slices belong to (same
    // partials, same order, same gamma: same bits in every block); only the block that holds a tensor's very first
    // slice writes gamma and the statistics.  Tensors without any chunk are handled by a grid-wide loop.
    const int warps = gridDim.x * (kThreads / 32);
    for (int w = blockIdx.x * (kThreads / 32) + warp; w < cs.n_tensors; w += warps) {
      if (tensors[w].n_chunks != 0 || lane != 0) continue;
      st.sumsq[w] = 0.0;
      adagc_decide(w, 0.0, cs, ema, st);
      if (w == 0) *st.steps_done += 1ull;
    }
  }
  int cur = -1, row_base = 0, first_chunk = -1;
  float h = 1.0f;
  Decision d = {};
  double s_cur = 0.0;
  for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
    const Chunk ck = chunks[u / kSlicesPerChunk];
    const int k = u % kSlicesPerChunk, begin = k * kSlice;
    if (begin >= ck.count) continue;
    if (ck.tensor != cur) {  // uniform over the block
      cur = ck.tensor;
      if (in_warmup) {
        h = __ldcg(st.h + cur);  // written by block 0 of this launch
      } else {
        __syncthreads();  // everyone has read h_shared of the previous tensor
        if (warp == 0) {
          const TensorEntry te = tensors[cur];
          s_cur = tensor_partial_sum(slice_partials, slices_of(te), lane);
          first_chunk = te.first_chunk;
          d = adagc_decision(s_cur, __ldcg(gamma_prev + cur), cs);
          if (lane == 0) h_shared = (float)d.h;
        }
        __syncthreads();
        h = h_shared;
      }
    }
    if (!in_warmup && threadIdx.x == 0 && k == 0 && ck.partial == first_chunk) {  // this block owns the tensor's record
      st.sumsq[cur] = s_cur;
      adagc_commit(cur, s_cur, d, ema, st);
      if (cur == 0) *st.steps_done += 1ull;
    }
    Chunk sub = ck;
    sub.start4 = ck.start4 + static_cast<uint32_t>(begin / 4);
    sub.count = min(kSlice, ck.count - begin);
    adamw_partial_chunk<kBF16, kThreads, kOptAdamW, kSB>(sub, h, row_base, params, grads, m_arena, v_arena, a, nullptr, &sr);
  }
}

}  // namespace
