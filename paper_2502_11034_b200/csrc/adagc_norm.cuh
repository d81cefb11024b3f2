// Phase 1: per-chunk sums of squares (Eq. 3 needs ||g_t,i||, Eq. 2 ||g_t||): the block-wide and warp-wide chunk sums and
// adagc_norm_kernel.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

// ------------------------------------------------------------------------------------------------
// phase 1: per-chunk sums of squares (Eq. 3: ||g_t,i||^2 = sum_j g_ij^2)
// ------------------------------------------------------------------------------------------------
// Sum of squares of `count` elements starting at the 16-byte aligned `vec`, by one block of kThreads
// threads: fixed element -> thread mapping, float64 per-thread accumulators, fixed shuffle tree, then a
// fixed-order sum of the warp totals.  The result is valid in thread 0.  Ends with a barrier, so
// `warp_part` can be reused at once.
// kKeepInL2: load with the evict_last policy (the step's norm phase, whose gradient is read again by the update).
// One 16-byte vector of gradients added to a thread's two accumulators (components alternate between them).
template <bool kBF16>
__device__ __forceinline__ void sq_acc_vec(const uint4& q, double& acc0, double& acc1) {
  if (kBF16) {
    acc0 = sq_acc(acc0, bf16_lo(q.x));
    acc1 = sq_acc(acc1, bf16_hi(q.x));
    acc0 = sq_acc(acc0, bf16_lo(q.y));
    acc1 = sq_acc(acc1, bf16_hi(q.y));
    acc0 = sq_acc(acc0, bf16_lo(q.z));
    acc1 = sq_acc(acc1, bf16_hi(q.z));
    acc0 = sq_acc(acc0, bf16_lo(q.w));
    acc1 = sq_acc(acc1, bf16_hi(q.w));
  } else {
    acc0 = sq_acc(acc0, __uint_as_float(q.x));
    acc1 = sq_acc(acc1, __uint_as_float(q.y));
    acc0 = sq_acc(acc0, __uint_as_float(q.z));
    acc1 = sq_acc(acc1, __uint_as_float(q.w));
  }
}

// kRounds rounds of the block over the vectors from `base` on: thread tid takes base + u * kThreads + tid, u = 0 ..
// kRounds - 1, all loads issued before the first addition.  Every vector exists (the caller checks).
template <bool kBF16, bool kKeepInL2, int kRounds>
__device__ __forceinline__ void sq_acc_rounds(const uint4* __restrict__ vec, int base, uint64_t keep, double& acc0,
                                              double& acc1) {
  uint4 q[kRounds];
#pragma unroll
  for (int u = 0; u < kRounds; ++u) {
    const uint4* ptr = vec + base + u * kThreads + threadIdx.x;
    q[u] = kKeepInL2 ? ld_nc_l2_hint(ptr, keep) : __ldg(ptr);
  }
#pragma unroll
  for (int u = 0; u < kRounds; ++u) sq_acc_vec<kBF16>(q[u], acc0, acc1);
}

// kTrailingBarrier = false leaves the second barrier out: the caller then alternates between two `warp_part` arrays
// from one call to the next (thread 0 reads one while the other warps already fill the other for the next chunk).
template <bool kBF16, bool kKeepInL2 = false, bool kTrailingBarrier = true>
__device__ __forceinline__ double block_chunk_sumsq(const uint4* __restrict__ vec, int count, double* warp_part) {
  constexpr int kEPV = kBF16 ? 8 : 4;  // elements per 16-byte vector
  const int tid = threadIdx.x;
  const int nvec = count / kEPV;
  double acc0 = 0.0, acc1 = 0.0;
  const uint64_t keep = kKeepInL2 ? l2_policy_evict_last() : 0ull;
  // Every thread adds its vectors (tid, tid + kThreads, ...) in increasing order.  Eight rounds at a time keep eight
  // independent loads per thread in flight; what is left after the last full eight goes in batches of four, two
  // and one round and a last, partial round, so that a short chunk executes instructions for its own vectors only
  // (the norm of a layout of many small tensors is bound by instruction issue, not by memory).
  int base = 0;
  for (; base + 8 * kThreads <= nvec; base += 8 * kThreads) sq_acc_rounds<kBF16, kKeepInL2, 8>(vec, base, keep, acc0, acc1);
  if (base + 4 * kThreads <= nvec) {
    sq_acc_rounds<kBF16, kKeepInL2, 4>(vec, base, keep, acc0, acc1);
    base += 4 * kThreads;
  }
  if (base + 2 * kThreads <= nvec) {
    sq_acc_rounds<kBF16, kKeepInL2, 2>(vec, base, keep, acc0, acc1);
    base += 2 * kThreads;
  }
  if (base + kThreads <= nvec) {
    sq_acc_rounds<kBF16, kKeepInL2, 1>(vec, base, keep, acc0, acc1);
    base += kThreads;
  }
  if (base + tid < nvec) sq_acc_rounds<kBF16, kKeepInL2, 1>(vec, base, keep, acc0, acc1);
  // ragged tail of a tensor's last chunk (fewer than one vector)
  const int t = nvec * kEPV + tid;
  if (t < count) {
    float x;
    if (kBF16) {
      x = __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(vec)[t]) << 16);
    } else {
      x = reinterpret_cast<const float*>(vec)[t];
    }
    acc0 = sq_acc(acc0, x);
  }
  const double w = warp_sum(acc0 + acc1);
  if ((tid & 31) == 0) warp_part[tid >> 5] = w;
  __syncthreads();
  double s = 0.0;
  if (tid == 0) {
    s = warp_part[0];
#pragma unroll
    for (int k = 1; k < kThreads / 32; ++k) s += warp_part[k];
  }
  if (kTrailingBarrier) __syncthreads();
  return s;
}

// A chunk of at most kThreads vectors gives every thread of block_chunk_sumsq at most one vector, so a single warp can
// stand in for the whole block with identical bits: in turn k it plays the block's warp k (lane l is thread 32 k + l:
// its one vector, then -- thread < 8 only -- its element of the ragged tail), takes that warp's shuffle-tree total, and
// adds the totals in warp order.  Warps of the block that hold no data contribute an exact +0 and are left out.
// The norm kernels hand such chunks to their warps one each (no block barrier, eight chunks in flight per block): with
// one short chunk at a time per block they are bound by the latency of a chunk, not by memory.
template <bool kBF16>
__device__ __forceinline__ bool warp_sized_chunk(int count) { return count / (kBF16 ? 8 : 4) <= kThreads; }

template <bool kBF16, bool kKeepInL2>
__device__ __forceinline__ double warp_chunk_sumsq(const uint4* __restrict__ vec, int count) {
  constexpr int kEPV = kBF16 ? 8 : 4;
  const int lane = threadIdx.x & 31;
  const int nvec = count / kEPV;  // <= kThreads
  const int turns = max(1, (nvec + 31) >> 5);
  const uint64_t keep = kKeepInL2 ? l2_policy_evict_last() : 0ull;
  double total = 0.0;
#pragma unroll 1
  for (int k0 = 0; k0 < turns; k0 += 4) {  // four turns' loads in flight at a time
    uint4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = 32 * (k0 + u) + lane;
      q[u] = i < nvec ? (kKeepInL2 ? ld_nc_l2_hint(vec + i, keep) : __ldg(vec + i)) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int k = k0 + u;
      if (k >= turns) break;  // uniform
      double acc0 = 0.0, acc1 = 0.0;
      if (32 * k + lane < nvec) sq_acc_vec<kBF16>(q[u], acc0, acc1);
      if (k == 0) {
        const int t = nvec * kEPV + lane;
        if (t < count) {
          const float x = kBF16 ? __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(vec)[t]) << 16)
                                : reinterpret_cast<const float*>(vec)[t];
          acc0 = sq_acc(acc0, x);
        }
      }
      const double w = warp_sum(acc0 + acc1);
      total = k == 0 ? w : total + w;
    }
  }
  return total;
}

// The warp-sized chunks among the table entries [lo, hi), dealt to the block's warps in turn; lane 0 of the warp that
// summed entry c stores the sum at partials[c] (kIndexIsEntry: the table is in chunk order) or at the entry's partial
// index.  Not inlined: the streaming loop of the calling kernel keeps its register allocation to itself.
template <bool kBF16, bool kIndexIsEntry>
__device__ __noinline__ void sum_warp_sized_chunks(const void* __restrict__ grads, const Chunk* __restrict__ chunks, int lo,
                                                   int hi, double* __restrict__ partials) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int seen = 0;  // warp-sized chunks before `base`
  for (int base = lo; base < hi; base += 32) {
    Chunk e{0u, 0, 0, 0};
    bool mine_is_small = false;
    if (base + lane < hi) {
      e = chunks[base + lane];
      mine_is_small = warp_sized_chunk<kBF16>(e.count);
    }
    const unsigned small = __ballot_sync(0xffffffffu, mine_is_small);
    for (unsigned rest = small; rest != 0; rest &= rest - 1) {  // uniform over the warp
      const int j = __ffs(rest) - 1;
      const int rank = seen + __popc(small & ((1u << j) - 1u));
      if ((rank & (kThreads / 32 - 1)) != warp) continue;
      const uint32_t start4 = __shfl_sync(0xffffffffu, e.start4, j);
      const int count = __shfl_sync(0xffffffffu, e.count, j);
      const int partial = __shfl_sync(0xffffffffu, e.partial, j);
      const uint4* vec = reinterpret_cast<const uint4*>(static_cast<const char*>(grads) +
                                                        static_cast<int64_t>(start4) * 4 * (kBF16 ? 2 : 4));
      const double s = warp_chunk_sumsq<kBF16, true>(vec, count);
      if (lane == 0) partials[kIndexIsEntry ? base + j : partial] = s;
    }
    seen += __popc(small);
  }
}

template <bool kBF16>
__global__ void __launch_bounds__(kThreads, 8)  // eight resident blocks per SM: the norm and scale grids are sized for that
adagc_norm_kernel(const void* __restrict__ grads, const Chunk* __restrict__ chunks,
                  const int32_t* __restrict__ block_begin, double* __restrict__ partials, Guard guard) {
  __shared__ double warp_part[2][kThreads / 32];  // alternating from chunk to chunk: one barrier per chunk
  const int c_begin = block_begin[blockIdx.x], c_end = block_begin[blockIdx.x + 1];
  ADAGC_CHECK_ENTRIES(chunks, c_begin, c_end, guard);
  if (c_begin >= c_end) return;
  Chunk ck = chunks[c_begin];
  int flip = 0;
  bool any_warp_sized = false;
  for (int c = c_begin; c < c_end; ++c) {
    // the next table entry is fetched while this chunk streams: a block of many small chunks would otherwise wait for
    // a dependent load before every chunk's first gradient load
    const Chunk ck_next = c + 1 < c_end ? chunks[c + 1] : ck;
    if (warp_sized_chunk<kBF16>(ck.count)) {
      any_warp_sized = true;  // left to the warps below
    } else {
      const uint4* vec =
          reinterpret_cast<const uint4*>(static_cast<const char*>(grads) + chunk_start(ck) * (kBF16 ? 2 : 4));
      const double s = block_chunk_sumsq<kBF16, true, false>(vec, ck.count, warp_part[flip]);
      flip ^= 1;
      if (threadIdx.x == 0) partials[ck.partial] = s;
    }
    ck = ck_next;
  }
  if (any_warp_sized)
    sum_warp_sized_chunks<kBF16, false>(grads, chunks, c_begin, c_end, partials);
}

}  // namespace
