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
// Host side (second half of the file): descriptor validation, the balanced per-block chunk tables
// built once at adagc_create, the entry points, and adagc_step_host, which pipelines groups of
// tensors behind the host-to-device copies.
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

namespace {

constexpr int kChunkElems = 16384;  // elements per chunk; multiple of 8 keeps every chunk 16-byte aligned
constexpr int kThreads = 256;
constexpr int kFinalizeThreads = 256;  // 8 warps = 8 tensors per block
constexpr int kWarmupThreads = 1024;
// The update kernel moves 7 streams (4 read, 3 written).  Measured on B200, DRAM efficiency of that mix
// peaks with about 57 KB of loads in flight per SM and drops by ~15 % with twice as many.
// Register-streaming variant: 512 threads x 112 bytes, i.e. a grid of two 256-thread blocks per SM, with
// the largest L1 carve-out (L1 lines hold the loads in flight; reserving 100 KB of shared memory per
// block cost 20 % of the bandwidth).  Bulk-async variant: one 512-thread block per SM with one 57 KB
// tile in flight; it measured 1-2 % faster on every layout tried (26.7 vs 27.2 ms on the 7B-shaped one)
// and is the default; the descriptor's flags can force either.
constexpr int kUpdateBlocksPerSM = 2;

struct Chunk {
  uint32_t start4;  // element offset into the arenas, in units of 4 elements
  int32_t count;    // elements in this chunk (<= kChunkElems)
  int32_t tensor;   // owning tensor
  int32_t partial;  // index of this chunk's partial sum: chunks of a tensor are numbered consecutively
};
static_assert(sizeof(Chunk) == 16, "chunk entries are 16 bytes");
__host__ __device__ __forceinline__ int64_t chunk_start(const Chunk& c) { return static_cast<int64_t>(c.start4) * 4; }

// What every kernel that walks a chunk table is told about the context, so that a build with -DADAGC_BOUNDS_CHECK can
// verify the entries it is about to use before the first access (a debugging build: the tables are written once by
// adagc_create from a validated descriptor, so a violation means a corrupted workspace or a defect of the table builder).
struct Guard {
  long long arena_elems;  // every chunk must end at or before this element
  int n_chunks;           // table length; also the number of partial sums
  int n_tensors;
  int* status;            // device status word: ADAGC_E_BOUNDS is set here
};

__host__ __device__ __forceinline__ bool chunk_entry_ok(const Chunk& c, long long arena_elems, int n_chunks, int n_tensors) {
  return c.count > 0 && c.count <= kChunkElems && c.tensor >= 0 && c.tensor < n_tensors && c.partial >= 0 &&
         c.partial < n_chunks && chunk_start(c) + c.count <= arena_elems;
}

// Chunks are handed to thread blocks by a table built once on the host: block b owns the entries
// [block_begin[b], block_begin[b+1]) of its kernel's table.  The assignment balances elements (plus a
// fixed cost per chunk) over the blocks; with equal chunks it is plain round-robin.
constexpr int kMaxGrid = 8192;          // entries reserved for each block_begin array
// per-chunk cost added to the element count; measured on the layout of 20 000 small tensors: the norm / scale grid
// (two block barriers and a table fetch per chunk) balances best with a larger constant than the update grid
constexpr int kChunkFixedCost = 1024;
constexpr int kChunkFixedCostWide = 8192;
constexpr int64_t kFusedMaxChunks = 4096;  // largest layout (64 Mi elements) the one-kernel step accepts
// adagc_step_host in steady state: the tensors are cut (in arena order) into at most kMaxGroups groups; each
// group's gradients are copied on a second stream while the previous groups run norm/finalize/update.
constexpr int kMaxGroups = 64;
constexpr int kGroupMaxGrid = 1536;              // blocks per group launch (per block_begin array)
constexpr int64_t kGroupMinBytes = 64ll << 20;   // smallest gradient slice worth its own launches

struct TensorEntry {
  int32_t first_chunk;
  int32_t n_chunks;
};

struct ClipScalars {
  double lambda_rel, beta, one_minus_beta, lambda_abs;
  int64_t step;
  int32_t n_tensors;
  int32_t seed;  // 1: gamma is seeded at this step (t = 1, unless the descriptor keeps the caller's gamma_0)
  double ema_cap;  // > 0: "thresholded initialization" -- seeding and warm-up set gamma = min(clipped norm, ema_cap)
};

struct AdamScalars {
  float beta1, one_minus_beta1, beta2, one_minus_beta2;
  float inv_bc2;    // 1 / (1 - beta2^t)
  float step_size;  // lr / (1 - beta1^t)
  float decay;      // 1 - lr * wd
  float eps;
};

// Scalars of one step kept in device memory: written by adagc_step_prologue_kernel from the device-side step
// counter, read by the phases of a capturable step (the launches then carry nothing that changes from step to step).
struct DeviceStep {
  ClipScalars cs;
  AdamScalars a;
  int32_t in_warmup;  // t <= T_start
  int32_t pad;
};

struct StepHyper {  // what the host hands to the prologue kernel
  double lr, beta1, beta2, eps, wd, lambda_rel, beta, lambda_abs, ema_cap;
  int64_t warmup;
  int32_t n_tensors, keep_initial;
};

// ------------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;  // identical in every lane: each level adds the same two values in both partners
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while its
// predecessor in the stream is still running, once every block of the predecessor has executed launch_dependents (or
// exited); griddep_wait returns when the predecessor grid has completed and its writes are visible.  Both are no-ops
// in a kernel that was launched the ordinary way.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// round-to-nearest-even float -> bf16 bits (NaN stays NaN)
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (u >> 16) | 0x40u;
  u += 0x7fffu + ((u >> 16) & 1u);
  return u >> 16;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}

// the same rounding by the conversion instruction (one instruction per pair; NaN becomes the canonical NaN)
__device__ __forceinline__ uint32_t pack_bf16_cvt(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// Stochastic rounding of stored bfloat16 moments (adagc_set_state_rounding).  Random numbers: Philox4x32-10, the
// counter-based generator of Salmon, Moraes, Dror and Shaw (SC 2011), from its definition: ten rounds that replace the
// counter (c0, c1, c2, c3) by (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)), the key bumped by
// (W0, W1) between rounds.  The four elements 4q .. 4q+3 of the arenas share one call with counter
// (lo q, hi q, lo step, hi step) and key (lo seed, hi seed); element 4q + l takes output word l, the low half for m,
// the high half for v.
struct StateRounding {
  uint32_t seed_lo, seed_hi, step_lo, step_hi;
  int stochastic;  // 0: round to nearest even
};
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
  constexpr uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u, kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(kM0, c0), lo0 = kM0 * c0, hi1 = __umulhi(kM1, c2), lo1 = kM1 * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += kW0;  // (the bump after the last round is never used)
    k1 += kW1;
  }
  return make_uint4(c0, c1, c2, c3);
}
__device__ __forceinline__ uint4 rounding_words(int64_t q, const StateRounding& sr) {
  return philox4x32_10(static_cast<uint32_t>(q), static_cast<uint32_t>(static_cast<uint64_t>(q) >> 32), sr.step_lo, sr.step_hi,
                       sr.seed_lo, sr.seed_hi);
}
// x moves to its bfloat16 neighbour of larger magnitude with probability (distance to the smaller one) / spacing: the
// 16-bit random number is added to the low half of the bit pattern and that half is dropped.  This is what the
// stochastic-rounding conversion instruction computes (checked on B200 against the integer formula for finite values,
// subnormals and overflow included: the low result takes the second source and random bits 15..0, the high result
// the first source and bits 31..16); infinities stay, NaN stays NaN.
__device__ __forceinline__ uint32_t pack_bf16_stochastic(float lo, float hi, uint32_t r_lo_hi) {
  uint32_t d;
  asm("cvt.rs.bf16x2.f32 %0, %1, %2, %3;" : "=r"(d) : "f"(hi), "f"(lo), "r"(r_lo_hi));
  return d;
}
// four values with the four words of their group; which = 0: low halves (m), 1: high halves (v)
__device__ __forceinline__ uint2 pack4_stochastic(const float4& x, const uint4& w, int which) {
  const uint32_t sel = which ? 0x7632u : 0x5410u;  // the chosen halves of two words, side by side
  return make_uint2(pack_bf16_stochastic(x.x, x.y, __byte_perm(w.x, w.y, sel)),
                    pack_bf16_stochastic(x.z, x.w, __byte_perm(w.z, w.w, sel)));
}

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }

// L2 eviction-priority policies (createpolicy) and loads that carry one.  The norm kernel marks the gradient lines
// it reads evict_last; the bulk-async update kernel marks everything it moves evict_first, and the register paths
// (partial chunks, the register-streaming update kernel, the clip-only scale kernel) make their one read of the
// gradient an evict_first load, which hands those lines back.  Measured on B200 with
// all three hints together: 29.12 -> 28.73 ms on the 7B-shaped layout, 5.36 -> 5.30 ms on the 1B-shaped one,
// 1.065 -> 1.039 ms on the layout of 20 000 small tensors, no change on the GPT-2-small-shaped one; any subset of
// the hints alone measured slower than none.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint4 ld_nc_l2_hint(const uint4* ptr, uint64_t policy) {
  uint4 v;
  asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr), "l"(policy));
  return v;
}

__device__ __forceinline__ uint4 ld_l2_hint(const uint4* ptr, uint64_t policy) {  // coherent variant (in-place users)
  uint4 v;
  asm volatile("ld.global.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr), "l"(policy)
               : "memory");
  return v;
}

__device__ __forceinline__ double sq_acc(double acc, float x) {
  const double d = (double)x;
  return fma(d, d, acc);
}

#ifdef ADAGC_BOUNDS_CHECK
// Checked build: the whole block verifies the table entries [first, last) it is about to walk.  On a violation the
// status bit is set and false is returned to every thread, and the block returns without touching the arenas.
__device__ __forceinline__ bool block_entries_ok(const Chunk* __restrict__ chunks, int first, int last, const Guard& g) {
  int ok = first >= 0 && first <= last && last <= g.n_chunks;
  if (ok)
    for (int c = first + threadIdx.x; c < last; c += blockDim.x)
      ok = ok && chunk_entry_ok(chunks[c], g.arena_elems, g.n_chunks, g.n_tensors);
  ok = __syncthreads_and(ok);
  if (!ok && threadIdx.x == 0) atomicOr(g.status, ADAGC_E_BOUNDS);
  return ok != 0;
}
#define ADAGC_CHECK_ENTRIES(chunks, first, last, guard) \
  if (!block_entries_ok(chunks, first, last, guard)) return
#else
#define ADAGC_CHECK_ENTRIES(chunks, first, last, guard) (void)(guard)
#endif

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

// ------------------------------------------------------------------------------------------------
// phase 3: AdamW on the clipped gradient (last four lines of Algorithm 1)
// ------------------------------------------------------------------------------------------------
// kOpt selects the optimizer applied to the clipped gradient: AdamW (Algorithm 1) or Lion (Section 4.2
// names it as another optimizer the clip is used with; its rule is c = beta1 m + (1-beta1) hat(g),
// theta -= lr (sign(c) + wd theta), m = beta2 m + (1-beta2) hat(g); one state stream, no v).
constexpr int kOptAdamW = 0;
constexpr int kOptLion = 1;
constexpr int kOptSgdM = 2;  // heavy-ball SGD: d = hat(g) + wd theta, m = momentum m + d, theta -= lr m (no v)

// The quotient m_hat / (sqrt(v_hat) + eps) by the approximate square root and reciprocal (subnormals flushed), four
// instructions instead of about twenty.  Used only where the moments are rounded stochastically to bfloat16: there
// the update already carries a random relative error of 2^-9 per moment, the kernel is bound by instruction issue (the
// random numbers cost about 22 instructions per element), and a few 1e-7 more on theta's increment are invisible.
__device__ __forceinline__ float quotient_approx(float m, float v_hat, float eps) {
  float s, r;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(s) : "f"(v_hat));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(s + eps));
  return m * r;
}
// (a subnormal v_hat is flushed to zero, which is harmless as long as eps is not itself vanishing)
__device__ __forceinline__ bool use_quotient_approx(const StateRounding* sr, const AdamScalars& a) {
  return sr != nullptr && sr->stochastic && a.eps >= 1e-30f;
}

template <int kOpt>
__device__ __forceinline__ void adamw_elem(float g, float h, float& p, float& m, float& v,
                                           const AdamScalars& a, bool fast = false) {
  const float gh = h * g;  // hat(g)
  if (kOpt == kOptLion) {
    // fp32 like the rest of the update; where the two terms nearly cancel the sign is a near-tie
    const float c = fmaf(a.beta1, m, a.one_minus_beta1 * gh);
    const float sgn = c > 0.0f ? 1.0f : (c < 0.0f ? -1.0f : c);  // 0 stays 0, NaN stays NaN
    p = fmaf(-a.step_size, sgn, p * a.decay);                    // step_size = lr, decay = 1 - lr wd
    m = fmaf(a.beta2, m, a.one_minus_beta2 * gh);
  } else if (kOpt == kOptSgdM) {
    const float d = fmaf(a.decay, p, gh);  // here decay holds wd itself, beta1 the momentum, step_size lr
    m = fmaf(a.beta1, m, d);
    p = fmaf(-a.step_size, m, p);
  } else {
    m = fmaf(a.beta1, m, a.one_minus_beta1 * gh);
    v = fmaf(a.beta2, v, a.one_minus_beta2 * (gh * gh));
    if (fast) {
      p = fmaf(-a.step_size, quotient_approx(m, v * a.inv_bc2, a.eps), p * a.decay);
    } else {
      const float denom = __fsqrt_rn(v * a.inv_bc2) + a.eps;  // sqrt(v_hat) + eps
      p = fmaf(-a.step_size, __fdiv_rn(m, denom), p * a.decay);
    }
  }
}

template <int kOpt>
__device__ __forceinline__ void adamw_vec4(const float g0, const float g1, const float g2, const float g3,
                                           float h, float4& p, float4& m, float4& v, const AdamScalars& a,
                                           bool fast = false) {
  adamw_elem<kOpt>(g0, h, p.x, m.x, v.x, a, fast);
  adamw_elem<kOpt>(g1, h, p.y, m.y, v.y, a, fast);
  adamw_elem<kOpt>(g2, h, p.z, m.z, v.z, a, fast);
  adamw_elem<kOpt>(g3, h, p.w, m.w, v.w, a, fast);
}

// Optimizer state (m, v) is stored as fp32 or as bfloat16 (kSB); arithmetic is fp32 either way.  A stored bfloat16
// is read exactly; the new moments are rounded to the nearest bfloat16 (ties to even) only where they are stored,
// after theta has been updated from the unrounded values.  Which neighbour is stored is decided by the fp32 value
// adamw_elem computes, in exactly its operation order (the header states it): with bfloat16 g and m and
// beta1 = 0.9 about one new m in twenty is an exact decimal tie in real arithmetic, so the order is part of the
// contract and must not be rearranged.
template <bool kSB>
__device__ __forceinline__ void load_state8(const void* __restrict__ base, int i, float4& a, float4& b) {
  if (kSB) {
    const uint4 q = __ldcs(static_cast<const uint4*>(base) + i);
    a = make_float4(bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y));
    b = make_float4(bf16_lo(q.z), bf16_hi(q.z), bf16_lo(q.w), bf16_hi(q.w));
  } else {
    a = ld_stream(static_cast<const float4*>(base) + 2 * i);
    b = ld_stream(static_cast<const float4*>(base) + 2 * i + 1);
  }
}
template <bool kSB>
__device__ __forceinline__ void store_state8(void* __restrict__ base, int i, const float4& a, const float4& b,
                                             bool stochastic = false, const uint4& wa = uint4(), const uint4& wb = uint4(),
                                             int which = 0) {
  if (kSB) {
    uint4 packed;
    if (stochastic) {
      const uint2 lo = pack4_stochastic(a, wa, which), hi = pack4_stochastic(b, wb, which);
      packed = make_uint4(lo.x, lo.y, hi.x, hi.y);
    } else {
      packed = make_uint4(pack_bf16_cvt(a.x, a.y), pack_bf16_cvt(a.z, a.w), pack_bf16_cvt(b.x, b.y), pack_bf16_cvt(b.z, b.w));
    }
    st_stream(static_cast<uint4*>(base) + i, packed);
  } else {
    st_stream(static_cast<float4*>(base) + 2 * i, a);
    st_stream(static_cast<float4*>(base) + 2 * i + 1, b);
  }
}
template <bool kSB>
__device__ __forceinline__ float load_state1(const void* __restrict__ base, int64_t j) {
  return kSB ? __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(base)[j]) << 16)
             : static_cast<const float*>(base)[j];
}
// one element at arena index `at`, rounded stochastically (which = 0: m, 1: v)
__device__ __forceinline__ void store_state1_stochastic(void* __restrict__ base, int64_t j, float x, int64_t at,
                                                        const StateRounding& sr, int which) {
  const uint4 w = rounding_words(at >> 2, sr);
  const uint32_t word = (at & 3) == 0 ? w.x : (at & 3) == 1 ? w.y : (at & 3) == 2 ? w.z : w.w;
  static_cast<uint16_t*>(base)[j] = static_cast<uint16_t>(pack_bf16_stochastic(x, 0.0f, (word >> (which ? 16 : 0)) & 0xffffu));
}
template <bool kSB>
__device__ __forceinline__ void store_state1(void* __restrict__ base, int64_t j, float x) {
  if (kSB) static_cast<uint16_t*>(base)[j] = static_cast<uint16_t>(pack_bf16_cvt(x, 0.0f));
  else static_cast<float*>(base)[j] = x;
}

// Eight consecutive elements of one chunk: 7 (bf16 gradients) or 8 (fp32) 16-byte loads, 6 stores
// (AdamW with fp32 state; Lion has no v stream; bfloat16 state halves the m and v accesses).
// mbase / vbase point at the chunk's first element of the m and v arenas.
template <bool kBF16, int kOpt, bool kSB>
__device__ __forceinline__ void adamw_group8(int i, const char* __restrict__ gbase, float4* __restrict__ p4,
                                             void* __restrict__ mbase, void* __restrict__ vbase, float h,
                                             const AdamScalars& a, uint4* __restrict__ lowp8 = nullptr,
                                             const StateRounding* sr = nullptr, int64_t q0 = 0) {
  float g[8];
  if (kBF16) {
    // the norm kernel left these lines marked evict_last; this last read of them hands them back
    const uint4 q = ld_nc_l2_hint(reinterpret_cast<const uint4*>(gbase) + i, l2_policy_evict_first());
    g[0] = bf16_lo(q.x); g[1] = bf16_hi(q.x); g[2] = bf16_lo(q.y); g[3] = bf16_hi(q.y);
    g[4] = bf16_lo(q.z); g[5] = bf16_hi(q.z); g[6] = bf16_lo(q.w); g[7] = bf16_hi(q.w);
  } else {
    const uint64_t done = l2_policy_evict_first();
    const uint4 qa = ld_nc_l2_hint(reinterpret_cast<const uint4*>(gbase) + 2 * i, done);
    const uint4 qb = ld_nc_l2_hint(reinterpret_cast<const uint4*>(gbase) + 2 * i + 1, done);
    const float4 ga = make_float4(__uint_as_float(qa.x), __uint_as_float(qa.y), __uint_as_float(qa.z), __uint_as_float(qa.w));
    const float4 gb = make_float4(__uint_as_float(qb.x), __uint_as_float(qb.y), __uint_as_float(qb.z), __uint_as_float(qb.w));
    g[0] = ga.x; g[1] = ga.y; g[2] = ga.z; g[3] = ga.w;
    g[4] = gb.x; g[5] = gb.y; g[6] = gb.z; g[7] = gb.w;
  }
  float4 pa = ld_stream(p4 + 2 * i), pb = ld_stream(p4 + 2 * i + 1);
  float4 ma, mb;
  load_state8<kSB>(mbase, i, ma, mb);
  float4 va = make_float4(0.f, 0.f, 0.f, 0.f), vb = va;
  if (kOpt == kOptAdamW) load_state8<kSB>(vbase, i, va, vb);
  const bool fast = kSB && use_quotient_approx(sr, a);
  adamw_vec4<kOpt>(g[0], g[1], g[2], g[3], h, pa, ma, va, a, fast);
  adamw_vec4<kOpt>(g[4], g[5], g[6], g[7], h, pb, mb, vb, a, fast);
  st_stream(p4 + 2 * i, pa); st_stream(p4 + 2 * i + 1, pb);
  if (kSB && sr && sr->stochastic) {  // q0: arena index / 4 of the chunk's first element; this group is elements 8i .. 8i+7
    const uint4 wa = rounding_words(q0 + 2 * i, *sr), wb = rounding_words(q0 + 2 * i + 1, *sr);
    store_state8<kSB>(mbase, i, ma, mb, true, wa, wb, 0);
    if (kOpt == kOptAdamW) store_state8<kSB>(vbase, i, va, vb, true, wa, wb, 1);
  } else {
    store_state8<kSB>(mbase, i, ma, mb);
    if (kOpt == kOptAdamW) store_state8<kSB>(vbase, i, va, vb);
  }
  if (lowp8)  // bf16 copy of the updated parameters (the model's working weights in mixed precision)
    st_stream(lowp8 + i, make_uint4(pack_bf16(pa.x, pa.y), pack_bf16(pa.z, pa.w), pack_bf16(pb.x, pb.y),
                                    pack_bf16(pb.z, pb.w)));
}

// A partial chunk (a small tensor, or the end of one).  Work is dealt in rows of 32 groups (256
// elements) and the rows of successive chunks go to the block's warps in one continuing round-robin:
// row_base counts the rows dealt so far.  Restarting at warp 0 for every chunk would give the low warps
// the extra rows every time and make them the critical path.
// One element at arena index e, with scalar accesses (the last count mod 8 elements of a chunk).
template <bool kBF16, int kOpt, bool kSB>
__device__ __forceinline__ void adamw_single(int64_t e, float h, float* __restrict__ params, const void* __restrict__ grads,
                                             void* __restrict__ m_arena, void* __restrict__ v_arena, const AdamScalars& a,
                                             uint16_t* __restrict__ lowp, const StateRounding* sr) {
  const float g = kBF16 ? __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(grads)[e]) << 16)
                        : static_cast<const float*>(grads)[e];
  float p = params[e], m = load_state1<kSB>(m_arena, e), v = 0.0f;
  if (kOpt == kOptAdamW) v = load_state1<kSB>(v_arena, e);
  adamw_elem<kOpt>(g, h, p, m, v, a, kSB && use_quotient_approx(sr, a));
  params[e] = p;
  if (kSB && sr && sr->stochastic) {
    store_state1_stochastic(m_arena, e, m, e, *sr, 0);
    if (kOpt == kOptAdamW) store_state1_stochastic(v_arena, e, v, e, *sr, 1);
  } else {
    store_state1<kSB>(m_arena, e, m);
    if (kOpt == kOptAdamW) store_state1<kSB>(v_arena, e, v);
  }
  if (lowp) lowp[e] = static_cast<uint16_t>(f32_to_bf16_bits(p));
}

// kWithTail = false leaves the chunk's last count mod 8 elements to the caller.
constexpr int kRowAlign = 256;  // elements
template <bool kBF16, int kBlockThreads, int kOpt, bool kSB, bool kWithTail = true>
__device__ __forceinline__ void adamw_partial_chunk(const Chunk& ck, float h, int& row_base, float* __restrict__ params,
                                                    const void* __restrict__ grads, void* __restrict__ m_arena,
                                                    void* __restrict__ v_arena, const AdamScalars& a,
                                                    uint16_t* __restrict__ lowp = nullptr,
                                                    const StateRounding* sr = nullptr) {
  constexpr int kWarps = kBlockThreads / 32;
  constexpr int kStateBytes = kSB ? 2 : 4;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Rows of 256 elements are laid from the last kRowAlign-element boundary at or before the chunk's start, so that a
  // warp's accesses fall on whole lines whatever the tensor's offset; the groups before the start are skipped.
  // A warp that gets no row of this chunk (most warps, for a short chunk) leaves after these few integer operations.
  const int pad = static_cast<int>(ck.start4 & (kRowAlign / 4 - 1)) << 2;  // a multiple of 8, like the start
  const int first8 = pad >> 3, n8 = ck.count >> 3;
  const int rows = (first8 + n8 + 31) >> 5;
  const int r0 = (warp - row_base) & (kWarps - 1);
  row_base = (row_base + rows) & (kWarps - 1);
  const bool has_tail = kWithTail && warp == row_base && (ck.count & 7) != 0;  // the next warp in turn takes the ragged tail
  if (r0 >= rows && !has_tail) return;
  const int64_t start = chunk_start(ck);
  const int64_t origin = start - pad;
  float4* __restrict__ p4 = reinterpret_cast<float4*>(params + origin);
  char* __restrict__ mbase = static_cast<char*>(m_arena) + origin * kStateBytes;
  char* __restrict__ vbase = kOpt == kOptAdamW ? static_cast<char*>(v_arena) + origin * kStateBytes : nullptr;
  const char* __restrict__ gbase = static_cast<const char*>(grads) + origin * (kBF16 ? 2 : 4);
#pragma unroll 2
  for (int r = r0; r < rows; r += kWarps) {
    const int i = (r << 5) + lane;
    if (i >= first8 && i < first8 + n8)
      adamw_group8<kBF16, kOpt, kSB>(i, gbase, p4, mbase, vbase, h, a, lowp ? reinterpret_cast<uint4*>(lowp + origin) : nullptr,
                                     sr, origin >> 2);
  }
  if (!has_tail) return;
  const int t = (n8 << 3) + lane;  // ragged tail: fewer than 8 elements
  if (t < ck.count) adamw_single<kBF16, kOpt, kSB>(start + t, h, params, grads, m_arena, v_arena, a, lowp, sr);
}

// Register-streaming update kernel: every thread loads eight elements of each stream into registers.
template <bool kBF16, int kOpt, bool kSB>
__global__ void __launch_bounds__(kThreads)
adagc_update_kernel(float* __restrict__ params, const void* __restrict__ grads, void* __restrict__ m_arena,
                    void* __restrict__ v_arena, const Chunk* __restrict__ chunks,
                    const int32_t* __restrict__ block_begin, const float* __restrict__ h_arr, AdamScalars a,
                    uint16_t* __restrict__ lowp, const AdamScalars* __restrict__ d_a, Guard guard, StateRounding sr) {
  constexpr int kStateBytes = kSB ? 2 : 4;
  const int tid = threadIdx.x;
  int c = block_begin[blockIdx.x];
  const int n_chunks = block_begin[blockIdx.x + 1];  // end of this block's entries
  ADAGC_CHECK_ENTRIES(chunks, c, n_chunks, guard);
  if (c >= n_chunks) return;
  Chunk ck = chunks[c];
  griddep_wait();     // the clip factors (and, in a capturable step, the coefficients) come from the preceding kernels
  if (d_a) a = *d_a;  // capturable step: coefficients from device memory
  float h = h_arr[ck.tensor];
  int row_base = 0;
  while (true) {
    // fetch the next chunk's table entry and clip factor now: with only two blocks resident per SM
    // nothing else would hide these two dependent loads between chunks
    const int c_next = c + 1;
    Chunk ck_next = ck;
    float h_next = h;
    if (c_next < n_chunks) {
      ck_next = chunks[c_next];
      h_next = h_arr[ck_next.tensor];
    }
    if (ck.count == kChunkElems) {  // full chunk: fixed trip count
      const int64_t start = chunk_start(ck);
      float4* __restrict__ p4 = reinterpret_cast<float4*>(params + start);
      char* __restrict__ mbase = static_cast<char*>(m_arena) + start * kStateBytes;
      char* __restrict__ vbase = kOpt == kOptAdamW ? static_cast<char*>(v_arena) + start * kStateBytes : nullptr;
      const char* __restrict__ gbase = static_cast<const char*>(grads) + start * (kBF16 ? 2 : 4);
#pragma unroll 2
      for (int k = 0; k < kChunkElems / 8 / kThreads; ++k)
        adamw_group8<kBF16, kOpt, kSB>(k * kThreads + tid, gbase, p4, mbase, vbase, h, a,
                                       lowp ? reinterpret_cast<uint4*>(lowp + start) : nullptr, &sr, start >> 2);
    } else {
      adamw_partial_chunk<kBF16, kThreads, kOpt, kSB>(ck, h, row_base, params, grads, m_arena, v_arena, a, lowp, &sr);
    }
    if (c_next >= n_chunks) break;
    c = c_next;
    ck = ck_next;
    h = h_next;
  }
}

// ------------------------------------------------------------------------------------------------
// Bulk-async (TMA) update kernel.  Full chunks are cut into tiles of kTile elements; an elected thread
// moves each tile's streams global -> shared with cp.async.bulk (completion on an mbarrier), all
// threads update the tile in shared memory, and the written streams go back with bulk stores.
// A ring of kStages stages: while tile j is computed, tiles j+1 .. j+kStages-1 are in flight and tile j-1
// drains.  fp32 state: tiles of 4096 elements, two stages (one 57 KB tile in flight per SM, the amount
// this access mix wants on B200).  bfloat16 state moves 10 instead of 14 bytes per element, and there the
// per-tile costs (barrier wait, block barrier, issue) weigh more: measured on the 7B-shaped layout, tiles of
// 2048 / 4096 / 8192 elements in two stages gave 5060 / 5650 / 6050 GB/s, more stages never helped (4096 x 3:
// 5700, 4096 x 4: 5670), and rounding with the conversion instruction instead of integer arithmetic took
// 8192 x 2 to 6650 GB/s.
// Partial chunks (a tensor's last, shorter chunk) come after the block's whole tiles.  With fp32 state they take the
// register path, which on its own reaches the whole tiles' rate down to chunks of about 2000 elements.  With
// bfloat16 state the register path is the slower one (5300 - 5500 GB/s), so there the partial chunks of at least half a
// tile go through the same ring, cut into tiles of their own length (measured on layouts of equal tensors of 12288 /
// 8192 / 6144 / 4096 elements: 6300 / 5950 / 6100 / 5460 GB/s against 5500 / 5380 / 5340 / 5290), and only shorter
// ones, and every chunk's last count mod 8 elements, are left to the register path.
// Every wait is bounded: after ~2 s without completion the block records ADAGC_E_TIMEOUT in the
// status word and leaves its remaining tiles untouched.
// ------------------------------------------------------------------------------------------------
constexpr int kTmaThreads = 512;
template <bool kSB>
struct TmaRing {  // fp32 state: 14 (16) bytes per element
  static constexpr int kTile = 4096, kStages = 2;
};
template <>
struct TmaRing<true> {  // bfloat16 state: 10 (12) bytes per element
  static constexpr int kTile = 8192, kStages = 2;
};
constexpr int kMaxDynamicSmem = 227 * 1024;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false if the phase did not complete within limit_ns (default ~2 s).
constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 63u) == 0 && global_timer_ns() - t0 > limit_ns) return false;
  }
}

// Test aid: waits on a barrier that nothing signals, with the same bounded wait as the update kernel.
__global__ void adagc_debug_wait_kernel(uint64_t limit_ns, int* __restrict__ status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool arrived = mbar_wait_bounded(&bar, 0, limit_ns);
  if (!__syncthreads_and(arrived ? 1 : 0) && threadIdx.x == 0) atomicOr(status, ADAGC_E_TIMEOUT);
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void bulk_store_hint(void* gdst, const void* smem_src, uint32_t bytes, uint64_t policy) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(gdst),
               "r"(smem_u32(smem_src)), "r"(bytes), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_smem_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_done() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_generic_to_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// bytes per element that the loads of one tile bring into a stage: theta, m (and v), g
__host__ __device__ constexpr int tma_elem_bytes(bool bf16, int opt, bool state_bf16) {
  return 4 + (opt == kOptAdamW ? 2 : 1) * (state_bf16 ? 2 : 4) + (bf16 ? 2 : 4);
}
template <bool kSB>
constexpr int tma_smem_bytes(bool bf16, int opt, bool emit_lowp = false) {
  return TmaRing<kSB>::kStages * TmaRing<kSB>::kTile * (tma_elem_bytes(bf16, opt, kSB) + (emit_lowp ? 2 : 0));
}

// One 4-element group of a tile's m or v region in shared memory, in the state dtype.
template <bool kSB>
__device__ __forceinline__ float4 smem_state4(const unsigned char* region, int q) {
  if (kSB) {
    const uint2 w = reinterpret_cast<const uint2*>(region)[q];
    return make_float4(bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y));
  }
  return reinterpret_cast<const float4*>(region)[q];
}
template <bool kSB>
__device__ __forceinline__ void smem_state4_store(unsigned char* region, int q, const float4& x) {
  if (kSB) reinterpret_cast<uint2*>(region)[q] = make_uint2(pack_bf16_cvt(x.x, x.y), pack_bf16_cvt(x.z, x.w));
  else reinterpret_cast<float4*>(region)[q] = x;
}

template <bool kBF16, int kOpt, bool kSB>
__global__ void __launch_bounds__(kTmaThreads, 1)
adagc_update_tma_kernel(float* __restrict__ params, const void* __restrict__ grads, void* __restrict__ m_arena,
                        void* __restrict__ v_arena, const Chunk* __restrict__ chunks,
                        const int32_t* __restrict__ block_begin, const int32_t* __restrict__ block_mid,
                        const float* __restrict__ h_arr, AdamScalars a, int* __restrict__ status,
                        uint16_t* __restrict__ lowp, const AdamScalars* __restrict__ d_a, Guard guard, StateRounding sr) {
  extern __shared__ __align__(128) unsigned char tile_smem[];
  constexpr int kTile = TmaRing<kSB>::kTile, kStages = TmaRing<kSB>::kStages;
  constexpr int kTilesPerChunk = kChunkElems / kTile;
  constexpr int kAhead = kStages - 1;  // tiles in flight beyond the one being computed
  static_assert(kChunkElems % kTile == 0 && kTile % (4 * kTmaThreads) == 0, "tiles divide chunks, threads divide tiles");
  static_assert(kAhead >= 1 && kAhead <= kTilesPerChunk, "the tile being fetched lies in this chunk or the next");
  constexpr int kGBytes = kBF16 ? 2 : 4;
  constexpr int kSBytes = kSB ? 2 : 4;                              // m, v element size
  constexpr int kMOff = kTile * 4;                                   // region offsets inside a stage: theta, m, v, g
  constexpr int kVOff = kMOff + kTile * kSBytes;
  constexpr int kGOff = kOpt == kOptAdamW ? kVOff + kTile * kSBytes : kVOff;
  constexpr uint32_t kStageBytes = kGOff + kTile * kGBytes;          // what the loads of one tile bring in
  static_assert(kStageBytes == static_cast<uint32_t>(kTile) * tma_elem_bytes(kBF16, kOpt, kSB), "stage layout");
  static_assert(kStages * (kStageBytes + kTile * 2) <= kMaxDynamicSmem, "the ring fits in shared memory");
  // with a bf16 copy of the parameters to emit, each stage has one more region that only the stores read
  const uint32_t stage_stride = kStageBytes + (lowp ? kTile * 2 : 0);
  __shared__ __align__(8) uint64_t full_bar[kStages];
  const int tid = threadIdx.x;
  const int begin = block_begin[blockIdx.x], mid = block_mid[blockIdx.x], end = block_begin[blockIdx.x + 1];
  ADAGC_CHECK_ENTRIES(chunks, begin, end, guard);
#ifdef ADAGC_BOUNDS_CHECK
  {  // the entries before `mid` are moved as whole tiles: they must be full chunks
    int full = mid >= begin && mid <= end;
    for (int c = begin + threadIdx.x; full && c < mid; c += blockDim.x) full = chunks[c].count == kChunkElems;
    full = __syncthreads_and(full);
    if (!full) {
      if (threadIdx.x == 0) atomicOr(guard.status, ADAGC_E_BOUNDS);
      return;
    }
  }
#endif
  const int n_tiles = (mid - begin) * kTilesPerChunk;

  __shared__ int abort_flag;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&full_bar[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    abort_flag = 0;
  }
  // The larger partial chunks go through the ring too (after the full chunks), in tiles of their own length; the
  // block lists them here, in table order, one candidate entry per thread.  Entries past the first kRingList
  // partial chunks, chunks shorter than kRingMin and the last (count mod 8) elements of a listed chunk take the
  // register path at the end.  (The list is kept small: with fp32 gradients, bfloat16 state and a bfloat16 copy
  // of the parameters the ring itself takes 224 of the 227 KB a block may have.)
  constexpr bool kRingPartials = kSB;  // fp32 state: none, the register path is the faster one there (kernel header)
  constexpr int kRingMin = kTile / 2, kRingList = 256;
  static_assert(kRingList <= kTmaThreads && kChunkElems <= 65536, "one candidate per thread; lengths fit 16 bits");
  static_assert(kStages * (kStageBytes + kTile * 2) + kRingList * 10 + 256 <= kMaxDynamicSmem, "ring and list fit");
  __shared__ uint32_t ring_start4[kRingList];
  __shared__ uint32_t ring_tensor_or_h[kRingList];  // the owning tensor until the clip factors are read, then the factor
  __shared__ uint16_t ring_n8[kRingList];
  __shared__ int ring_warp_count[kTmaThreads / 32];
  const int listed_end = min(end, mid + kRingList);  // entries [mid, listed_end) are the candidates
  int n_listed = 0;
  if (kRingPartials) {
    const int c = mid + tid;
    Chunk cand{0u, 0, 0, 0};
    if (c < listed_end) cand = chunks[c];
    const bool take = (cand.count & ~7) >= kRingMin;
    const unsigned takers = __ballot_sync(0xffffffffu, take);
    if ((tid & 31) == 0) ring_warp_count[tid >> 5] = __popc(takers);
    __syncthreads();
    int before = 0;
    for (int w = 0; w < kTmaThreads / 32; ++w) {
      const int n_w = ring_warp_count[w];
      if (w < (tid >> 5)) before += n_w;
      n_listed += n_w;
    }
    if (take) {
      const int pos = before + __popc(takers & ((1u << (tid & 31)) - 1u));
      ring_start4[pos] = cand.start4;
      ring_n8[pos] = static_cast<uint16_t>(cand.count & ~7);
      ring_tensor_or_h[pos] = static_cast<uint32_t>(cand.tensor);
    }
  }
  __syncthreads();

  const uint64_t stream_policy = l2_policy_evict_first();  // every byte this kernel moves is used once
  // thread 0 only: start the loads of n elements from arena element e into stage s (n a multiple of 8: every copy
  // is then a multiple of 16 bytes and starts on a 16-byte boundary)
  auto issue_span = [&](int64_t e, int n, int s) {
    unsigned char* b = tile_smem + static_cast<size_t>(s) * stage_stride;
    mbar_arrive_expect_tx(&full_bar[s], static_cast<uint32_t>(n) * tma_elem_bytes(kBF16, kOpt, kSB));
    bulk_load_hint(b, params + e, n * 4, &full_bar[s], stream_policy);
    bulk_load_hint(b + kMOff, static_cast<const char*>(m_arena) + e * kSBytes, n * kSBytes, &full_bar[s], stream_policy);
    if (kOpt == kOptAdamW)
      bulk_load_hint(b + kVOff, static_cast<const char*>(v_arena) + e * kSBytes, n * kSBytes, &full_bar[s], stream_policy);
    bulk_load_hint(b + kGOff, static_cast<const char*>(grads) + e * kGBytes, n * kGBytes, &full_bar[s], stream_policy);
  };
  // tile `sub` of the full chunk that starts at element e0
  auto issue_tile = [&](int64_t e0, int sub, int s) { issue_span(e0 + static_cast<int64_t>(sub) * kTile, kTile, s); };
  // thread 0 only: write the updated streams of a stage back and commit them as one group
  auto store_span = [&](int64_t e, int n, unsigned char* b) {
    bulk_store_hint(params + e, b, n * 4, stream_policy);
    bulk_store_hint(static_cast<char*>(m_arena) + e * kSBytes, b + kMOff, n * kSBytes, stream_policy);
    if (kOpt == kOptAdamW) bulk_store_hint(static_cast<char*>(v_arena) + e * kSBytes, b + kVOff, n * kSBytes, stream_policy);
    if (lowp) bulk_store_hint(lowp + e, b + kStageBytes, n * 2, stream_policy);
    bulk_commit();
  };
  // all threads: update the groups of four elements of one stage in place.  One copy of the loop per rounding mode,
  // so that rounding to nearest carries none of the other mode's code, and per tile kind, so that a whole tile's
  // trip count is a constant.  group0 is the arena index, in groups of four, of the stage's first element.
  auto update_tile = [&](auto stochastic_tag, auto whole_tag, unsigned char* b, int n_groups, float h, int64_t group0) {
    constexpr bool kStochastic = decltype(stochastic_tag)::value;
    constexpr bool kWhole = decltype(whole_tag)::value;
    const bool fast = kStochastic && use_quotient_approx(&sr, a);
    float4* p4 = reinterpret_cast<float4*>(b);
    const int n_q = kWhole ? kTile / 4 : n_groups;
#pragma unroll
    for (int q = tid; q < n_q; q += kTmaThreads) {
      float g0, g1, g2, g3;
      if (kBF16) {
        const uint2 w = reinterpret_cast<const uint2*>(b + kGOff)[q];
        g0 = bf16_lo(w.x); g1 = bf16_hi(w.x); g2 = bf16_lo(w.y); g3 = bf16_hi(w.y);
      } else {
        const float4 w = reinterpret_cast<const float4*>(b + kGOff)[q];
        g0 = w.x; g1 = w.y; g2 = w.z; g3 = w.w;
      }
      float4 p = p4[q], m = smem_state4<kSB>(b + kMOff, q), v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (kOpt == kOptAdamW) v = smem_state4<kSB>(b + kVOff, q);
      adamw_vec4<kOpt>(g0, g1, g2, g3, h, p, m, v, a, fast);
      p4[q] = p;
      if (kStochastic) {  // elements 4q .. 4q+3 of this stage: one group of the arenas
        const uint4 w = rounding_words(group0 + q, sr);
        reinterpret_cast<uint2*>(b + kMOff)[q] = pack4_stochastic(m, w, 0);
        if (kOpt == kOptAdamW) reinterpret_cast<uint2*>(b + kVOff)[q] = pack4_stochastic(v, w, 1);
      } else {
        smem_state4_store<kSB>(b + kMOff, q, m);
        if (kOpt == kOptAdamW) smem_state4_store<kSB>(b + kVOff, q, v);
      }
      if (lowp) reinterpret_cast<uint2*>(b + kStageBytes)[q] = make_uint2(pack_bf16(p.x, p.y), pack_bf16(p.z, p.w));
    }
  };

  bool healthy = true;
  int j_fail = 0;
  // Everything up to here, the table entries and the first loads below touch nothing that the preceding kernels of the
  // step write (they write the clip factors, gamma and statistics only), so with a programmatic dependent launch this
  // much overlaps the tail of the norm phase.
  if (n_tiles == 0) {
    griddep_wait();
    if (d_a) a = *d_a;
  } else {
    // table entries are kept two chunks ahead in registers, so that neither the elected thread's issue path
    // nor the consumers ever wait for a table load
    Chunk ck = chunks[begin];
    Chunk ck_next = ck, ck_next2 = ck;
    if (begin + 1 < mid) ck_next = chunks[begin + 1];
    if (begin + 2 < mid) ck_next2 = chunks[begin + 2];
    if (tid == 0)
      for (int k = 0; k < kAhead && k < n_tiles; ++k) issue_tile(chunk_start(ck), k, k);  // kAhead <= tiles per chunk
    griddep_wait();
    if (d_a) a = *d_a;  // capturable step: coefficients from device memory
    float h = h_arr[ck.tensor];
    float h_next = h_arr[ck_next.tensor], h_next2 = h_arr[ck_next2.tensor];
    int s = 0;           // stage of tile j
    uint32_t phase = 0;  // parity of the barrier phase tile j completes: flips each time the ring wraps
    for (int j = 0; j < n_tiles; ++j) {
      const int sub = j % kTilesPerChunk;
      const bool last_of_chunk = sub == kTilesPerChunk - 1;
      if (tid == 0 && j + kAhead < n_tiles) {
        bulk_wait_smem_read();  // the stores of tile j-1 have finished reading the stage that is refilled now
        const int sub_f = sub + kAhead;  // tile j + kAhead: in this chunk or in the next
        const int s_f = s == 0 ? kStages - 1 : s - 1;
        if (sub_f >= kTilesPerChunk) issue_tile(chunk_start(ck_next), sub_f - kTilesPerChunk, s_f);
        else issue_tile(chunk_start(ck), sub_f, s_f);
      }
      unsigned char* b = tile_smem + static_cast<size_t>(s) * stage_stride;
      if (mbar_wait_bounded(&full_bar[s], phase)) {
        const int64_t group0 = (chunk_start(ck) >> 2) + sub * (kTile / 4);
        if (kSB && sr.stochastic) update_tile(std::true_type{}, std::true_type{}, b, 0, h, group0);
        else update_tile(std::false_type{}, std::true_type{}, b, 0, h, group0);
        fence_generic_to_async_smem();  // the updated tile must be visible to the bulk-copy engine
      } else {
        abort_flag = 1;  // this thread gave up; the barrier below tells every thread
      }
      __syncthreads();
      if (abort_flag) {  // uniform: written before the barrier, read after it
        healthy = false;
        j_fail = j;
        break;
      }
      if (tid == 0) store_span(chunk_start(ck) + static_cast<int64_t>(sub) * kTile, kTile, b);
      if (last_of_chunk) {
        ck = ck_next;
        h = h_next;
        ck_next = ck_next2;
        h_next = h_next2;
        const int c3 = begin + j / kTilesPerChunk + 3;
        if (c3 < mid) {
          ck_next2 = chunks[c3];
          h_next2 = h_arr[ck_next2.tensor];
        }
      }
      if (++s == kStages) {
        s = 0;
        phase ^= 1u;
      }
    }
    if (tid == 0) {
      bulk_wait_done();
      if (!healthy) {
        atomicOr(status, ADAGC_E_TIMEOUT);
        // loads may still be in flight into this block's shared memory: give each of them one more bounded
        // chance to land before the block (and its shared memory) goes away
        for (int k = 0; k <= kAhead && j_fail + k < n_tiles; ++k) {
          const int jj = j_fail + k;
          (void)mbar_wait_bounded(&full_bar[jj % kStages], (jj / kStages) & 1);
        }
      }
    }
    __syncthreads();
  }
  if (!healthy) return;

  if (mid >= end) return;

  // ---- listed partial chunks: the same ring, continuing its stage and phase count after the n_tiles whole tiles.
  // A chunk of n8 elements is cut into ceil(n8 / kTile) tiles of (nearly) equal length, each a multiple of 8.
  if (kRingPartials && n_listed > 0) {
    if (tid < n_listed) ring_tensor_or_h[tid] = __float_as_uint(h_arr[ring_tensor_or_h[tid]]);
    __syncthreads();
    struct Cursor {
      int i, k, n_t, len, n8;  // listed chunk, tile within it, tiles of the chunk, tile length, elements of the chunk
      int64_t e0;              // the chunk's first arena element
    };
    auto open_chunk = [&](Cursor& cu) {
      cu.k = 0;
      if (cu.i < n_listed) {
        cu.n8 = ring_n8[cu.i];
        cu.n_t = (cu.n8 + kTile - 1) / kTile;
        cu.len = ((cu.n8 + cu.n_t - 1) / cu.n_t + 7) & ~7;
        cu.e0 = static_cast<int64_t>(ring_start4[cu.i]) * 4;
      }
    };
    auto next_tile = [&](Cursor& cu) {
      if (++cu.k == cu.n_t) {
        ++cu.i;
        open_chunk(cu);
      }
    };
    Cursor fetch{0, 0, 0, 0, 0, 0}, work{0, 0, 0, 0, 0, 0};  // thread 0's issue position; every thread's compute position
    open_chunk(fetch);
    open_chunk(work);
    int issued = 0, done = 0;  // tiles of this phase (issued: thread 0 only)
    auto issue_next = [&]() {
      const int off = fetch.k * fetch.len;
      issue_span(fetch.e0 + off, min(fetch.len, fetch.n8 - off), (n_tiles + issued) % kStages);
      ++issued;
      next_tile(fetch);
    };
    if (tid == 0)
      for (int k = 0; k < kAhead && fetch.i < n_listed; ++k) issue_next();
    while (work.i < n_listed) {
      const int ring_pos = n_tiles + done;
      const int s = ring_pos % kStages;
      if (tid == 0 && fetch.i < n_listed) {
        bulk_wait_smem_read();  // the stores of the previous tile have finished reading the stage that is refilled now
        issue_next();
      }
      unsigned char* b = tile_smem + static_cast<size_t>(s) * stage_stride;
      const int off = work.k * work.len;
      const int n = min(work.len, work.n8 - off);
      if (mbar_wait_bounded(&full_bar[s], (ring_pos / kStages) & 1)) {
        const float h = __uint_as_float(ring_tensor_or_h[work.i]);
        const int64_t group0 = (work.e0 + off) >> 2;
        if (kSB && sr.stochastic) update_tile(std::true_type{}, std::false_type{}, b, n >> 2, h, group0);
        else update_tile(std::false_type{}, std::false_type{}, b, n >> 2, h, group0);
        fence_generic_to_async_smem();
      } else {
        abort_flag = 1;
      }
      __syncthreads();
      if (abort_flag) {
        healthy = false;
        break;
      }
      if (tid == 0) store_span(work.e0 + off, n, b);
      ++done;
      next_tile(work);
    }
    if (tid == 0) {
      bulk_wait_done();
      if (!healthy) {
        atomicOr(status, ADAGC_E_TIMEOUT);
        for (int jj = n_tiles + done; jj < n_tiles + issued; ++jj)  // loads still in flight into this block's shared memory
          (void)mbar_wait_bounded(&full_bar[jj % kStages], (jj / kStages) & 1);
      }
    }
    __syncthreads();
    if (!healthy) return;
  }

  // ---- what is left, on the register path: short chunks, entries past the listed range, and the last (count mod 8)
  // elements of the listed chunks.  Table entry and clip factor are fetched one chunk ahead, so that a warp moving
  // from one small chunk to the next never waits on two dependent loads with nothing else in flight.
  int row_base = 0;
  Chunk ck = chunks[mid];
  float h = h_arr[ck.tensor];
  for (int c = mid; c < end; ++c) {
    Chunk ck_next = ck;
    float h_next = h;
    if (c + 1 < end) {
      ck_next = chunks[c + 1];
      h_next = h_arr[ck_next.tensor];
    }
    const bool listed = kRingPartials && c < listed_end && (ck.count & ~7) >= kRingMin;  // done but for its ragged tail
    if (!listed)
      adamw_partial_chunk<kBF16, kTmaThreads, kOpt, kSB, false>(ck, h, row_base, params, grads, m_arena, v_arena, a, lowp, &sr);
    ck = ck_next;
    h = h_next;
  }
  // The ragged tails (count mod 8 elements) of all partial chunks, four chunks per warp at a time: lane l takes
  // element l mod 8 of the tail of entry c0 + l / 8.  One at a time, each tail would cost its warp a memory latency.
  const int warp = tid >> 5, lane = tid & 31;
  for (int c0 = mid + warp * 4; c0 < end; c0 += (kTmaThreads / 32) * 4) {
    const int c = c0 + (lane >> 3);
    if (c >= end) continue;
    const Chunk tc = chunks[c];
    if ((lane & 7) < (tc.count & 7))
      adamw_single<kBF16, kOpt, kSB>(chunk_start(tc) + (tc.count & ~7) + (lane & 7), h_arr[tc.tensor], params, grads, m_arena,
                                     v_arena, a, lowp, &sr);
  }
}

// Clip-only: hat(g) = h * g written in the gradient dtype.  In place, chunks with h == 1 are skipped.
template <bool kBF16>
__device__ __forceinline__ uint4 scale_vec(uint4 q, float h) {
  if (kBF16) {
    q.x = pack_bf16(h * bf16_lo(q.x), h * bf16_hi(q.x));
    q.y = pack_bf16(h * bf16_lo(q.y), h * bf16_hi(q.y));
    q.z = pack_bf16(h * bf16_lo(q.z), h * bf16_hi(q.z));
    q.w = pack_bf16(h * bf16_lo(q.w), h * bf16_hi(q.w));
  } else {
    q.x = __float_as_uint(h * __uint_as_float(q.x));
    q.y = __float_as_uint(h * __uint_as_float(q.y));
    q.z = __float_as_uint(h * __uint_as_float(q.z));
    q.w = __float_as_uint(h * __uint_as_float(q.w));
  }
  return q;
}

template <bool kBF16>
__global__ void __launch_bounds__(kThreads)
adagc_scale_kernel(const void* gin, void* gout /* may alias gin: in-place clipping */, const Chunk* __restrict__ chunks,
                   const int32_t* __restrict__ block_begin, const float* __restrict__ h_arr, int in_place, Guard guard) {
  constexpr int kEPV = kBF16 ? 8 : 4;
  constexpr int kWarps = kThreads / 32;
#ifndef ADAGC_SCALE_BATCH
#define ADAGC_SCALE_BATCH 1
#endif
  constexpr int kBatch = ADAGC_SCALE_BATCH;  // 16-byte loads in flight per thread
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int row_base = 0;  // rows (32 vectors) dealt so far: successive chunks continue one round-robin over the warps
  const uint64_t done = l2_policy_evict_first();
  const int c_end = block_begin[blockIdx.x + 1];
  ADAGC_CHECK_ENTRIES(chunks, block_begin[blockIdx.x], c_end, guard);
  for (int c = block_begin[blockIdx.x]; c < c_end; ++c) {
    const Chunk ck = chunks[c];
    const float h = h_arr[ck.tensor];
    if (in_place && h == 1.0f) continue;
    const int64_t boff = chunk_start(ck) * (kBF16 ? 2 : 4);
    const uint4* src = reinterpret_cast<const uint4*>(static_cast<const char*>(gin) + boff);
    uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(gout) + boff);
    const int nvec = ck.count / kEPV;
    const int rows = (nvec + 31) >> 5;
    for (int r0 = (warp - row_base) & (kWarps - 1); r0 < rows; r0 += kWarps * kBatch) {
      uint4 q[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = ((r0 + u * kWarps) << 5) + lane;
        if (i < nvec) q[u] = ld_l2_hint(src + i, done);  // last read of lines the norm kernel marked evict_last
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = ((r0 + u * kWarps) << 5) + lane;
        if (i < nvec) st_stream(dst + i, scale_vec<kBF16>(q[u], h));
      }
    }
    row_base = (row_base + rows) & (kWarps - 1);
    const int t = nvec * kEPV + lane;  // ragged tail (fewer than one vector): the next warp in turn
    if (warp == row_base && t < ck.count) {
      if (kBF16) {
        const uint16_t b = reinterpret_cast<const uint16_t*>(src)[t];
        const float x = h * __uint_as_float(static_cast<uint32_t>(b) << 16);
        reinterpret_cast<uint16_t*>(dst)[t] = static_cast<uint16_t>(f32_to_bf16_bits(x));
      } else {
        reinterpret_cast<float*>(dst)[t] = h * reinterpret_cast<const float*>(src)[t];
      }
    }
  }
}

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

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {  // byte offsets of the workspace sections
  size_t chunks_range, begin_range, chunks_wide, chunks_upd, begin_wide, begin_upd, mid_upd, g_chunks_wide, g_chunks_upd, g_begin_wide,
      g_begin_upd, g_mid_upd, g_order, tensors, partials, sumsq, norm, h, clip_count, scalars, dev_step, gamma_prev, slice_partials, flag,
      tickets, total;
};

Layout make_layout(int64_t n_chunks, int64_t T, bool fused_small = false) {
  Layout L;
  size_t o = 0;
  L.chunks_range = o; o = align_up(o + sizeof(Chunk) * n_chunks, 256);  // original order, cut into one range per block
  L.begin_range = o;  o = align_up(o + sizeof(int32_t) * (kMaxGrid + 1), 256);
  L.chunks_wide = o; o = align_up(o + sizeof(Chunk) * n_chunks, 256);  // order of the norm / scale grid
  L.chunks_upd = o;  o = align_up(o + sizeof(Chunk) * n_chunks, 256);  // order of the update grid
  L.begin_wide = o;  o = align_up(o + sizeof(int32_t) * (kMaxGrid + 1), 256);
  L.begin_upd = o;   o = align_up(o + sizeof(int32_t) * (kMaxGrid + 1), 256);
  L.mid_upd = o;     o = align_up(o + sizeof(int32_t) * (kMaxGrid + 1), 256);
  // the same tables once more, cut into groups of tensors for the pipelined host step
  L.g_chunks_wide = o; o = align_up(o + sizeof(Chunk) * n_chunks, 256);
  L.g_chunks_upd = o;  o = align_up(o + sizeof(Chunk) * n_chunks, 256);
  L.g_begin_wide = o;  o = align_up(o + sizeof(int32_t) * kMaxGroups * (kGroupMaxGrid + 1), 256);
  L.g_begin_upd = o;   o = align_up(o + sizeof(int32_t) * kMaxGroups * (kGroupMaxGrid + 1), 256);
  L.g_mid_upd = o;     o = align_up(o + sizeof(int32_t) * kMaxGroups * (kGroupMaxGrid + 1), 256);
  L.g_order = o;       o = align_up(o + sizeof(int32_t) * T, 256);
  L.tensors = o;    o = align_up(o + sizeof(TensorEntry) * T, 256);
  L.partials = o;   o = align_up(o + sizeof(double) * n_chunks, 256);
  L.sumsq = o;      o = align_up(o + sizeof(double) * T, 256);
  L.norm = o;       o = align_up(o + sizeof(float) * T, 256);
  L.h = o;          o = align_up(o + sizeof(float) * T, 256);
  L.clip_count = o; o = align_up(o + sizeof(uint64_t) * T, 256);
  L.scalars = o;    o = align_up(o + 256, 256);  // steps_done (u64) at +0, status (i32) at +8
  L.dev_step = o;   o = align_up(o + sizeof(DeviceStep), 256);
  L.gamma_prev = o; o = align_up(o + sizeof(float) * T, 256);  // one-kernel step: gamma as it was before the step
  L.slice_partials = o;  // one-kernel step: one partial per slice of a chunk
  if (fused_small) o = align_up(o + sizeof(double) * n_chunks * 4, 256);
  L.flag = o;       o = align_up(o + T, 256);
  L.tickets = o;    o = align_up(o + sizeof(uint32_t) * T, 256);  // per tensor: chunks of it summed so far in this launch
  L.total = o;
  return L;
}

int validate_desc(const adagc_desc* d, int64_t* n_chunks_out, int64_t* arena_elems_out) {
  if (!d || !d->tensors || d->n_tensors < 1 || d->n_tensors > (1 << 24)) return ADAGC_E_INVALID_ARG;
  if (d->param_dtype != ADAGC_F32) return ADAGC_E_DTYPE;
  if (d->state_dtype != ADAGC_F32 && d->state_dtype != ADAGC_BF16) return ADAGC_E_DTYPE;
  if (d->grad_dtype != ADAGC_F32 && d->grad_dtype != ADAGC_BF16) return ADAGC_E_DTYPE;
  if (!(d->lambda_abs > 0.0) || !std::isfinite(d->lambda_abs)) return ADAGC_E_INVALID_ARG;
  constexpr int kKnownFlags =
      ADAGC_UPDATE_PATH_MASK | ADAGC_EMA_KEEP_INITIAL | ADAGC_CLIP_GLOBAL_ADAPTIVE | ADAGC_ALLOW_EMPTY |
      ADAGC_FUSED_SMALL | ADAGC_SEPARATE_FINALIZE;
  if ((d->flags & ADAGC_FUSED_SMALL) && (d->flags & ADAGC_CLIP_GLOBAL_ADAPTIVE)) return ADAGC_E_INVALID_ARG;
  const bool allow_empty = (d->flags & ADAGC_ALLOW_EMPTY) != 0;
  if ((d->flags & ~kKnownFlags) != 0 || (d->flags & ADAGC_UPDATE_PATH_MASK) == 3) return ADAGC_E_INVALID_ARG;
  // every arena must start each tensor on a 16-byte boundary: 8 elements as soon as one arena holds 2-byte elements
  const int64_t align = (d->grad_dtype == ADAGC_BF16 || d->state_dtype == ADAGC_BF16) ? 8 : 4;
  int64_t n_chunks = 0, extent = 0;
  std::vector<std::pair<int64_t, int64_t>> spans;
  spans.reserve(d->n_tensors);
  for (int32_t i = 0; i < d->n_tensors; ++i) {
    const adagc_tensor& t = d->tensors[i];
    if (allow_empty && t.numel == 0) continue;  // this rank holds nothing of the tensor; its offset is ignored
    if (t.numel <= 0 || t.offset < 0 || t.ndim < 0 || t.ndim > 4) return ADAGC_E_INVALID_ARG;
    if (t.numel > (int64_t(1) << 34) || t.offset + t.numel > (int64_t(1) << 34)) return ADAGC_E_INVALID_ARG;
    if (t.ndim > 0) {
      int64_t prod = 1;
      for (int k = 0; k < t.ndim; ++k) {
        if (t.shape[k] <= 0) return ADAGC_E_INVALID_ARG;
        prod *= t.shape[k];
      }
      if (prod != t.numel) return ADAGC_E_INVALID_ARG;
    }
    if (t.offset % align != 0) return ADAGC_E_MISALIGNED;
    n_chunks += (t.numel + kChunkElems - 1) / kChunkElems;
    extent = std::max(extent, t.offset + t.numel);
    spans.emplace_back(t.offset, t.offset + t.numel);
  }
  if (n_chunks > int64_t(0x7fffffff)) return ADAGC_E_INVALID_ARG;
  std::sort(spans.begin(), spans.end());
  for (size_t k = 1; k < spans.size(); ++k)
    if (spans[k].first < spans[k - 1].second) return ADAGC_E_OVERLAP;
  if (n_chunks_out) *n_chunks_out = n_chunks;
  if (arena_elems_out) *arena_elems_out = extent;
  return ADAGC_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// List scheduling in table order: each chunk goes to the block with the least work so far (ties to the
// lowest block index, so equal chunks are dealt round-robin); a block keeps its chunks in arrival order.
// With block_mid, a block's full chunks come first: [block_begin[b], block_mid[b]) are full
// (kChunkElems elements), [block_mid[b], block_begin[b+1]) are partial.
void balance_chunks(const std::vector<Chunk>& chunks, int grid, std::vector<Chunk>* table,
                    std::vector<int32_t>* block_begin, std::vector<int32_t>* block_mid = nullptr) {
  const int fixed_cost = block_mid ? kChunkFixedCost : kChunkFixedCostWide;  // update tables carry block_mid
  using Load = std::pair<int64_t, int>;  // (work assigned, block)
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int b = 0; b < grid; ++b) heap.emplace(0, b);
  std::vector<int32_t> owner(chunks.size());
  std::vector<int32_t> count(grid, 0);
  for (size_t i = 0; i < chunks.size(); ++i) {
    const Load top = heap.top();
    heap.pop();
    owner[i] = top.second;
    count[top.second] += 1;
    heap.emplace(top.first + chunks[i].count + fixed_cost, top.second);
  }
  block_begin->assign(grid + 1, 0);
  for (int b = 0; b < grid; ++b) (*block_begin)[b + 1] = (*block_begin)[b] + count[b];
  std::vector<int32_t> pos(block_begin->begin(), block_begin->end() - 1);
  table->resize(chunks.size());
  for (size_t i = 0; i < chunks.size(); ++i) (*table)[pos[owner[i]]++] = chunks[i];
  if (block_mid) {
    block_mid->assign(grid + 1, 0);
    for (int b = 0; b < grid; ++b) {
      auto first = table->begin() + (*block_begin)[b], last = table->begin() + (*block_begin)[b + 1];
      auto mid = std::stable_partition(first, last, [](const Chunk& c) { return c.count == kChunkElems; });
      (*block_mid)[b] = static_cast<int32_t>(mid - table->begin());
    }
  }
}

// Every tensor of a validated descriptor cut into chunks of kChunkElems elements (the last one shorter), in tensor
// order; chunk k's partial sum has index k.
void cut_into_chunks(const adagc_desc* desc, int64_t n_chunks, std::vector<Chunk>* chunks, std::vector<TensorEntry>* tensors) {
  chunks->reserve(n_chunks);
  tensors->reserve(desc->n_tensors);
  for (int32_t i = 0; i < desc->n_tensors; ++i) {
    const adagc_tensor& t = desc->tensors[i];
    TensorEntry te;
    te.first_chunk = static_cast<int32_t>(chunks->size());
    for (int64_t o = 0; o < t.numel; o += kChunkElems) {
      Chunk c;
      c.start4 = static_cast<uint32_t>((t.offset + o) / 4);
      c.count = static_cast<int32_t>(std::min<int64_t>(kChunkElems, t.numel - o));
      c.tensor = i;
      c.partial = static_cast<int32_t>(chunks->size());
      chunks->push_back(c);
    }
    te.n_chunks = static_cast<int32_t>(chunks->size()) - te.first_chunk;
    tensors->push_back(te);
  }
}

// The chunks in their original order cut into `grid` consecutive ranges of about equal cost (elements plus the fixed
// cost per chunk): block b of adagc_norm_decide_kernel owns [out[b], out[b+1]).
std::vector<int32_t> contiguous_ranges(const std::vector<Chunk>& chunks, int grid) {
  int64_t total = 0;
  for (const Chunk& c : chunks) total += c.count + kChunkFixedCostWide;
  std::vector<int32_t> out(grid + 1, static_cast<int32_t>(chunks.size()));
  out[0] = 0;
  int64_t acc = 0;
  int b = 1;
  for (size_t i = 0; i < chunks.size() && b < grid; ++i) {
    acc += chunks[i].count + kChunkFixedCostWide;
    while (b < grid && acc * grid >= total * b) out[b++] = static_cast<int32_t>(i + 1);  // cut after chunk i
  }
  return out;
}

}  // namespace

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
