// Constants, the chunk-table entry, the bounds-check guard of the debugging build and the small device helpers
// (shuffle-tree sum, bfloat16 unpacking, cache-hinted loads, programmatic-dependent-launch controls) shared by every kernel.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

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

}  // namespace
