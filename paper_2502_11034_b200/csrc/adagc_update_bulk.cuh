// Phase 3, bulk-async update kernel: cp.async.bulk + mbarrier ring through shared memory.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

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

}  // namespace
