// Phase 3: the optimizer applied to the clipped gradient (last four lines of Algorithm 1; Lion; momentum SGD), the
// rounding of bfloat16-stored moments, the register path for partial chunks and the register-streaming update kernel.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

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

}  // namespace
