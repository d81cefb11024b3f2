// Clip-only mode: the kernel that writes the clipped gradient.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

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

}  // namespace
