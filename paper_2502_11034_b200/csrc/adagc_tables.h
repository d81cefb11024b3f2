// Host side: descriptor validation, the chunk tables and their balancing over thread blocks, workspace layout.
// Part of the single translation unit adagc.cu (included there, in order; not compiled on its own).
#pragma once

namespace {

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
