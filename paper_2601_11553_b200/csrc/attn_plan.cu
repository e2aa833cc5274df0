// Host-side scheduling of the attention kernel: which persistent CTA runs which (tile, unit, context range).
//
// A tile is up to 128 consecutive new rows of one prompt; it has `units_per_tile` independent units (KV
// head x pair of its query heads), each needing the tile's n_blocks context blocks.  Tiles differ a lot in
// length (a row at position p sees p + 1 slots), and a batch may have fewer units than the GPU has SMs,
// so units are not dealt whole: the sequence of all (unit, block) pairs is cut into one contiguous span per
// CTA, all spans costing the same.  A unit cut by a span boundary is "split": each part writes an
// unnormalised partial result and a merge kernel combines them.  When dealing the units whole
// (longest first, each to the least loaded CTA) is no worse, that plan is taken instead: it needs no merge.
#include <algorithm>
#include <functional>
#include <queue>
#include <vector>

#include "kernels.h"

namespace pc {

namespace {
// costs in quarter blocks (one block = the two heads' work on 128 context slots)
constexpr int64_t BLOCK_COST = 4;
constexpr int64_t ITEM_COST = 12;       // Q load, pipeline fill, output rows (measured: 6 and 16 are both slower)
constexpr int64_t PARTIAL_COST = 2;     // fp32 partial output instead of fp16 rows
constexpr int64_t MERGE_COST = 16;      // the merge kernel behind the attention kernel
constexpr int MIN_PART = 3;             // blocks; shorter parts are not worth an item
}  // namespace

int64_t plan_attention(const std::vector<AttnBaseTile>& tiles, int units_per_tile, int n_sms, int max_partial_slots,
                       std::vector<AttnItem>* items, std::vector<int32_t>* cta_first, std::vector<AttnMerge>* merges) {
  items->clear();
  cta_first->clear();
  merges->clear();
  const int G = units_per_tile;
  const int64_t n_units = static_cast<int64_t>(tiles.size()) * G;
  if (n_units == 0 || n_sms <= 0) { cta_first->push_back(0); return 0; }
  auto make_item = [&](const AttnBaseTile& t, int unit, int b0, int b1, int slot) {
    AttnItem it{};
    it.row0 = t.row0; it.n_rows = t.n_rows; it.ctx0 = t.ctx0;
    it.blk_begin = b0; it.blk_end = b1; it.partial_slot = slot; it.unit = unit;
    return it;
  };

  // ---- plan A: whole units, longest first, each to the least loaded CTA
  const int n_ctas_a = static_cast<int>(std::min<int64_t>(n_sms, n_units));
  std::vector<int32_t> order(tiles.size());
  for (size_t i = 0; i < tiles.size(); ++i) order[i] = static_cast<int32_t>(i);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return tiles[a].n_blocks > tiles[b].n_blocks; });
  typedef std::pair<int64_t, int> Load;   // (load, cta)
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int c = 0; c < n_ctas_a; ++c) heap.push(Load(0, c));
  std::vector<std::vector<std::pair<int32_t, int32_t>>> lists_a(static_cast<size_t>(n_ctas_a));   // (tile, unit)
  int64_t makespan_a = 0;
  for (int32_t ti : order)
    for (int u = 0; u < G; ++u) {
      Load ld = heap.top();
      heap.pop();
      ld.first += tiles[ti].n_blocks * BLOCK_COST + ITEM_COST;
      makespan_a = std::max(makespan_a, ld.first);
      lists_a[static_cast<size_t>(ld.second)].push_back(std::make_pair(ti, u));
      heap.push(ld);
    }

  // ---- plan B: contiguous spans of equal cost
  struct Part { int32_t tile, unit, b0, b1, cta; bool partial; };
  std::vector<Part> parts;
  auto walk = [&](int64_t T, bool emit, int* ctas_used, int* n_partial) {
    int c = 0, partials = 0;
    int64_t load = 0;
    for (size_t ti = 0; ti < tiles.size(); ++ti)
      for (int u = 0; u < G; ++u) {
        const int L = tiles[ti].n_blocks;
        int b = 0;
        while (b < L) {
          const int rem = L - b;
          const int64_t need_all = rem * BLOCK_COST + ITEM_COST + (b > 0 ? PARTIAL_COST : 0);
          if (load + need_all <= T) {
            if (emit) parts.push_back(Part{static_cast<int32_t>(ti), u, b, L, c, b > 0});
            partials += b > 0 ? 1 : 0;
            load += need_all;
            b = L;
            continue;
          }
          const int64_t room = (T - load - ITEM_COST - PARTIAL_COST) / BLOCK_COST;
          const int take = static_cast<int>(std::min<int64_t>(room, rem - MIN_PART));
          if (take >= MIN_PART) {
            if (emit) parts.push_back(Part{static_cast<int32_t>(ti), u, b, b + take, c, true});
            ++partials;
            b += take;
          } else if (load == 0) {
            return false;          // not even the shortest part fits an empty CTA
          }
          ++c;
          load = 0;
          if (c >= n_sms) return false;
        }
      }
    *ctas_used = c + 1;
    *n_partial = partials;
    return partials <= max_partial_slots;
  };
  int64_t total_cost = 0, longest = 0;
  for (const AttnBaseTile& t : tiles) {
    total_cost += G * (t.n_blocks * BLOCK_COST + ITEM_COST);
    longest = std::max<int64_t>(longest, t.n_blocks * BLOCK_COST + ITEM_COST);
  }
  int64_t T = std::max<int64_t>((total_cost + n_sms - 1) / n_sms, MIN_PART * BLOCK_COST + ITEM_COST + PARTIAL_COST);
  const int64_t step = std::max<int64_t>(1, T / 128);
  int ctas_b = 0, partials_b = 0;
  bool have_b = false;
  for (; T <= total_cost + PARTIAL_COST * 2; T += step)
    if (walk(T, false, &ctas_b, &partials_b)) { have_b = true; break; }
  const int64_t makespan_b = T + (partials_b > 0 ? MERGE_COST : 0);

  if (have_b && makespan_b < makespan_a) {
    walk(T, true, &ctas_b, &partials_b);
    int next_slot = 0;
    cta_first->assign(static_cast<size_t>(ctas_b) + 1, 0);
    for (size_t i = 0; i < parts.size(); ++i) {
      const Part& p = parts[i];
      const AttnBaseTile& t = tiles[static_cast<size_t>(p.tile)];
      int slot = -1;
      if (p.partial) {
        slot = next_slot++;
        if (p.b0 == 0) {
          AttnMerge mg{};
          mg.row0 = t.row0; mg.n_rows = t.n_rows; mg.partial_slot0 = slot; mg.n_parts = 0; mg.unit = p.unit;
          merges->push_back(mg);
        }
        merges->back().n_parts += 1;
      }
      items->push_back(make_item(t, p.unit, p.b0, p.b1, slot));
      (*cta_first)[static_cast<size_t>(p.cta) + 1] = static_cast<int32_t>(i + 1);
    }
    for (size_t c = 1; c < cta_first->size(); ++c)          // a CTA the walk skipped keeps an empty range
      (*cta_first)[c] = std::max((*cta_first)[c], (*cta_first)[c - 1]);
    return makespan_b;
  }
  cta_first->assign(static_cast<size_t>(n_ctas_a) + 1, 0);
  for (int c = 0; c < n_ctas_a; ++c) {
    for (const auto& tu : lists_a[static_cast<size_t>(c)]) {
      const AttnBaseTile& t = tiles[static_cast<size_t>(tu.first)];
      items->push_back(make_item(t, tu.second, 0, t.n_blocks, -1));
    }
    (*cta_first)[static_cast<size_t>(c) + 1] = static_cast<int32_t>(items->size());
  }
  return makespan_a;
}

}  // namespace pc
