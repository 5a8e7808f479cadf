// Decode work scheduling (host only).
//
// The compressed cache is head-heterogeneous: a retrieval head holds the whole context, every other
// head holds sinks + window only (Algorithm 1), and a serving batch mixes context lengths.  One
// launch covers them all, so the token streams are cut into page ranges of near-equal size; the
// kernel's warps pull ranges from a queue.  A head cut into several parts produces one partial
// (m, l, o) record per part; the warp that finishes a head's last part merges them.
#include <algorithm>
#include <cstdint>

#include "razor_internal.h"

namespace razor {

int build_schedule(const int32_t* pages, int n_heads, int target_items, int max_items, WorkItem* out,
                   int* chunk_pages_out) {
  long long total = 0;
  for (int h = 0; h < n_heads; ++h) total += pages[h];
  if (target_items < 1) target_items = 1;
  // Every head costs one item at least; the rest of the budget is spread by size.
  int budget = std::max(1, std::min(target_items, max_items - n_heads));
  long long chunk = (total + budget - 1) / budget;
  if (chunk < kMinChunkPages) chunk = kMinChunkPages;
  if (chunk_pages_out) *chunk_pages_out = (int)chunk;

  int n = 0, slot = 0;
  for (int h = 0; h < n_heads; ++h) {
    const int p = pages[h];
    int parts = (int)((p + chunk - 1) / chunk);
    if (parts < 1) parts = 1;
    for (int i = 0; i < parts; ++i) {
      if (n >= max_items) return -1;
      WorkItem w;
      w.head = h;
      w.page_begin = (int)((long long)p * i / parts);
      w.page_end = (i == parts - 1) ? -1 : (int)((long long)p * (i + 1) / parts);
      w.part_idx = i;
      w.n_parts = parts;
      w.part_base = slot;
      w.pad0 = w.pad1 = 0;
      out[n++] = w;
    }
    slot += parts;
  }
  // Longest parts first: the queue then ends on the short ones, which trims the tail of the launch.
  std::stable_sort(out, out + n, [&](const WorkItem& a, const WorkItem& b) {
    const int la = (a.page_end < 0 ? pages[a.head] : a.page_end) - a.page_begin;
    const int lb = (b.page_end < 0 ? pages[b.head] : b.page_end) - b.page_begin;
    return la > lb;
  });
  return n;
}

}  // namespace razor
