// Decode work scheduling (host only).
//
// The compressed cache is head-heterogeneous: a retrieval head holds the whole context, every other
// head holds sinks + window only (Algorithm 1), and a serving batch mixes context lengths.  One
// launch covers them all, so the token streams are cut into page ranges of near-equal size (work
// items); the kernel's CTAs pull items from a queue and each streams its item with all of its warps.
// A head cut into several parts produces one partial (m, l, o) record per part; records are merged
// by a tree of fan-in kMergeFanIn whose nodes are closed by whichever CTA delivers a node's last
// input, so no merge is longer than kMergeFanIn records however long the head is.
#include <algorithm>
#include <cstdint>

#include "razor_internal.h"

namespace razor {

void tree_sizes(int n_parts, int* n_recs, int* n_tickets) {
  int recs = 0, tickets = 0;
  if (n_parts > 1) {
    int n = n_parts;
    recs = n;
    while (n > 1) {
      n = (n + kMergeFanIn - 1) / kMergeFanIn;
      tickets += n;          // one counter per node of this level
      if (n > 1) recs += n;  // the root writes the output, not a record
    }
  }
  *n_recs = recs;
  *n_tickets = tickets;
}

int build_schedule(const int32_t* pages, int n_heads, int target_items, int min_chunk, int max_items, int max_recs,
                   int max_tickets, WorkItem* out, int* chunk_pages_out) {
  long long total = 0;
  for (int h = 0; h < n_heads; ++h) total += pages[h];
  if (target_items < 1) target_items = 1;
  if (min_chunk < 1) min_chunk = 1;
  long long chunk = (total + target_items - 1) / target_items;
  if (chunk < min_chunk) chunk = min_chunk;
  // Every head costs one item at least; grow the chunk until the items fit.
  for (;;) {
    long long n = 0;
    for (int h = 0; h < n_heads; ++h) n += std::max<long long>(1, (pages[h] + chunk - 1) / chunk);
    if (n <= max_items) break;
    if (chunk > total) return -1;
    chunk += (chunk + 3) / 4;
  }
  if (chunk_pages_out) *chunk_pages_out = (int)chunk;

  int n = 0, rec = 0, ticket = 0;
  for (int h = 0; h < n_heads; ++h) {
    const int p = pages[h];
    int parts = (int)((p + chunk - 1) / chunk);
    if (parts < 1) parts = 1;
    int n_recs, n_tickets;
    tree_sizes(parts, &n_recs, &n_tickets);
    if (rec + n_recs > max_recs || ticket + n_tickets > max_tickets) return -1;
    for (int i = 0; i < parts; ++i) {
      WorkItem w;
      w.head = h;
      w.page_begin = (int)((long long)p * i / parts);
      w.page_end = (i == parts - 1) ? -1 : (int)((long long)p * (i + 1) / parts);
      w.part_idx = i;
      w.n_parts = parts;
      w.rec_base = rec;
      w.ticket_base = ticket;
      w.pad = 0;
      out[n++] = w;
    }
    rec += n_recs;
    ticket += n_tickets;
  }
  // Heads with the deepest combine trees first (their merges then overlap the streaming of the
  // rest), longer parts before shorter ones within equal depth: the queue ends on short items of
  // heads whose final merge is a single node.
  std::stable_sort(out, out + n, [&](const WorkItem& a, const WorkItem& b) {
    if (a.n_parts != b.n_parts) return a.n_parts > b.n_parts;
    const int la = (a.page_end < 0 ? pages[a.head] : a.page_end) - a.page_begin;
    const int lb = (b.page_end < 0 ? pages[b.head] : b.page_end) - b.page_begin;
    return la > lb;
  });
  return n;
}

}  // namespace razor
