// Decode work scheduling (host only).
//
// The compressed cache is head-heterogeneous: a retrieval head holds the whole context, every other
// head holds sinks + window only (Algorithm 1), and a serving batch mixes context lengths.  One
// launch covers them all.  The heads' page streams are laid end to end (longest head first) and cut
// in two regions:
//   * the first `static_pct` percent is cut into one equal SPAN per CTA.  A span crosses head
//     boundaries where it must, so it is a short run of work items (one per head it touches), and
//     the long heads end up in few, large parts;
//   * the rest is cut into TAIL items that the CTAs pull one at a time as they finish their spans, which
//     evens out whatever difference in speed there was.  Their sizes shrink along the stream (guided
//     self-scheduling): each is 1 / tail_items_per_cta of an equal share of the tail that is left, but
//     not less than min_chunk pages, so the queue ends on small items without starting on them.
// A job is what a CTA pops from the queue: a span (several consecutive items) or one tail item.
// A head cut into several parts produces one partial (m, l, o) record per part.  Heads in few parts are merged
// by the streaming kernel itself (the part written last folds them); a small combine kernel that follows it
// merges the others, one CTA per such head.
#include <algorithm>
#include <cstdint>
#include <numeric>
#include <vector>

#include "razor_internal.h"

namespace razor {

namespace {

struct Piece {
  int head, begin, end;   // pages [begin, end) of the head
  int job;                // span index, or n_spans + running index for tail pieces
};

}  // namespace

int build_schedule(const int32_t* pages, int n_heads, const SchedParams& sp, int max_items, WorkItem* out,
                   int32_t* jobs, MultiHead* multi, SchedInfo* info) {
  const int n_ctas = std::max(1, sp.n_ctas);
  const int min_chunk = std::max(1, sp.min_chunk_pages);
  const int static_pct = std::min(100, std::max(0, sp.static_pct));
  const int tail_per_cta = std::max(1, sp.tail_items_per_cta);

  std::vector<int> order(n_heads);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return pages[a] > pages[b]; });
  long long total = 0;
  for (int h = 0; h < n_heads; ++h) total += pages[h];

  // Spans: equal, at least min_chunk pages, at most one per CTA.
  const long long static_pages = total * static_pct / 100;
  long long span = (static_pages + n_ctas - 1) / n_ctas;
  if (span < min_chunk) span = min_chunk;
  const long long n_spans = std::min<long long>(n_ctas, static_pages / span);
  const long long static_end = n_spans * span;
  const long long tail_pages = total - static_end;
  long long floor_chunk = min_chunk;   // smallest tail item; grows only if the items would not fit
  long long first_chunk = 0;

  std::vector<Piece> pieces;
  for (;;) {   // grow the smallest tail item until the items fit
    pieces.clear();
    long long pos = 0, tail_left = tail_pages;
    int tail_jobs = 0;
    first_chunk = 0;
    for (int oi = 0; oi < n_heads; ++oi) {
      const int h = order[oi];
      const int p = pages[h];
      int at = 0;
      while (at < p && pos + at < static_end) {   // static region: cut at span boundaries
        const long long k = (pos + at) / span;
        const int stop = (int)std::min<long long>(p, (k + 1) * span - pos);
        pieces.push_back({h, at, stop, (int)k});
        at = stop;
      }
      if (p == 0) pieces.push_back({h, 0, 0, (int)n_spans + tail_jobs++});   // an empty head gets one empty item
      while (at < p) {   // dynamic region: guided sizes, cut at the head's end
        long long chunk = (tail_left + (long long)n_ctas * tail_per_cta - 1) / ((long long)n_ctas * tail_per_cta);
        if (chunk < floor_chunk) chunk = floor_chunk;
        if (first_chunk == 0) first_chunk = chunk;
        int stop = (int)std::min<long long>(p, at + chunk);
        if (p - stop < floor_chunk / 2) stop = p;   // no crumbs at the end of a head
        pieces.push_back({h, at, stop, (int)n_spans + tail_jobs++});
        tail_left -= stop - at;
        at = stop;
      }
      pos += p;
    }
    if ((long long)pieces.size() <= max_items) break;
    if (floor_chunk > total) return -1;
    floor_chunk += (floor_chunk + 3) / 4;
  }

  // Per head: partial records for the heads in several parts (never more records than items).
  std::vector<int> n_parts(n_heads, 0), rec_base(n_heads, 0), next_part(n_heads, 0);
  for (const Piece& pc : pieces) n_parts[pc.head] += 1;
  int rec = 0, n_multi = 0;
  for (int oi = 0; oi < n_heads; ++oi) {   // longest heads first: they have the most parts to merge
    const int h = order[oi];
    if (n_parts[h] < 2) continue;
    rec_base[h] = rec;
    // heads in few parts are folded by the streaming kernel itself; only the others go on the combine kernel's list
    if (n_parts[h] > sp.merge_max_parts) multi[n_multi++] = MultiHead{h, rec, n_parts[h], 0};
    rec += n_parts[h];
  }
  // Job order: spans in stream order, then the tail items.  Jobs are numbered along the stream, so the
  // pieces of one head stay in page order and part indices can be handed out as the pieces come.
  std::stable_sort(pieces.begin(), pieces.end(), [](const Piece& a, const Piece& b) { return a.job < b.job; });
  int n = 0, n_jobs = 0, last_job = -1, first_tail_job = -1;
  for (const Piece& pc : pieces) {
    if (pc.job != last_job) {
      if (pc.job >= n_spans && first_tail_job < 0) first_tail_job = n_jobs;
      jobs[n_jobs++] = n;
      last_job = pc.job;
    }
    WorkItem w;
    w.head = pc.head;
    w.page_begin = pc.begin;
    w.page_end = (pc.end == pages[pc.head]) ? -1 : pc.end;   // the head's last part grows with appends
    w.part_idx = next_part[pc.head]++;
    w.n_parts = n_parts[pc.head];
    w.rec_base = rec_base[pc.head];
    w.merge_here = (n_parts[pc.head] > 1 && n_parts[pc.head] <= sp.merge_max_parts) ? 1 : 0;
    w.pad1 = 0;
    out[n++] = w;
  }
  jobs[n_jobs] = n;
  if (info) {
    info->n_items = n;
    info->n_jobs = n_jobs;
    info->n_spans = first_tail_job < 0 ? n_jobs : first_tail_job;
    info->span_pages = (int)span;
    info->chunk_pages = (int)floor_chunk;
    info->n_multi = n_multi;
  }
  return n;
}

}  // namespace razor
