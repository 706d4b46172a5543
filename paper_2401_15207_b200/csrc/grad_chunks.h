// Chunks of a group's flat gradient in the order the backward pass completes them (host logic only).
//
// The backward pass walks a group's tensors from the top of its span to the bottom, so the flat
// gradient becomes final from its end towards its start.  A data-parallel run can therefore start
// reducing the tail of the buffer over the ranks while the head is still being computed.  The
// planner is told the tensors of the span (ascending offsets) and then, one by one, which tensor's
// gradient has just become final; whenever the finished suffix of the span has grown by at least
// `min_elems` (or has reached the start of the span) it hands out that piece as the next chunk.
#pragma once
#include <stddef.h>

#include <vector>

namespace hift {

struct GradChunkPlanner {
  struct Tensor { size_t off, n; bool done; };
  std::vector<Tensor> t;
  size_t span = 0;        // elements in the whole span
  size_t mark = 0;        // everything at or above this offset has been handed out
  size_t min_elems = 1;

  void reset(size_t span_elems, size_t min_chunk_elems) {
    t.clear();
    span = mark = span_elems;
    min_elems = min_chunk_elems ? min_chunk_elems : 1;
  }
  int add(size_t off, size_t n) { t.push_back(Tensor{off, n, false}); return (int)t.size() - 1; }
  // Tensor `idx` is final.  Returns true and the piece [*off, *off + *n) when a chunk is due.
  bool complete(int idx, size_t* off, size_t* n) {
    if (idx < 0 || idx >= (int)t.size()) return false;
    t[idx].done = true;
    int i = (int)t.size();
    while (i > 0 && t[i - 1].done) --i;               // tensors i .. end are all final
    const size_t wm = i == 0 ? 0 : (i == (int)t.size() ? span : t[i].off);
    if (wm < mark && (mark - wm >= min_elems || i == 0)) {
      *off = wm; *n = mark - wm; mark = wm;
      return true;
    }
    return false;
  }
  // Whatever has not been handed out yet (tensors that never reported): the last chunk.
  bool flush(size_t* off, size_t* n) {
    if (mark == 0) return false;
    *off = 0; *n = mark; mark = 0;
    return true;
  }
};

}  // namespace hift
