// Host-side bookkeeping of the paged compressed cache: which 64-slot pages each sequence
// holds, how many sequences share a page, and which pages must be allocated or copied before a
// sequence may write a slot.  Closed slots are immutable (Section 4.1: only the newest slot of
// a sequence is ever written), so beams that fork from one hypothesis share every page except
// the one that holds their newest slot, which is copied on the first write.
//
// Pure host code: it decides, the caller enqueues the device work it is told about (page-table
// entries to set, pages to copy) on its stream before the kernels that rely on them.
#pragma once

#include <vector>

namespace mtla {

constexpr int kPageSlots = 64;   // one page = one tile of the decode attention

struct PageSet {     // page_table[seq][index] = page
  int seq, index, page;
};
struct PageCopy {    // rows [0, rows) of page src -> page dst
  int src, dst, rows;
};

class PagePool {
 public:
  PagePool(int n_pages, int max_seqs, int max_pages_per_seq)
      : n_pages_(n_pages), max_seqs_(max_seqs), max_pages_(max_pages_per_seq), cur_(0) {
    for (int i = 0; i < 2; ++i) {
      table_[i].assign((size_t)max_seqs * max_pages_per_seq, -1);
      held_[i].assign(max_seqs, 0);
    }
    reset();
  }

  void reset() {
    ref_.assign(n_pages_, 0);
    free_.clear();
    for (int p = n_pages_ - 1; p >= 0; --p) free_.push_back(p);   // page 0 is handed out first
    held_[cur_].assign(max_seqs_, 0);
  }

  int n_pages() const { return n_pages_; }
  int max_pages_per_seq() const { return max_pages_; }
  int pages_free() const { return (int)free_.size(); }
  int pages_in_use() const { return n_pages_ - (int)free_.size(); }
  int pages_held(int seq) const { return held_[cur_][seq]; }
  const int* row(int seq) const { return &table_[cur_][(size_t)seq * max_pages_]; }
  int ref(int page) const { return ref_[page]; }

  // Pages `prepare` would take from the free list for the same arguments.
  int pages_needed(int seq, int n_slots, int write_slot) const {
    const int have = held_[cur_][seq], want = pages_for(n_slots);
    int need = want > have ? want - have : 0;
    if (write_slot >= 0) {
      const int k = write_slot / kPageSlots;
      if (k < have && ref_[row(seq)[k]] > 1) ++need;
    }
    return need;
  }

  // Makes slots [0, n_slots) of `seq` addressable and, if write_slot >= 0, the page that
  // holds it private to `seq`.  Appends the device work this implies.  The caller has checked
  // pages_needed() against pages_free() for the whole batch; returns false on exhaustion or a
  // sequence longer than the table row.
  bool prepare(int seq, int n_slots, int write_slot, std::vector<PageSet>* sets,
               std::vector<PageCopy>* copies) {
    const int want = pages_for(n_slots);
    if (want > max_pages_) return false;
    int* r = &table_[cur_][(size_t)seq * max_pages_];
    int& have = held_[cur_][seq];
    while (have < want) {
      const int p = take();
      if (p < 0) return false;
      r[have] = p;
      sets->push_back({seq, have, p});
      ++have;
    }
    if (write_slot >= 0) {
      const int k = write_slot / kPageSlots;
      if (k >= have) return false;
      const int old = r[k];
      if (ref_[old] > 1) {
        const int p = take();
        if (p < 0) return false;
        --ref_[old];
        r[k] = p;
        sets->push_back({seq, k, p});
        // The slot being written is rewritten in full; only the rows before it carry state.
        const int rows = write_slot % kPageSlots;
        if (rows > 0) copies->push_back({old, p, rows});
      }
    }
    return true;
  }

  // Drops every page of `seq`.
  void release(int seq) {
    int* r = &table_[cur_][(size_t)seq * max_pages_];
    for (int k = 0; k < held_[cur_][seq]; ++k) drop(r[k]);
    held_[cur_][seq] = 0;
  }

  // Beam reordering: sequence b of the new batch becomes a copy of old sequence parents[b]
  // (sharing its pages); old sequences that nobody continues give their pages back.  The
  // tables are double-buffered and the device mirrors the flip.
  void reorder(const int* parents, int n_new, int n_old) {
    const int nxt = cur_ ^ 1;
    for (int b = 0; b < n_new; ++b) {
      const int p = parents[b];
      const int* src = &table_[cur_][(size_t)p * max_pages_];
      int* dst = &table_[nxt][(size_t)b * max_pages_];
      const int n = held_[cur_][p];
      for (int k = 0; k < n; ++k) {
        dst[k] = src[k];
        ++ref_[src[k]];
      }
      held_[nxt][b] = n;
    }
    for (int b = n_new; b < max_seqs_; ++b) held_[nxt][b] = 0;
    for (int b = 0; b < n_old; ++b) release(b);
    cur_ = nxt;
  }

  int current_buffer() const { return cur_; }

  static int pages_for(int n_slots) { return (n_slots + kPageSlots - 1) / kPageSlots; }

 private:
  int take() {
    if (free_.empty()) return -1;
    const int p = free_.back();
    free_.pop_back();
    ref_[p] = 1;
    return p;
  }
  void drop(int page) {
    if (--ref_[page] == 0) free_.push_back(page);
  }

  int n_pages_, max_seqs_, max_pages_, cur_;
  std::vector<int> table_[2];
  std::vector<int> held_[2];
  std::vector<int> ref_;
  std::vector<int> free_;
};

}  // namespace mtla
