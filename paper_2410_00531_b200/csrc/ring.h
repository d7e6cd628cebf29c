// Sliding-window block ring: host-side ordering logic of the memory scheduler
// (Sec. 3.3 / Appendix A.2), independent of CUDA so that it can be driven by a
// recording back end in tests.
//
// Blocks execute in the fixed cyclic order attention_0, ffn_0, attention_1, ...
// (2L blocks per pass, repeated for every token).  The window holds at most w
// blocks, the executing one included (Prop. 5): floor(w/2) attention-sized slots
// and ceil(w/2) FFN-sized slots (w = 1: one slot shared by both kinds).  Loads
// are issued strictly in execution order on one copy queue; a load into a slot
// waits until the slot's previous occupant has been released by the compute
// queue ("wait" and "release" of the paper's context manager).
#pragma once
#include <stdint.h>

#include <vector>

namespace tpi {

struct RingBackend {
  void* ctx = nullptr;
  // copy queue: wait until compute released `slot`; copy `block` into `slot`; mark slot loaded
  int (*copy_wait_released)(void* ctx, int slot) = nullptr;
  int (*copy_block)(void* ctx, int slot, int block) = nullptr;
  int (*copy_record_loaded)(void* ctx, int slot) = nullptr;
  // compute queue: wait until `slot` is loaded; mark slot released
  int (*compute_wait_loaded)(void* ctx, int slot) = nullptr;
  int (*compute_record_released)(void* ctx, int slot) = nullptr;
};

class Ring {
 public:
  // retained (may be null): retained[b] != 0 marks block b as kept resident outside the window (the paper's
  // block retention, Prop. 6): such blocks are never loaded and take no slot; the loader cycles over the rest.
  void configure(int n_blocks, int window, const RingBackend& be, const char* retained = nullptr) {
    n_blocks_ = n_blocks;
    w_ = window;
    be_ = be;
    if (window <= 1) { nA_ = 0; nF_ = 1; }
    else { nA_ = window / 2; nF_ = (window + 1) / 2; }
    holds_.assign(nA_ + nF_, -1);
    released_.assign(nA_ + nF_, 1);
    next_exec_ = next_load_ = 0;
    loads_issued_ = 0;
    retained_.assign(n_blocks, 0);
    seq_.clear();
    rank_.clear();
    kind_count_[0] = kind_count_[1] = 0;
    for (int b = 0; b < n_blocks; ++b) {
      if (retained && retained[b]) { retained_[b] = 1; continue; }
      seq_.push_back(b);
      rank_.push_back(kind_count_[b & 1]++);
    }
  }
  int n_slots() const { return nA_ + nF_; }
  int n_attn_slots() const { return nA_; }
  int n_ffn_slots() const { return nF_; }
  int64_t loads_issued() const { return loads_issued_; }
  int64_t next_exec() const { return next_exec_; }
  bool is_retained(int block) const { return retained_[block] != 0; }
  int n_streamed() const { return (int)seq_.size(); }

  // c counts streamed blocks since the start; slots are dealt per kind in arrival order
  int slot_of(int64_t c) const {
    if (nA_ == 0) return 0;
    const int n = (int)seq_.size();
    const int i = (int)(c % n);
    const int kind = seq_[i] & 1;
    const int64_t idx = (c / n) * kind_count_[kind] + rank_[i];  // running index among blocks of the same kind
    return kind == 0 ? (int)(idx % nA_) : nA_ + (int)(idx % nF_);
  }

  // Issue every load whose slot is free, in order.  Returns 0 or a back-end error.
  int pump() {
    if (seq_.empty()) return 0;
    for (;;) {
      const int s = slot_of(next_load_);
      if (holds_[s] >= 0 && !released_[s]) return 0;  // previous occupant still in use
      int rc;
      if (holds_[s] >= 0 && (rc = be_.copy_wait_released(be_.ctx, s))) return rc;
      if ((rc = be_.copy_block(be_.ctx, s, seq_[(size_t)(next_load_ % (int64_t)seq_.size())]))) return rc;
      if ((rc = be_.copy_record_loaded(be_.ctx, s))) return rc;
      holds_[s] = next_load_;
      released_[s] = 0;
      ++next_load_;
      ++loads_issued_;
    }
  }

  // "wait": make the compute queue wait for the next streamed block in order; returns its slot (< 0: error).
  int acquire(int block) {
    if (seq_.empty() || block != seq_[(size_t)(next_exec_ % (int64_t)seq_.size())]) return -1000;
    int rc = pump();
    if (rc) return rc < 0 ? rc : -rc;
    const int s = slot_of(next_exec_);
    if (holds_[s] != next_exec_) return -1001;  // cannot happen while slots >= 1
    if ((rc = be_.compute_wait_loaded(be_.ctx, s))) return rc < 0 ? rc : -rc;
    return s;
  }

  // "release": the block's last kernel has been enqueued.
  int release(int block) {
    if (seq_.empty() || block != seq_[(size_t)(next_exec_ % (int64_t)seq_.size())]) return -1000;
    const int s = slot_of(next_exec_);
    int rc = be_.compute_record_released(be_.ctx, s);
    if (rc) return rc;
    released_[s] = 1;
    ++next_exec_;
    return pump();
  }

 private:
  int n_blocks_ = 0, w_ = 0, nA_ = 0, nF_ = 1;
  RingBackend be_;
  std::vector<int64_t> holds_;
  std::vector<char> released_, retained_;
  std::vector<int> seq_, rank_;  // streamed block ids in execution order; rank among blocks of the same kind
  int kind_count_[2] = {0, 0};
  int64_t next_exec_ = 0, next_load_ = 0, loads_issued_ = 0;
};

}  // namespace tpi
