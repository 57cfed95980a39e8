// Host-side slot planner of the HBM expert cache (one table per layer).
//
// The paper's own policy is load-use-evict per layer (Sec. V-C "Per-token Prefetch Budget
// Distribution": each layer's experts are loaded, used and evicted before the next layer); that
// is cache_reuse = false.  With cache_reuse = true the C slots persist across decode steps and
// a victim is the slot with the smallest (stamp, slot index) whose expert is not protected.
// All decisions are integer-only and depend on sets, never on the order inside a set.
#pragma once
#include <algorithm>
#include <cstdint>
#include <vector>

namespace apex {

struct SlotCopy {
  int32_t expert;
  int32_t slot;
  int32_t wave;  // 0 = prefetch, >= 1 = demand wave
};

class SlotTable {
 public:
  SlotTable(int N, int C, bool cache_reuse)
      : N_(N), C_(C), reuse_(cache_reuse), slot_expert_(C, -1), expert_slot_(N, -1), slot_stamp_(C, -1) {}

  int N() const { return N_; }
  int C() const { return C_; }
  int64_t clock() const { return clock_; }
  const std::vector<int32_t>& expert_slot() const { return expert_slot_; }
  const std::vector<int32_t>& slot_expert() const { return slot_expert_; }
  const std::vector<int64_t>& slot_stamp() const { return slot_stamp_; }

  uint64_t resident_mask() const {
    uint64_t m = 0;
    for (int e = 0; e < N_; ++e)
      if (expert_slot_[e] >= 0) m |= (1ull << e);
    return m;
  }

  void begin_step() {
    ++clock_;
    if (!reuse_) clear();
  }

  void clear() {
    std::fill(slot_expert_.begin(), slot_expert_.end(), -1);
    std::fill(expert_slot_.begin(), expert_slot_.end(), -1);
    std::fill(slot_stamp_.begin(), slot_stamp_.end(), (int64_t)-1);
  }

  void touch(int e) {
    if (e >= 0 && e < N_ && expert_slot_[e] >= 0) slot_stamp_[expert_slot_[e]] = clock_;
  }

  // Takes e out of the table and leaves its slot empty (never used): for a planned install whose copy
  // could not be issued.  The previous occupant was already taken out by the plan.
  void drop(int e) {
    if (e < 0 || e >= N_ || expert_slot_[e] < 0) return;
    const int s = expert_slot_[e];
    expert_slot_[e] = -1;
    slot_expert_[s] = -1;
    slot_stamp_[s] = -1;
  }

  // Candidate lists of B tokens -> prefetch set U: experts ordered by (number of tokens that want
  // them descending, index ascending), truncated to C; planned in ascending index with U protected.
  // Returns false if no slot could be found (cannot happen while |U| <= C).
  bool plan_prefetch(const int32_t* cand, const int32_t* ncand, int B, int stride, std::vector<SlotCopy>* copies,
                     uint64_t* U_mask_out = nullptr) {
    int count[64] = {0};
    for (int b = 0; b < B; ++b)
      for (int j = 0; j < ncand[b]; ++j) {
        int e = cand[(size_t)b * stride + j];
        if (e >= 0 && e < N_) ++count[e];
      }
    std::vector<int> wanted;
    for (int e = 0; e < N_; ++e)
      if (count[e] > 0) wanted.push_back(e);
    std::stable_sort(wanted.begin(), wanted.end(), [&](int a, int b) { return count[a] > count[b]; });
    if ((int)wanted.size() > C_) wanted.resize(C_);
    uint64_t U = 0;
    for (int e : wanted) U |= (1ull << e);
    if (U_mask_out) *U_mask_out = U;
    for (int e = 0; e < N_; ++e) {
      if (!((U >> e) & 1)) continue;
      if (!acquire(e, U, 0, 0, copies)) return false;
    }
    return true;
  }

  // Routed sets of B tokens (exact mode).  Resident members of Need are touched; the missing ones
  // are installed in ascending index, in chunks of at most C (wave 1, 2, ...), the chunk being
  // protected and members of Need being the last choice as victims.
  bool plan_demand(const int32_t* K_r, int B, int k, std::vector<SlotCopy>* copies, uint64_t* need_mask_out = nullptr) {
    uint64_t need = 0;
    for (int i = 0; i < B * k; ++i)
      if (K_r[i] >= 0 && K_r[i] < N_) need |= (1ull << K_r[i]);
    if (need_mask_out) *need_mask_out = need;
    std::vector<int> missing;
    for (int e = 0; e < N_; ++e) {
      if (!((need >> e) & 1)) continue;
      if (expert_slot_[e] >= 0)
        touch(e);
      else
        missing.push_back(e);
    }
    int wave = 0;
    for (size_t i = 0; i < missing.size(); i += C_) {
      ++wave;
      uint64_t chunk = 0;
      size_t end = std::min(missing.size(), i + (size_t)C_);
      for (size_t j = i; j < end; ++j) chunk |= (1ull << missing[j]);
      for (size_t j = i; j < end; ++j)
        if (!acquire(missing[j], chunk, need, wave, copies)) return false;
    }
    return true;
  }

  void get(int32_t* expert_slot, int64_t* slot_stamp, int64_t* clock) const {
    if (expert_slot) std::copy(expert_slot_.begin(), expert_slot_.end(), expert_slot);
    if (slot_stamp) std::copy(slot_stamp_.begin(), slot_stamp_.end(), slot_stamp);
    if (clock) *clock = clock_;
  }

  // Returns false when two experts name one slot or an index is out of range.
  bool set(const int32_t* expert_slot, const int64_t* slot_stamp, int64_t clock) {
    std::vector<int32_t> se(C_, -1);
    for (int e = 0; e < N_; ++e) {
      int s = expert_slot[e];
      if (s < -1 || s >= C_) return false;
      if (s >= 0) {
        if (se[s] != -1) return false;
        se[s] = e;
      }
    }
    slot_expert_ = se;
    expert_slot_.assign(expert_slot, expert_slot + N_);
    slot_stamp_.assign(slot_stamp, slot_stamp + C_);
    clock_ = clock;
    return true;
  }

 private:
  // Makes e resident.  A hit is touched.  Otherwise the victim minimises
  // (holds a deprioritised expert ? 1 : 0, stamp, slot index) over slots not holding a protected expert.
  bool acquire(int e, uint64_t protect, uint64_t deprioritise, int wave, std::vector<SlotCopy>* copies) {
    if (expert_slot_[e] >= 0) {
      touch(e);
      return true;
    }
    int best = -1;
    int best_dep = 0;
    for (int s = 0; s < C_; ++s) {
      int held = slot_expert_[s];
      if (held >= 0 && ((protect >> held) & 1)) continue;
      int dep = (held >= 0 && ((deprioritise >> held) & 1)) ? 1 : 0;
      if (best < 0 || dep < best_dep || (dep == best_dep && slot_stamp_[s] < slot_stamp_[best])) {
        best = s;
        best_dep = dep;
      }
    }
    if (best < 0) return false;
    if (slot_expert_[best] >= 0) expert_slot_[slot_expert_[best]] = -1;
    slot_expert_[best] = e;
    expert_slot_[e] = best;
    slot_stamp_[best] = clock_;
    if (copies) copies->push_back({e, best, wave});
    return true;
  }

  int N_, C_;
  bool reuse_;
  std::vector<int32_t> slot_expert_, expert_slot_;
  std::vector<int64_t> slot_stamp_;
  int64_t clock_ = 0;
};

}  // namespace apex
