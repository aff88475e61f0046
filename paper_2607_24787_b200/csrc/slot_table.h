// Expert slot table: which routed experts of each layer hold an HBM cache slot.
//
// Host-side integer logic of the prefetch controller (Section 3.3 of the paper):
// an expert "has a slot" from the moment a transfer into the slot is issued, so the
// set of experts with a slot is exactly A ∪ U (available or in transfer) and is what
// the budgeted selection excludes. Eviction is least-recently-used on one global
// tick; equal ticks are broken by the lower expert id and empty slots are taken
// lowest index first, so which experts are resident never depends on placement.
// Pure C++ (no CUDA): the GPU context and the host-only simulator share this class.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "../../include/spm.h"

namespace spm {

enum Origin : uint8_t { kDemand = 0, kPrefetch = 1 };

struct Placement {
    int32_t expert;
    int32_t slot;
    int32_t wave;
    int32_t missed;   // 1: a host->HBM copy into `slot` is required
};

class SlotTable {
public:
    SlotTable(int n_layers, int n_experts, int slots, bool plain_lru)
        : L_(n_layers), n_(n_experts), S_(slots), plain_lru_(plain_lru) { reset(); }

    void reset() {
        tick_ = 0;
        step_ = 0;
        slot_expert_.assign(size_t(L_) * S_, -1);
        slot_tick_.assign(size_t(L_) * S_, 0);
        slot_origin_.assign(size_t(L_) * S_, kDemand);
        slot_used_.assign(size_t(L_) * S_, 0);
        expert_slot_.assign(size_t(L_) * n_, -1);
        events_.clear();
        stats_ = spm_stats{};
    }

    void reset_accounting() {
        events_.clear();
        stats_ = spm_stats{};
    }

    int layers() const { return L_; }
    int experts() const { return n_; }
    int slots() const { return S_; }
    int step() const { return step_; }
    void end_step() { ++step_; }
    void set_plain_lru(bool on) { plain_lru_ = on; }
    void set_event_cap(size_t cap) { event_cap_ = cap; }
    int slot_of(int layer, int e) const { return expert_slot_[size_t(layer) * n_ + e]; }
    int expert_in(int layer, int s) const { return slot_expert_[size_t(layer) * S_ + s]; }
    const std::vector<spm_event>& events() const { return events_; }
    spm_stats& stats() { return stats_; }

    // Resolve the demand of `layer`. `need` may hold duplicates and any order; it is
    // processed by ascending expert id: hits first (they keep their slots and become
    // most recently used), then misses, each into the LRU victim. When every slot is
    // taken by the current wave a new wave starts: the experts placed so far must be
    // computed before their slots are reused.
    void demand(int layer, const int32_t* need, int count, std::vector<Placement>& out, int* n_waves) {
        out.clear();
        mark_.assign(n_, 0);
        for (int i = 0; i < count; ++i) mark_[need[i]] = 1;
        ++tick_;
        int wave = 0;
        for (int e = 0; e < n_; ++e) {
            if (!mark_[e]) continue;
            int s = slot_of(layer, e);
            if (s < 0) continue;
            size_t k = size_t(layer) * S_ + s;
            bool first_use = slot_origin_[k] == kPrefetch && !slot_used_[k];
            log(layer, first_use ? SPM_EV_HIT_PREFETCHED : SPM_EV_HIT, e, s);
            stats_.hits++;
            stats_.hits_prefetched += first_use;
            slot_used_[k] = 1;
            slot_tick_[k] = tick_;
            out.push_back({e, s, 0, 0});
            mark_[e] = 0;
        }
        for (int e = 0; e < n_; ++e) {
            if (!mark_[e]) continue;
            int s = victim(layer);
            if (s < 0) {
                ++wave;
                log(layer, SPM_EV_WAVE, wave, -1);
                stats_.waves++;
                ++tick_;
                s = victim(layer);
            }
            install(layer, s, e, kDemand);
            log(layer, SPM_EV_MISS, e, s);
            stats_.misses++;
            out.push_back({e, s, wave, 1});
        }
        if (n_waves) *n_waves = wave + 1;
    }

    // Budgeted selection for pool `layer`: first min(budget, S) experts of `order` without a
    // slot; `protect` receives the resident experts the predicted-use touch will refresh.
    void plan(int layer, const int32_t* order, int n_ranked, int budget, bool protect_all,
              std::vector<int32_t>& sel, std::vector<int32_t>& protect) const {
        sel.clear();
        protect.clear();
        int limit = budget < S_ ? budget : S_;
        int last = -1;
        for (int pos = 0; pos < n_ranked && int(sel.size()) < limit; ++pos) {
            if (slot_of(layer, order[pos]) < 0) {
                sel.push_back(order[pos]);
                last = pos;
            }
        }
        if (plain_lru_) return;
        int upto = protect_all ? n_ranked : (sel.empty() ? 0 : last);
        for (int pos = 0; pos < upto; ++pos)
            if (slot_of(layer, order[pos]) >= 0) protect.push_back(order[pos]);
    }

    // Install `ids` (descending priority) into pool `layer`. out_slots[i] = slot, or -1 when
    // the request was not issued (already has a slot, dropped, or no unprotected slot left).
    int prefetch(int layer, const int32_t* ids, int count, const int32_t* protect, int n_protect,
                 int drop_modulo, int32_t* out_slots) {
        ++tick_;
        for (int i = 0; i < n_protect; ++i) {
            int s = slot_of(layer, protect[i]);
            if (s < 0) continue;
            slot_tick_[size_t(layer) * S_ + s] = tick_;
            log(layer, SPM_EV_TOUCH_PRED, protect[i], s);
            stats_.touches++;
        }
        int issued = 0;
        bool full = false;
        for (int i = 0; i < count; ++i) {
            out_slots[i] = -1;
            int e = ids[i];
            if (full || slot_of(layer, e) >= 0) continue;
            if (drop_modulo > 0 && (step_ + e) % drop_modulo == 0) {
                log(layer, SPM_EV_DROPPED, e, -1);
                stats_.dropped++;
                continue;
            }
            int s = victim(layer);
            if (s < 0) { full = true; continue; }
            install(layer, s, e, kPrefetch);
            log(layer, SPM_EV_PREFETCH, e, s);
            stats_.prefetch_issued++;
            out_slots[i] = s;
            ++issued;
        }
        return issued;
    }

    void plan_only(int layer, const int32_t* ids, int count) {
        for (int i = 0; i < count; ++i) {
            log(layer, SPM_EV_PLAN, ids[i], -1);
            stats_.planned++;
        }
    }

    // Structural invariants of the table: slot -> expert and expert -> slot are inverse maps, no
    // expert sits in two slots of a layer, no tick lies ahead of the global tick, flags are 0/1.
    // Returns -1 when they hold, else the index (layer * slots + slot, or L*S + layer*n + expert
    // for a dangling expert entry) of the first violation.
    long long check() const {
        for (int l = 0; l < L_; ++l) {
            for (int sl = 0; sl < S_; ++sl) {
                const size_t k = size_t(l) * S_ + sl;
                const int e = slot_expert_[k];
                if (e < -1 || e >= n_ || slot_tick_[k] > tick_ || slot_origin_[k] > 1 || slot_used_[k] > 1) return (long long)k;
                if (e >= 0 && expert_slot_[size_t(l) * n_ + e] != sl) return (long long)k;
            }
            for (int e = 0; e < n_; ++e) {
                const int sl = expert_slot_[size_t(l) * n_ + e];
                if (sl < -1 || sl >= S_ || (sl >= 0 && slot_expert_[size_t(l) * S_ + sl] != e))
                    return (long long)(size_t(L_) * S_ + size_t(l) * n_ + e);
            }
        }
        return -1;
    }

    // Checkpoint of the table as 64-bit words (no weights): {tick, step}, then per slot of every
    // layer {expert or -1, LRU tick, origin, used}. Accounting (statistics, event log) is not part of it.
    static size_t state_words(int n_layers, int slots) { return 2 + size_t(4) * n_layers * slots; }
    size_t state_words() const { return state_words(L_, S_); }
    void export_state(int64_t* out) const {
        out[0] = int64_t(tick_);
        out[1] = step_;
        for (size_t k = 0; k < size_t(L_) * S_; ++k) {
            out[2 + 4 * k] = slot_expert_[k];
            out[3 + 4 * k] = int64_t(slot_tick_[k]);
            out[4 + 4 * k] = slot_origin_[k];
            out[5 + 4 * k] = slot_used_[k];
        }
    }
    // Returns false (table untouched) when the words do not describe a valid table of this shape:
    // expert ids in range and at most once per layer, ticks not above the global tick, flags 0/1.
    bool import_state(const int64_t* in, size_t count) {
        if (count != state_words() || in[0] < 0 || in[1] < 0 || in[1] > INT32_MAX) return false;
        std::vector<int32_t> es(size_t(L_) * n_, -1);
        for (int l = 0; l < L_; ++l)
            for (int sl = 0; sl < S_; ++sl) {
                const size_t k = size_t(l) * S_ + sl;
                const int64_t e = in[2 + 4 * k], tk = in[3 + 4 * k], og = in[4 + 4 * k], us = in[5 + 4 * k];
                if (e < -1 || e >= n_ || tk < 0 || tk > in[0] || og < 0 || og > 1 || us < 0 || us > 1) return false;
                if (e >= 0) {
                    if (es[size_t(l) * n_ + e] >= 0) return false;
                    es[size_t(l) * n_ + e] = sl;
                }
            }
        tick_ = uint64_t(in[0]);
        step_ = int32_t(in[1]);
        for (size_t k = 0; k < size_t(L_) * S_; ++k) {
            slot_expert_[k] = int32_t(in[2 + 4 * k]);
            slot_tick_[k] = uint64_t(in[3 + 4 * k]);
            slot_origin_[k] = uint8_t(in[4 + 4 * k]);
            slot_used_[k] = uint8_t(in[5 + 4 * k]);
        }
        expert_slot_ = es;
        reset_accounting();
        return true;
    }

private:
    // The event log is bounded: once `event_cap_` records are held, further events are counted in
    // stats().events_dropped instead of being stored (statistics are unaffected).
    void log(int layer, int kind, int expert, int slot) {
        if (events_.size() >= event_cap_) { ++stats_.events_dropped; return; }
        events_.push_back({step_, layer, kind, expert, slot});
    }

    int victim(int layer) const {
        const size_t b = size_t(layer) * S_;
        for (int s = 0; s < S_; ++s)
            if (slot_expert_[b + s] < 0) return s;
        int best = -1;
        for (int s = 0; s < S_; ++s) {
            if (slot_tick_[b + s] >= tick_) continue;
            if (best < 0 || slot_tick_[b + s] < slot_tick_[b + best] ||
                (slot_tick_[b + s] == slot_tick_[b + best] && slot_expert_[b + s] < slot_expert_[b + best]))
                best = s;
        }
        return best;
    }

    void install(int layer, int s, int e, Origin origin) {
        size_t k = size_t(layer) * S_ + s;
        int v = slot_expert_[k];
        if (v >= 0) {
            bool wasted = slot_origin_[k] == kPrefetch && !slot_used_[k];
            log(layer, wasted ? SPM_EV_EVICT_WASTED : SPM_EV_EVICT, v, s);
            stats_.evictions++;
            stats_.wasted += wasted;
            expert_slot_[size_t(layer) * n_ + v] = -1;
        }
        slot_expert_[k] = e;
        slot_tick_[k] = tick_;
        slot_origin_[k] = origin;
        slot_used_[k] = origin == kDemand;
        expert_slot_[size_t(layer) * n_ + e] = s;
    }

    int L_, n_, S_;
    bool plain_lru_;
    uint64_t tick_ = 0;
    int32_t step_ = 0;
    std::vector<int32_t> slot_expert_, expert_slot_;
    std::vector<uint64_t> slot_tick_;
    std::vector<uint8_t> slot_origin_, slot_used_, mark_;
    std::vector<spm_event> events_;
    size_t event_cap_ = size_t(1) << 20;       // records kept between two resets of the accounting
    spm_stats stats_{};
};

}  // namespace spm
