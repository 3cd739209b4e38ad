// Delivery schedule and staleness bookkeeping (host only; no GPU is touched).
#include "schedule.h"

#include <algorithm>

#include "philox.cuh"

namespace tensair {

uint64_t Schedule::Bits::word(uint64_t w) const {
    if (w < first_word) return ~0ULL;
    const uint64_t i = w - first_word;
    return i < words.size() ? words[i] : 0ULL;
}

void Schedule::Bits::set(uint64_t bit) {
    const uint64_t w = bit >> 6;
    if (w < first_word) return;
    const uint64_t i = w - first_word;
    if (i >= words.size()) words.resize(i + 1, 0ULL);
    words[i] |= 1ULL << (bit & 63);
}

Schedule::Schedule(uint32_t W, uint32_t max_delay, uint64_t seed)
    : W_(W), D_(max_delay), seed_(seed), G_(W), slots_((size_t)W * (max_delay + 1)), inbox_(W), log_(W) {}

uint32_t Schedule::delay(uint64_t step, uint32_t sender, uint32_t receiver) const {
    const Philox4 r = philox4x32_10(Philox4{(uint32_t)step, sender, receiver, kTagDelay}, (uint32_t)seed_,
                                    (uint32_t)(seed_ >> 32));
    return hi_product(r.x, D_ + 1);
}

uint64_t Schedule::distance(const Bits& a, const Bits& b) const {
    // symmetric difference; both sets hold everything below the floor
    uint64_t hi = std::max(a.first_word + a.words.size(), b.first_word + b.words.size());
    uint64_t n = 0;
    for (uint64_t w = floor_word_; w < hi; ++w) n += (uint64_t)__builtin_popcountll(a.word(w) ^ b.word(w));
    return n;
}

// Drops leading words that are full in every replica's set and in every snapshot still to be delivered.
void Schedule::trim() {
    for (;;) {
        const uint64_t w = floor_word_;
        if ((w + 1) * 64 > next_seq_) return;
        for (const Bits& g : G_) if (g.word(w) != ~0ULL) return;
        for (const Slot& s : slots_) if (s.used && s.outstanding && s.snapshot.word(w) != ~0ULL) return;
        ++floor_word_;
        for (Bits& g : G_) {
            if (g.first_word == w) {
                if (!g.words.empty()) g.words.erase(g.words.begin());
                g.first_word = w + 1;
            }
        }
    }
}

int Schedule::on_train(uint32_t replica, uint64_t step) {
    if (replica >= W_) return TENSAIR_EINVAL;
    const uint32_t si = slot_of(replica, step);
    Slot& s = slots_[si];
    if (s.used && s.outstanding) return TENSAIR_EPENDING;
    s.used = true;
    s.step = step;
    s.outstanding = W_ - 1;
    s.snapshot = G_[replica];            // G_i at the time the gradient is computed
    s.seq = next_seq_++;
    G_[replica].set(s.seq);              // local application, staleness 0
    for (uint32_t j = 0; j < W_; ++j)
        if (j != replica) inbox_[j].push_back(Pending{step + delay(step, replica, j), step, replica, si});
    if ((s.seq & 63) == 63) trim();
    return TENSAIR_OK;
}

std::vector<Due> Schedule::take_due(uint32_t receiver, uint64_t step, bool drain) {
    std::vector<Pending>& in = inbox_[receiver];
    std::vector<Pending> due, rest;
    for (const Pending& p : in) (drain || p.due <= step ? due : rest).push_back(p);
    std::sort(due.begin(), due.end(), [drain](const Pending& a, const Pending& b) {
        if (drain && a.due != b.due) return a.due < b.due;
        if (a.origin != b.origin) return a.origin < b.origin;
        return a.sender < b.sender;
    });
    in.swap(rest);
    std::vector<Due> out;
    out.reserve(due.size());
    for (const Pending& p : due) {
        Slot& s = slots_[p.slot];
        const uint64_t st = distance(s.snapshot, G_[receiver]);
        G_[receiver].set(s.seq);
        --s.outstanding;
        out.push_back(Due{p.due, p.origin, p.sender, p.slot, st});
        std::vector<tensair_delivery>& lg = log_[receiver];
        if (lg.size() >= (1u << 20)) lg.erase(lg.begin(), lg.begin() + (1u << 19));
        lg.push_back(tensair_delivery{p.origin, p.sender, p.due, drain ? p.due : step, st});
    }
    return out;
}

}  // namespace tensair

using tensair::Schedule;

struct tensair_schedule {
    Schedule impl;
    tensair_schedule(uint32_t W, uint32_t D, uint64_t seed) : impl(W, D, seed) {}
};

extern "C" {

uint32_t tensair_delay(uint64_t seed, uint32_t max_delay, uint64_t step, uint32_t sender, uint32_t receiver) {
    return Schedule(1, max_delay, seed).delay(step, sender, receiver);
}

int tensair_route(uint64_t seed, uint32_t W, uint32_t token, uint32_t* replica) {
    if (!replica || W == 0) return TENSAIR_EINVAL;
    const tensair::Philox4 r = tensair::philox4x32_10(tensair::Philox4{token, 0u, 0u, tensair::kTagRoute}, (uint32_t)seed, (uint32_t)(seed >> 32));
    *replica = (uint32_t)(((uint64_t)r.x * W) >> 32);
    return TENSAIR_OK;
}

void tensair_philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]) {
    const tensair::Philox4 r =
        tensair::philox4x32_10(tensair::Philox4{counter[0], counter[1], counter[2], counter[3]}, key[0], key[1]);
    out[0] = r.x; out[1] = r.y; out[2] = r.z; out[3] = r.w;
}

int tensair_schedule_create(uint32_t W, uint32_t max_delay, uint64_t seed, tensair_schedule** out) {
    if (!out || W < 1 || W > 256 || max_delay > 64) return TENSAIR_EINVAL;
    *out = new tensair_schedule(W, max_delay, seed);
    return TENSAIR_OK;
}

void tensair_schedule_destroy(tensair_schedule* s) { delete s; }

int tensair_schedule_on_train(tensair_schedule* s, uint32_t replica, uint64_t step) {
    if (!s) return TENSAIR_EINVAL;
    return s->impl.on_train(replica, step);
}

int tensair_schedule_take_due(tensair_schedule* s, uint32_t receiver, uint64_t step, int drain, uint64_t max_records,
                              tensair_delivery* out, uint64_t* n) {
    if (!s || receiver >= s->impl.W()) return TENSAIR_EINVAL;
    const std::vector<tensair::Due> due = s->impl.take_due(receiver, step, drain != 0);
    for (uint64_t i = 0; i < due.size() && i < max_records && out; ++i)
        out[i] = tensair_delivery{due[i].origin, due[i].sender, due[i].due, drain ? due[i].due : step, due[i].staleness};
    if (n) *n = due.size();
    return TENSAIR_OK;
}

int tensair_schedule_pending(const tensair_schedule* s, uint32_t receiver, uint64_t* n) {
    if (!s || !n || receiver >= s->impl.W()) return TENSAIR_EINVAL;
    *n = s->impl.pending(receiver);
    return TENSAIR_OK;
}

}  // extern "C"
