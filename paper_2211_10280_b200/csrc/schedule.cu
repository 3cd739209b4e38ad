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

namespace {

struct Writer {
    std::vector<uint8_t>& out;
    void u64(uint64_t v) { for (int i = 0; i < 8; ++i) out.push_back((uint8_t)(v >> (8 * i))); }
    void words(const std::vector<uint64_t>& w) { u64(w.size()); for (uint64_t x : w) u64(x); }
};
struct Reader {
    const uint8_t* p;
    size_t left;
    bool ok = true;
    uint64_t u64() {
        if (left < 8) { ok = false; return 0; }
        uint64_t v = 0;
        for (int i = 0; i < 8; ++i) v |= (uint64_t)p[i] << (8 * i);
        p += 8; left -= 8;
        return v;
    }
    // a length read from the blob is believed only as far as the bytes that are left can back it
    uint64_t count(uint64_t bytes_each) {
        const uint64_t n = u64();
        if (bytes_each && n > left / bytes_each) { ok = false; return 0; }
        return n;
    }
    void words(std::vector<uint64_t>& w) {
        const uint64_t n = count(8);
        w.assign(ok ? n : 0, 0);
        for (uint64_t& x : w) x = u64();
    }
};
constexpr uint64_t kScheduleMagic = 0x3144454853524941ull;   // "AIRSHED1"

}  // namespace

void Schedule::save(std::vector<uint8_t>& out) const {
    Writer w{out};
    w.u64(kScheduleMagic); w.u64(W_); w.u64(D_); w.u64(seed_); w.u64(next_seq_); w.u64(floor_word_);
    for (const Bits& g : G_) { w.u64(g.first_word); w.words(g.words); }
    for (const Slot& s : slots_) {
        w.u64(s.used ? 1 : 0); w.u64(s.step); w.u64(s.outstanding); w.u64(s.seq);
        w.u64(s.snapshot.first_word); w.words(s.snapshot.words);
    }
    for (const std::vector<Pending>& in : inbox_) {
        w.u64(in.size());
        for (const Pending& p : in) { w.u64(p.due); w.u64(p.origin); w.u64(p.sender); w.u64(p.slot); }
    }
    for (const std::vector<tensair_delivery>& lg : log_) {
        w.u64(lg.size());
        for (const tensair_delivery& d : lg) { w.u64(d.origin_step); w.u64(d.sender); w.u64(d.due_step); w.u64(d.applied_at); w.u64(d.staleness); }
    }
}

bool Schedule::load(const uint8_t* data, size_t bytes) {
    Reader r{data, bytes};
    if (r.u64() != kScheduleMagic || r.u64() != W_ || r.u64() != D_ || r.u64() != seed_ || !r.ok) return false;
    Schedule t(W_, D_, seed_);
    t.next_seq_ = r.u64();
    t.floor_word_ = r.u64();
    for (Bits& g : t.G_) { g.first_word = r.u64(); r.words(g.words); }
    for (Slot& s : t.slots_) {
        s.used = r.u64() != 0; s.step = r.u64(); s.outstanding = (uint32_t)r.u64(); s.seq = r.u64();
        s.snapshot.first_word = r.u64(); r.words(s.snapshot.words);
        if (s.outstanding >= W_) r.ok = false;
    }
    for (std::vector<Pending>& in : t.inbox_) {
        const uint64_t n = r.count(32);
        for (uint64_t i = 0; i < n && r.ok; ++i) {
            Pending p{r.u64(), r.u64(), 0, 0};
            p.sender = (uint32_t)r.u64();
            p.slot = (uint32_t)r.u64();
            if (p.sender >= W_ || p.slot >= t.slots_.size()) r.ok = false;
            in.push_back(p);
        }
    }
    for (std::vector<tensair_delivery>& lg : t.log_) {
        const uint64_t n = r.count(40);
        for (uint64_t i = 0; i < n && r.ok; ++i) {
            tensair_delivery d;
            d.origin_step = r.u64(); d.sender = r.u64(); d.due_step = r.u64(); d.applied_at = r.u64(); d.staleness = r.u64();
            lg.push_back(d);
        }
    }
    if (!r.ok || r.left != 0) return false;
    *this = std::move(t);
    return true;
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

int tensair_schedule_save(const tensair_schedule* s, void* dst, uint64_t capacity, uint64_t* bytes) {
    if (!s || !bytes) return TENSAIR_EINVAL;
    std::vector<uint8_t> blob;
    s->impl.save(blob);
    *bytes = blob.size();
    if (!dst) return TENSAIR_OK;                    // size query
    if (capacity < blob.size()) return TENSAIR_ENOMEM;
    std::copy(blob.begin(), blob.end(), static_cast<uint8_t*>(dst));
    return TENSAIR_OK;
}

int tensair_schedule_load(tensair_schedule* s, const void* src, uint64_t bytes) {
    if (!s || !src) return TENSAIR_EINVAL;
    return s->impl.load(static_cast<const uint8_t*>(src), bytes) ? TENSAIR_OK : TENSAIR_EINVAL;
}

int tensair_schedule_pending(const tensair_schedule* s, uint32_t receiver, uint64_t* n) {
    if (!s || !n || receiver >= s->impl.W()) return TENSAIR_EINVAL;
    *n = s->impl.pending(receiver);
    return TENSAIR_OK;
}

}  // extern "C"
