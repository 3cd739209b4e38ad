// Host-side delivery schedule of the sparse gradient messages and the staleness bookkeeping.
//
// Stands in for the asynchronous message queues between Model instances (Section 3.3): a message
// computed by replica i at step t reaches replica j at step t + delay(t, i, j), delay drawn from the
// counter-based generator, and a receiver works off what is due in (origin step, sender) order after
// its own local step (Section 3.1).  Also keeps the applied-gradient sets G_i as bit sets indexed by
// a global gradient sequence number, so that |G_i u G_j| - |G_i n G_j| is a popcount of an XOR.
#pragma once
#include <stdint.h>

#include <vector>

#include "../../include/tensair.h"

namespace tensair {

struct Due {
    uint64_t due, origin;
    uint32_t sender;
    uint32_t slot;        // sender * (max_delay + 1) + origin % (max_delay + 1)
    uint64_t staleness;
};

class Schedule {
public:
    Schedule(uint32_t W, uint32_t max_delay, uint64_t seed);
    uint32_t delay(uint64_t step, uint32_t sender, uint32_t receiver) const;
    uint32_t slot_of(uint32_t replica, uint64_t step) const { return replica * (D_ + 1) + (uint32_t)(step % (D_ + 1)); }
    // TENSAIR_EPENDING when the slot that (replica, step) would take still has recipients outstanding.
    int on_train(uint32_t replica, uint64_t step);
    // Pops what is due for `receiver`; see tensair_schedule_take_due.
    std::vector<Due> take_due(uint32_t receiver, uint64_t step, bool drain);
    uint64_t pending(uint32_t receiver) const { return inbox_[receiver].size(); }
    const std::vector<tensair_delivery>& log(uint32_t receiver) const { return log_[receiver]; }
    bool slot_busy(uint32_t slot) const { return slots_[slot].used && slots_[slot].outstanding; }
    bool slot_holds(uint32_t slot, uint64_t step) const { return slots_[slot].used && slots_[slot].step == step; }
    uint32_t W() const { return W_; }
    // The whole book-keeping (pending deliveries, slots, applied-gradient sets, delivery logs) as bytes, and back.
    // load() accepts only what a schedule of the same W, max_delay and seed saved; on failure nothing is changed.
    void save(std::vector<uint8_t>& out) const;
    bool load(const uint8_t* data, size_t bytes);

private:
    struct Bits {                      // bit set over gradient sequence numbers >= 64 * first_word
        uint64_t first_word = 0;
        std::vector<uint64_t> words;
        bool test_word_full(uint64_t w) const;
        uint64_t word(uint64_t w) const;
        void set(uint64_t bit);
    };
    struct Slot {
        bool used = false;
        uint64_t step = 0;
        uint32_t outstanding = 0;
        Bits snapshot;                 // G_sender when the gradient was computed
        uint64_t seq = 0;
    };
    struct Pending {
        uint64_t due, origin;
        uint32_t sender, slot;
    };
    void trim();
    uint64_t distance(const Bits& a, const Bits& b) const;

    uint32_t W_, D_;
    uint64_t seed_;
    uint64_t next_seq_ = 0;
    uint64_t floor_word_ = 0;          // every set holds all sequence numbers below 64 * floor_word_
    std::vector<Bits> G_;
    std::vector<Slot> slots_;
    std::vector<std::vector<Pending>> inbox_;
    std::vector<std::vector<tensair_delivery>> log_;
};

}  // namespace tensair
