// Host-side bookkeeping of the submission ring: which IOCB indices and which
// ranges of the SGL arena are reserved.  Pure host code (no CUDA), O(1) per call.
//
// IOCB indices are monotonically increasing 32-bit counters; index i uses ring
// slot i mod depth (depth is a power of two, so this survives counter wrap).  A
// "group" is what one build (or one tutti_ring_reserve) reserved: consecutive IOCB
// indices plus one contiguous range of SGL entries.  Groups are released in FIFO
// order once every IOCB in them has been polled — the analogue of consuming
// completion entries in io_uring (paper Section 3.2, steps 1-4).
#pragma once
#include <cstdint>
#include <deque>
#include <vector>

namespace tutti {

struct Group {
    uint32_t first_iocb;
    uint32_t n_iocb;
    uint32_t sgl_begin;
    uint32_t sgl_count;
    uint32_t n_released;
};

class HostRing {
public:
    HostRing(uint32_t depth, uint32_t sgl_capacity);

    // Reserve n_iocb consecutive indices and n_sgl contiguous arena entries.
    // 0 on success, -1 invalid (n_iocb == 0, more than the ring can ever hold),
    // -3 no room right now.
    int reserve(uint32_t n_iocb, uint32_t n_sgl, uint32_t *first_iocb, uint32_t *sgl_base);

    // Undo the most recent reserve() (its kernels could not be launched).  -1 if `first_iocb`
    // is not the start of the newest group.
    int cancel_last(uint32_t first_iocb);

    // Mark one IOCB as polled.  Releases whole groups from the front of the FIFO.
    // -1 if the index is not live or was released before.
    int release(uint32_t iocb_idx);

    bool is_live(uint32_t iocb_idx) const { return iocb_idx - tail_ < head_ - tail_; }
    const Group *group_of(uint32_t iocb_idx) const;

    uint32_t live_iocbs() const { return head_ - tail_; }
    uint32_t live_sgl() const;
    uint32_t depth() const { return depth_; }
    uint32_t sgl_capacity() const { return sgl_cap_; }

private:
    uint32_t depth_, sgl_cap_;
    uint32_t head_ = 0, tail_ = 0;          // IOCB index window [tail_, head_)
    uint32_t sgl_head_ = 0;                 // next free arena entry
    std::deque<Group> groups_;
    std::vector<uint8_t> released_;         // per slot
    std::vector<uint32_t> slot_group_seq_;  // per slot: sequence number of its group
    uint32_t seq_front_ = 0;                // sequence number of groups_.front()
};

}  // namespace tutti
