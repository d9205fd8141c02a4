#include "host_ring.h"

namespace tutti {

HostRing::HostRing(uint32_t depth, uint32_t sgl_capacity)
    : depth_(depth), sgl_cap_(sgl_capacity), released_(depth, 0), slot_group_seq_(depth, 0) {}

uint32_t HostRing::live_sgl() const {
    uint32_t n = 0;
    for (const Group &g : groups_) n += g.sgl_count;
    return n;
}

const Group *HostRing::group_of(uint32_t iocb_idx) const {
    if (!is_live(iocb_idx)) return nullptr;
    uint32_t k = slot_group_seq_[iocb_idx & (depth_ - 1)] - seq_front_;
    if (k >= groups_.size()) return nullptr;
    return &groups_[k];
}

int HostRing::reserve(uint32_t n_iocb, uint32_t n_sgl, uint32_t *first_iocb, uint32_t *sgl_base) {
    if (n_iocb == 0 || n_iocb > depth_ || n_sgl > sgl_cap_) return -1;
    if (head_ - tail_ + n_iocb > depth_) return -3;
    // The live arena entries form a circular span from the oldest group's begin
    // to sgl_head_.  A range never wraps: if the tail end of the arena is too
    // short, the range starts again at entry 0.
    uint32_t begin;
    if (groups_.empty()) {
        begin = 0;
    } else {
        uint32_t tail = groups_.front().sgl_begin;
        bool wrapped = sgl_head_ < tail || (sgl_head_ == tail && live_sgl() > 0);
        if (!wrapped) {
            if (sgl_cap_ - sgl_head_ >= n_sgl) begin = sgl_head_;
            else if (tail >= n_sgl) begin = 0;
            else return -3;
        } else {
            if (tail - sgl_head_ >= n_sgl) begin = sgl_head_;
            else return -3;
        }
    }
    Group g{head_, n_iocb, begin, n_sgl, 0};
    uint32_t seq = seq_front_ + (uint32_t)groups_.size();
    for (uint32_t i = 0; i < n_iocb; ++i) {
        uint32_t slot = (head_ + i) & (depth_ - 1);
        released_[slot] = 0;
        slot_group_seq_[slot] = seq;
    }
    groups_.push_back(g);
    sgl_head_ = begin + n_sgl;
    *first_iocb = head_;
    *sgl_base = begin;
    head_ += n_iocb;
    return 0;
}

int HostRing::cancel_last(uint32_t first_iocb) {
    if (groups_.empty() || groups_.back().first_iocb != first_iocb || groups_.back().n_released)
        return -1;
    const Group g = groups_.back();
    groups_.pop_back();
    head_ = g.first_iocb;
    // the arena head goes back to where the previous group ends (or to 0 when none is left)
    sgl_head_ = groups_.empty() ? 0 : groups_.back().sgl_begin + groups_.back().sgl_count;
    return 0;
}

int HostRing::release(uint32_t iocb_idx) {
    if (!is_live(iocb_idx)) return -1;
    uint32_t slot = iocb_idx & (depth_ - 1);
    if (released_[slot]) return -1;
    uint32_t k = slot_group_seq_[slot] - seq_front_;
    if (k >= groups_.size()) return -1;
    released_[slot] = 1;
    groups_[k].n_released++;
    while (!groups_.empty() && groups_.front().n_released == groups_.front().n_iocb) {
        tail_ += groups_.front().n_iocb;
        groups_.pop_front();
        ++seq_front_;
    }
    if (groups_.empty()) sgl_head_ = 0;
    return 0;
}

}  // namespace tutti
