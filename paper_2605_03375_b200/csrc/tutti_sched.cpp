// Slack-aware I/O scheduler (paper Section 3.3): a lookup table, filled offline, says
// for every (input length, prefix length) how long the next slack window of a layer is
// and how many SMs it leaves free; a second table says how long the read / write
// kernels take for a given number of IOCBs on a given number of SMs.  Before each
// layer the scheduler launches as many queued read IOCBs as fit the window — or, when
// nothing fits, the reads the layer cannot run without — and only then, if window is
// left, writes; writes that do not fit stay queued (reads and writes never share a
// window slot: they run back to back, never concurrently) and are flushed during decode.
// Pure host code: no CUDA call, no allocation after the tables are filled.
#include <algorithm>
#include <cstdint>
#include <deque>
#include <map>
#include <new>
#include <vector>

#include "../../include/tutti.h"

namespace {

struct SlackEntry {
    float us = 0.f;
    uint32_t sms = 0;
};

struct Curve {                       // kernel time against IOCB count, for one SM count
    std::vector<std::pair<uint32_t, float>> pts;   // sorted by n
    float at(uint32_t n) const {
        if (n == 0 || pts.empty()) return 0.f;
        if (pts.size() == 1) return pts[0].second * (float)n / (float)pts[0].first;
        if (n <= pts.front().first)
            return pts.front().second * (float)n / (float)pts.front().first;
        for (size_t i = 1; i < pts.size(); ++i) {
            if (n <= pts[i].first) {
                float f = (float)(n - pts[i - 1].first) / (float)(pts[i].first - pts[i - 1].first);
                return pts[i - 1].second + f * (pts[i].second - pts[i - 1].second);
            }
        }
        const auto &a = pts[pts.size() - 2], &b = pts.back();
        float slope = (b.second - a.second) / (float)(b.first - a.first);
        return b.second + slope * (float)(n - b.first);
    }
};

struct Pending {
    uint32_t layer, iocb;
};

}  // namespace

struct tutti_sched {
    uint32_t n_layers, step, ni, nj;
    std::vector<SlackEntry> slack;                 // [ni][nj]
    SlackEntry decode;
    std::map<uint32_t, Curve> io[2];               // opcode -> sm_count -> curve
    std::deque<Pending> reads, writes;             // FIFO; reads kept sorted by layer (stable)

    const Curve *curve(uint32_t op, uint32_t sms) const {
        const auto &m = io[op];
        if (m.empty()) return nullptr;
        // 0 means "all SMs" and is profiled under key 0; otherwise the largest profiled
        // SM count that does not exceed the budget, else the smallest one profiled
        auto it = m.find(sms);
        if (it != m.end()) return &it->second;
        const Curve *best = nullptr;
        for (const auto &kv : m)
            if (kv.first != 0 && kv.first <= sms) best = &kv.second;
        if (best) return best;
        for (const auto &kv : m)
            if (kv.first != 0) return &kv.second;
        return &m.begin()->second;
    }
    float io_time(uint32_t op, uint32_t sms, uint32_t n) const {
        const Curve *c = curve(op, sms);
        return c ? c->at(n) : 0.f;
    }
    // largest n <= limit whose kernel time fits the budget
    uint32_t max_fit(uint32_t op, uint32_t sms, float budget_us, uint32_t limit) const {
        if (!curve(op, sms)) return 0;
        uint32_t n = 0;
        while (n < limit && io_time(op, sms, n + 1) <= budget_us) ++n;
        return n;
    }
};

static void emit(tutti_launch_t *out, uint32_t max_out, uint32_t &n_out, uint32_t op, uint32_t layer,
                 uint32_t iocb, uint32_t sms) {
    if (n_out > 0) {
        tutti_launch_t &p = out[n_out - 1];
        if (p.opcode == op && p.sm_count == sms && p.first_iocb + p.n_iocb == iocb) {
            p.n_iocb++;
            return;
        }
    }
    if (n_out < max_out) {
        out[n_out].opcode = op;
        out[n_out].first_iocb = iocb;
        out[n_out].n_iocb = 1;
        out[n_out].sm_count = sms;
        out[n_out].layer = layer;
        out[n_out].est_us = 0.f;
    }
    ++n_out;
}

extern "C" {

int tutti_sched_create(uint32_t n_layers, uint32_t token_step, uint32_t max_input_tokens,
                       uint32_t max_prefix_tokens, tutti_sched_t **out) {
    if (!out || !n_layers || !token_step) return TUTTI_EINVAL;
    uint64_t ni = (uint64_t)max_input_tokens / token_step + 1, nj = (uint64_t)max_prefix_tokens / token_step + 1;
    if (ni * nj > (1ull << 26)) return TUTTI_EINVAL;
    tutti_sched *s = new (std::nothrow) tutti_sched();
    if (!s) return TUTTI_ENOMEM;
    s->n_layers = n_layers;
    s->step = token_step;
    s->ni = (uint32_t)ni;
    s->nj = (uint32_t)nj;
    s->slack.assign((size_t)(ni * nj), SlackEntry());
    *out = s;
    return TUTTI_OK;
}

int tutti_sched_destroy(tutti_sched_t *s) {
    if (!s) return TUTTI_EINVAL;
    delete s;
    return TUTTI_OK;
}

int tutti_sched_set_slack(tutti_sched_t *s, uint32_t l_input, uint32_t l_prefix, float slack_us,
                          uint32_t sm_budget) {
    if (!s || slack_us < 0.f) return TUTTI_EINVAL;
    uint32_t i = l_input / s->step, j = l_prefix / s->step;
    if (i >= s->ni || j >= s->nj) return TUTTI_EINVAL;
    s->slack[(size_t)i * s->nj + j] = SlackEntry{slack_us, sm_budget};
    return TUTTI_OK;
}

int tutti_sched_set_decode_slack(tutti_sched_t *s, float slack_us, uint32_t sm_budget) {
    if (!s || slack_us < 0.f) return TUTTI_EINVAL;
    s->decode = SlackEntry{slack_us, sm_budget};
    return TUTTI_OK;
}

int tutti_sched_set_io_time(tutti_sched_t *s, uint32_t opcode, uint32_t sm_count, uint32_t n_iocb,
                            float us) {
    if (!s || opcode > 1 || n_iocb == 0 || us < 0.f) return TUTTI_EINVAL;
    Curve &c = s->io[opcode][sm_count];
    auto it = std::lower_bound(c.pts.begin(), c.pts.end(), std::make_pair(n_iocb, -1.f));
    if (it != c.pts.end() && it->first == n_iocb) it->second = us;
    else c.pts.insert(it, std::make_pair(n_iocb, us));
    return TUTTI_OK;
}

int tutti_sched_enqueue(tutti_sched_t *s, uint32_t opcode, uint32_t layer, uint32_t first_iocb,
                        uint32_t n_iocb) {
    if (!s || opcode > 1 || layer >= s->n_layers) return TUTTI_EINVAL;
    for (uint32_t k = 0; k < n_iocb; ++k) {
        Pending p{layer, first_iocb + k};
        if (opcode == TUTTI_OP_READ) {
            // reads are served in layer order (the next layer's KV first), FIFO within a layer
            auto it = std::upper_bound(s->reads.begin(), s->reads.end(), p,
                                       [](const Pending &a, const Pending &b) { return a.layer < b.layer; });
            s->reads.insert(it, p);
        } else {
            s->writes.push_back(p);
        }
    }
    return TUTTI_OK;
}

int tutti_sched_pending(const tutti_sched_t *s, uint32_t *reads, uint32_t *writes) {
    if (!s) return TUTTI_EINVAL;
    if (reads) *reads = (uint32_t)s->reads.size();
    if (writes) *writes = (uint32_t)s->writes.size();
    return TUTTI_OK;
}

int tutti_sched_io_time(const tutti_sched_t *s, uint32_t opcode, uint32_t sm_count, uint32_t n_iocb,
                        float *us) {
    if (!s || opcode > 1 || !us) return TUTTI_EINVAL;
    *us = s->io_time(opcode, sm_count, n_iocb);
    return TUTTI_OK;
}

int tutti_sched_next(tutti_sched_t *s, uint32_t phase, uint32_t layer, uint32_t l_input,
                     uint32_t l_prefix, tutti_launch_t *out, uint32_t max_out, uint32_t *n_out) {
    if (!s || !n_out || (max_out && !out) || phase > TUTTI_PHASE_DECODE) return TUTTI_EINVAL;
    if (phase == TUTTI_PHASE_PREFILL && layer >= s->n_layers) return TUTTI_EINVAL;
    uint32_t n = 0;
    SlackEntry w = s->decode;
    if (phase == TUTTI_PHASE_PREFILL) {
        uint32_t i = std::min(l_input / s->step, s->ni - 1), j = std::min(l_prefix / s->step, s->nj - 1);
        w = s->slack[(size_t)i * s->nj + j];
    }
    // decide first, consume the queues only when the caller's array can hold the answer
    uint32_t take_r = 0, take_w = 0;
    float t_r = 0.f, t_w = 0.f, left = w.us;
    if (phase == TUTTI_PHASE_PREFILL) {
        // reads first: as many as the window holds, but never fewer than the layer needs
        uint32_t required = 0;
        for (const Pending &p : s->reads)
            if (p.layer <= layer) ++required;
        uint32_t fit = (w.us > 0.f) ? s->max_fit(TUTTI_OP_READ, w.sms, w.us, (uint32_t)s->reads.size()) : 0;
        take_r = std::max(fit, required);
        t_r = s->io_time(TUTTI_OP_READ, w.sms, take_r);
        left = (take_r > fit) ? 0.f : w.us - t_r;     // forced reads used the window up
    }
    // writes only with window left, oldest first
    if (left > 0.f && !s->writes.empty()) {
        take_w = s->max_fit(TUTTI_OP_WRITE, w.sms, left, (uint32_t)s->writes.size());
        t_w = s->io_time(TUTTI_OP_WRITE, w.sms, take_w);
    }
    uint32_t need = 0;
    for (uint32_t k = 0; k < take_r; ++k)
        if (k == 0 || s->reads[k].iocb != s->reads[k - 1].iocb + 1) ++need;
    for (uint32_t k = 0; k < take_w; ++k)
        if (k == 0 || s->writes[k].iocb != s->writes[k - 1].iocb + 1) ++need;
    if (need > max_out) {
        *n_out = need;
        return TUTTI_EAGAIN;
    }
    uint32_t first_out = n;
    for (uint32_t k = 0; k < take_r; ++k) {
        Pending p = s->reads.front();
        s->reads.pop_front();
        emit(out, max_out, n, TUTTI_OP_READ, p.layer, p.iocb, w.sms);
    }
    if (take_r) out[first_out].est_us = t_r;
    first_out = n;
    for (uint32_t k = 0; k < take_w; ++k) {
        Pending p = s->writes.front();
        s->writes.pop_front();
        emit(out, max_out, n, TUTTI_OP_WRITE, p.layer, p.iocb, w.sms);
    }
    if (take_w) out[first_out].est_us = t_w;
    *n_out = n;
    return TUTTI_OK;
}

}  // extern "C"
