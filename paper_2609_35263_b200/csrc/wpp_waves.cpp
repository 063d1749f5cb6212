// Wave-budget planner and FCFS packing (Section 4.5): host code, integer arithmetic only.
// Every comparison of the wave estimate n(b) = max(W / b, N_{>b/2}) with a whole number k is done without
// division: n(b) >= k  <=>  W >= k * b  or  N >= k;   n(b) <= k  <=>  W <= k * b  and  N <= k.
#include <stdint.h>

#include <vector>

#include "../../include/wpp.h"

namespace {

struct Pieces {
    const int64_t* a;
    int32_t na;
    const int64_t* b;
    int32_t nb;
    int64_t total;   // W
    template <typename F>
    void each(F f) const {
        for (int32_t i = 0; i < na; ++i)
            if (a[i] > 0) f(a[i]);
        for (int32_t i = 0; i < nb; ++i)
            if (b[i] > 0) f(b[i]);
    }
};

bool valid_config(const wpp_wave_config* c) {
    if (!c || c->num_stages < 1 || c->fill_factor < 1 || c->block_size < 1 || c->max_lanes < 1) return false;
    const int64_t B = c->block_size;
    if (c->max_budget % B != 0 || c->min_budget % B != 0) return false;
    if (c->min_budget < B || c->min_budget > c->max_budget || c->max_budget > INT32_MAX) return false;
    return true;
}

// Eq. (design-budget)
std::vector<int64_t> make_ladder(const wpp_wave_config& c) {
    std::vector<int64_t> l(1, c.max_budget);
    while (l.back() > c.min_budget) {
        const int64_t half = l.back() / 2;
        const int64_t down = half - half % c.block_size;
        l.push_back(down > c.min_budget ? down : c.min_budget);
    }
    return l;
}

int64_t pieces_above_half(const Pieces& p, int64_t b) {
    int64_t n = 0;
    p.each([&](int64_t x) { n += (2 * x > b) ? 1 : 0; });
    return n;
}
bool waves_at_least(const Pieces& p, int64_t b, int64_t k) { return p.total >= k * b || pieces_above_half(p, b) >= k; }
bool waves_at_most(const Pieces& p, int64_t b, int64_t k) { return p.total <= k * b && pieces_above_half(p, b) <= k; }

// tokens in pieces that fit b_large whole but not b_small
int64_t newly_split(const Pieces& p, int64_t b_large, int64_t b_small) {
    int64_t t = 0;
    p.each([&](int64_t x) { t += (x > b_small && x <= b_large) ? x : 0; });
    return t;
}

}  // namespace

extern "C" int wpp_wave_ladder(const wpp_wave_config* cfg, int64_t* ladder_out, int32_t capacity, int32_t* count) {
    if (!valid_config(cfg) || !count || capacity < 0 || (capacity > 0 && !ladder_out)) return WPP_ERR_INVALID_ARG;
    const std::vector<int64_t> l = make_ladder(*cfg);
    for (int32_t i = 0; i < capacity && i < (int32_t)l.size(); ++i) ladder_out[i] = l[(size_t)i];
    *count = (int32_t)l.size();
    return WPP_OK;
}

extern "C" int wpp_plan_waves(const wpp_wave_config* cfg, wpp_wave_state* state, const int64_t* remaining,
                              int32_t num_requests, const int64_t* inflight, int32_t num_inflight, int32_t flags,
                              int32_t* chunk_lens, wpp_wave_info* info) {
    if (!valid_config(cfg) || !state || !info || num_requests < 0 || num_inflight < 0) return WPP_ERR_INVALID_ARG;
    if ((num_requests > 0 && (!remaining || !chunk_lens)) || (num_inflight > 0 && !inflight)) return WPP_ERR_INVALID_ARG;
    const std::vector<int64_t> ladder = make_ladder(*cfg);
    const int32_t L = (int32_t)ladder.size();
    if (state->cur < 0 || state->cur >= L || state->direction < -1 || state->direction > 1 || state->count < 0)
        return WPP_ERR_INVALID_ARG;
    Pieces p = {remaining, num_requests, inflight, num_inflight, 0};
    for (int32_t i = 0; i < num_requests; ++i) {
        if (remaining[i] < 0) return WPP_ERR_INVALID_ARG;
        p.total += remaining[i];
    }
    for (int32_t i = 0; i < num_inflight; ++i) {
        if (inflight[i] < 0) return WPP_ERR_INVALID_ARG;
        p.total += inflight[i];
    }
    const int64_t R = 2 * (int64_t)cfg->num_stages;
    const int64_t S = R + ((int64_t)cfg->fill_factor - 1) * cfg->num_stages;

    // ---- selection: walk down from M while the budget supplies fewer than S waves; a budget that supplies R
    //      waves is only left if the newly split pieces are at most an eighth of W
    int32_t target = 0;
    while (target + 1 < L && !waves_at_least(p, ladder[(size_t)target], S)) {
        if (waves_at_least(p, ladder[(size_t)target], R) &&
            8 * newly_split(p, ladder[(size_t)target], ladder[(size_t)target + 1]) > p.total)
            break;
        ++target;
    }

    // ---- persistence rules
    wpp_wave_state st = *state;
    if (target == st.cur) {
        st.direction = 0;
        st.count = 0;
    } else if (target < st.cur) {
        if (st.cur - target >= 2) {                      // burst: at once
            st.cur = target;
            st.direction = 0;
            st.count = 0;
        } else {
            st.count = (st.direction == -1) ? st.count + 1 : 1;
            st.direction = -1;
            if (st.count >= R / 2) {
                st.cur -= 1;
                st.direction = 0;
                st.count = 0;
            }
        }
    } else {
        st.count = (st.direction == 1) ? st.count + 1 : 1;
        st.direction = 1;
        if (st.count >= R && waves_at_most(p, ladder[(size_t)st.cur], S - 1)) {
            st.cur += 1;
            st.direction = 0;
            st.count = 0;
        }
    }
    st.reserved = 0;
    *state = st;
    const int64_t b = ladder[(size_t)st.cur];

    // ---- first come, first served
    int64_t space = b, tokens = 0;
    int32_t lanes = 0;
    bool open = true;
    const int64_t min_fragment2 = 2 * cfg->min_budget > b ? 2 * cfg->min_budget : b;     // 2 * max(b_min, b / 2)
    for (int32_t i = 0; i < num_requests; ++i) {
        chunk_lens[i] = 0;
        const int64_t r = remaining[i];
        if (!open || r == 0) continue;
        if (lanes == cfg->max_lanes || space == 0) {
            open = false;
            continue;
        }
        int64_t take = r;
        if (r > space) {
            if (2 * space < min_fragment2) {
                open = false;
                continue;
            }
            take = space;
        }
        chunk_lens[i] = (int32_t)take;
        space -= take;
        tokens += take;
        ++lanes;
    }

    info->budget = b;
    info->work = p.total;
    info->wave_tokens = tokens;
    info->target_index = target;
    info->budget_index = st.cur;
    info->lanes = lanes;
    info->defer = ((flags & WPP_WAVE_RING_BUSY) && (flags & WPP_WAVE_ADMISSION_PENDING) &&
                   !(flags & WPP_WAVE_ALREADY_DEFERRED) && lanes == 1 && 2 * tokens < b)
                      ? 1
                      : 0;
    return WPP_OK;
}
