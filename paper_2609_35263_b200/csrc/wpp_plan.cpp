// Host side of the library that needs no CUDA: argument checks, the work split (wpp_plan_tiles)
// and the optional aliasing check (wpp_validate_batch).  Integer arithmetic only.
#include <algorithm>
#include <cstring>
#include <queue>
#include <unordered_map>
#include <vector>

#include "../../include/wpp.h"
#include "wpp_host.h"
#include "wpp_plan_format.h"

const char* wpp_status_string(int s) {
    switch (s) {
        case WPP_OK: return "WPP_OK";
        case WPP_ERR_INVALID_ARG: return "WPP_ERR_INVALID_ARG";
        case WPP_ERR_UNSUPPORTED: return "WPP_ERR_UNSUPPORTED";
        case WPP_ERR_BOUNDS: return "WPP_ERR_BOUNDS";
        case WPP_ERR_POSITION_MISMATCH: return "WPP_ERR_POSITION_MISMATCH";
        case WPP_ERR_WORKSPACE_TOO_SMALL: return "WPP_ERR_WORKSPACE_TOO_SMALL";
        case WPP_ERR_PLAN_MISMATCH: return "WPP_ERR_PLAN_MISMATCH";
        case WPP_ERR_CUDA: return "WPP_ERR_CUDA";
        case WPP_ERR_TIMEOUT: return "WPP_ERR_TIMEOUT";
        case WPP_ERR_ALIASED_APPEND: return "WPP_ERR_ALIASED_APPEND";
        default: return "WPP_ERR_UNKNOWN";
    }
}

// Fill in default strides and check what the host can check about a description.
int wpp_resolve_desc(const wpp_batch_desc* in, wpp_batch_desc* d) {
    if (!in) return WPP_ERR_INVALID_ARG;
    *d = *in;
    if (d->num_requests < 0 || d->num_q_heads <= 0 || d->num_kv_heads <= 0 || d->max_blocks_per_req < 0 ||
        d->num_pages < 0 || d->head_dim <= 0 || d->page_size <= 0 || !(d->sm_scale >= 0.0f))
        return WPP_ERR_INVALID_ARG;
    if (d->dtype != WPP_BF16) return WPP_ERR_UNSUPPORTED;
    if (d->head_dim != 64 && d->head_dim != 128) return WPP_ERR_UNSUPPORTED;
    if (d->page_size != 16 && d->page_size != 32 && d->page_size != 64 && d->page_size != 128)
        return WPP_ERR_UNSUPPORTED;
    if (d->num_q_heads % d->num_kv_heads != 0) return WPP_ERR_UNSUPPORTED;
    const int64_t dd = d->head_dim;
    if (!d->kv_token_stride) d->kv_token_stride = dd;
    if (!d->kv_head_stride) d->kv_head_stride = d->kv_token_stride * d->page_size;
    if (!d->kv_page_stride) d->kv_page_stride = d->kv_head_stride * d->num_kv_heads;
    if (!d->q_head_stride) d->q_head_stride = dd;
    if (!d->q_token_stride) d->q_token_stride = d->q_head_stride * d->num_q_heads;
    if (!d->kvnew_head_stride) d->kvnew_head_stride = dd;
    if (!d->kvnew_token_stride) d->kvnew_token_stride = d->kvnew_head_stride * d->num_kv_heads;
    if (!d->o_head_stride) d->o_head_stride = dd;
    if (!d->o_token_stride) d->o_token_stride = d->o_head_stride * d->num_q_heads;
    const int64_t strides[] = {d->kv_page_stride, d->kv_head_stride, d->kv_token_stride, d->q_token_stride,
                               d->q_head_stride, d->kvnew_token_stride, d->kvnew_head_stride,
                               d->o_token_stride, d->o_head_stride};
    for (int64_t s : strides)
        if (s < dd || (s % 8) != 0) return WPP_ERR_INVALID_ARG;  // 8 bf16 = 16 bytes
    return WPP_OK;
}

static uint64_t fnv1a(uint64_t h, const void* p, size_t n) {
    const unsigned char* b = static_cast<const unsigned char*>(p);
    for (size_t i = 0; i < n; ++i) { h ^= b[i]; h *= 0x100000001b3ull; }
    return h;
}

// Hash of everything a plan depends on except the lengths.  Those travel inside the plan (row offsets and a copy
// of prefix_lens); the kernels compare them with the device arrays they are launched with and refuse a request
// whose span differs (WPP_ERR_PLAN_MISMATCH in the status word).
uint64_t wpp_desc_hash(const wpp_batch_desc* d) {
    uint64_t h = 0xcbf29ce484222325ull;
    const int32_t ints[] = {d->num_requests, d->num_q_heads, d->num_kv_heads, d->head_dim, d->page_size,
                            d->max_blocks_per_req, d->num_pages, d->dtype};
    h = fnv1a(h, ints, sizeof(ints));
    const int64_t strides[] = {d->kv_page_stride, d->kv_head_stride, d->kv_token_stride, d->q_token_stride,
                               d->q_head_stride, d->kvnew_token_stride, d->kvnew_head_stride,
                               d->o_token_stride, d->o_head_stride};
    return fnv1a(h, strides, sizeof(strides));
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The model behind the automatic cut of the last round's tiles; costs in 128 x 128 key steps of one half (0.74 us at
// the tensor rate): a tile's start and end, what a part adds (it writes fp32 partials), the combine pass.
constexpr int kTailSplitMaxRounds = 16, kTailSplitMaxParts = 4, kTailSplitMinSteps = 8, kTailSplitMinGainPct = 10;
constexpr int64_t kTileFixedCost = 3, kPartExtraCost = 2, kCombineCost = 20;

static int resolve_opts(const wpp_ctx* ctx, const wpp_plan_opts* in, wpp_plan_opts* o) {
    wpp_plan_opts z = {0, 0, 0, 0, 0, 0};
    *o = in ? *in : z;
    if (!o->tile_m) o->tile_m = WPP_DEFAULT_TILE_M;
    if (!o->tile_n) o->tile_n = WPP_TILE_N;
    if (!o->max_ctas) o->max_ctas = ctx ? wpp_ctx_sm_count(ctx) : 148;
    if (o->tile_m != 128 && o->tile_m != 256) return WPP_ERR_UNSUPPORTED;
    if (o->tile_m > WPP_MAX_TILE_M) return WPP_ERR_UNSUPPORTED;
    if (o->tile_n != WPP_TILE_N) return WPP_ERR_UNSUPPORTED;
    if (o->force_kv_splits < 0 || o->force_kv_splits > 64 || o->max_ctas < 1 || o->max_ctas > 4096 ||
        o->order < 0 || o->order > 1 || o->shape < 0 || o->shape > 2)
        return WPP_ERR_INVALID_ARG;
    return WPP_OK;
}

static size_t plan_bytes_bound(const wpp_batch_desc* d, const wpp_plan_opts* o, int64_t T) {
    const int64_t q_tiles = T / WPP_HALF_M + d->num_requests;   // worst case: the planner falls back to 128-row tiles
    const int64_t base = q_tiles * d->num_q_heads;
    // automatic cuts add at most max_ctas parts (few tiles) or kTailSplitMaxParts per tile of one round (tail)
    const int64_t units = o->force_kv_splits >= 2 ? base * o->force_kv_splits : base + kTailSplitMaxParts * (int64_t)o->max_ctas;
    size_t n = sizeof(WppPlanHeader);
    n += 2 * align_up(sizeof(int32_t) * (size_t)(d->num_requests + 1), 16);   // row offsets, prefix copy
    n += align_up(sizeof(int32_t) * (size_t)(o->max_ctas + 1), 16);
    n += sizeof(WppUnit) * (size_t)units;
    n += sizeof(WppCombine) * (size_t)base * 2;
    return align_up(n, 256);
}

size_t wpp_plan_bytes(const wpp_ctx* ctx, const wpp_batch_desc* desc, int64_t total_new_tokens,
                      const wpp_plan_opts* opts_or_null) {
    wpp_batch_desc d;
    wpp_plan_opts o;
    if (wpp_resolve_desc(desc, &d) != WPP_OK || total_new_tokens < 0) return 0;
    if (resolve_opts(ctx, opts_or_null, &o) != WPP_OK) return 0;
    return plan_bytes_bound(&d, &o, total_new_tokens);
}

int wpp_plan_tiles(const wpp_ctx* ctx, const wpp_batch_desc* desc, const int32_t* prefix_lens,
                   const int32_t* chunk_lens, const int32_t* cached_lens, const wpp_plan_opts* opts_in,
                   void* plan_host, size_t plan_host_bytes, wpp_plan_info* info) {
    wpp_batch_desc d;
    wpp_plan_opts o;
    int rc = wpp_resolve_desc(desc, &d);
    if (rc != WPP_OK) return rc;
    rc = resolve_opts(ctx, opts_in, &o);
    if (rc != WPP_OK) return rc;
    const bool auto_tile_m = !(opts_in && opts_in->tile_m);
    const int R = d.num_requests;
    if (!plan_host || !info || (R > 0 && (!prefix_lens || !chunk_lens))) return WPP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(plan_host) & 15) != 0) return WPP_ERR_INVALID_ARG;
    const int B = d.page_size, Hq = d.num_q_heads;

    int64_t T = 0, pairs = 0;
    for (int i = 0; i < R; ++i) {
        const int64_t P = prefix_lens[i], C = chunk_lens[i];
        if (P < 0 || C < 0) return WPP_ERR_INVALID_ARG;
        if (P + C > (int64_t)0x7fffffff - 4 * WPP_TILE_N) return WPP_ERR_INVALID_ARG;
        if (cached_lens && cached_lens[i] != prefix_lens[i]) return WPP_ERR_POSITION_MISMATCH;
        if (C > 0 && (P + C + B - 1) / B > d.max_blocks_per_req) return WPP_ERR_BOUNDS;
        T += C;
        pairs += C * P + C * (C + 1) / 2;
    }
    if (T > 0x7fffffff) return WPP_ERR_INVALID_ARG;
    if (plan_host_bytes < plan_bytes_bound(&d, &o, T)) return WPP_ERR_PLAN_MISMATCH;

    // ---- row blocks of every request.  A tile is a row block times the heads it takes (one head, or 2..16 heads of
    //      one KV group for short blocks), so everything but the heads is worked out once per row block.
    struct RowBlock {
        int32_t request, r0, rows[2], row0_b, head_b, pack, per_tile, steps, end[2];   // head_b: second half's first head
                                                                                        // minus the first's; end[h]: key steps half h can see
        int32_t cost() const { return end[0] + end[1]; }                       // 128x128 steps over both halves
    };
    const int G = Hq / d.num_kv_heads;
    auto steps_for = [](int64_t last_visible_plus1) { return (int32_t)((last_visible_plus1 + WPP_TILE_N - 1) / WPP_TILE_N); };
    std::vector<RowBlock> rbs;
    std::vector<int32_t> rb_first((size_t)R + 1);
    auto build_rows = [&](int tile_m) -> int64_t {
        rbs.clear();
        int64_t n_tiles = 0;
        for (int i = 0; i < R; ++i) {
            rb_first[(size_t)i] = (int32_t)rbs.size();
            const int64_t P = prefix_lens[i], C = chunk_lens[i];
            for (int64_t r0 = 0; r0 < C; r0 += tile_m) {
                const int32_t rows = (int32_t)std::min<int64_t>(tile_m, C - r0);
                RowBlock rb;
                rb.request = i;
                rb.r0 = (int32_t)r0;
                rb.steps = steps_for(P + r0 + rows);
                if (rows <= WPP_HALF_M) {
                    // short block: each half takes `pack` heads of one KV group over the same rows (pack is the
                    // largest power of two that divides the group size and leaves 128/pack >= rows tensor rows
                    // per head); with 256-row tiles the second half takes the next heads of the group
                    int pack = 1;
                    while (pack < 8 && G % (2 * pack) == 0 && WPP_HALF_M / (2 * pack) >= rows) pack *= 2;
                    rb.pack = pack;
                    rb.per_tile = (tile_m == 256 && G % (2 * pack) == 0) ? 2 * pack : pack;
                    rb.rows[0] = rows;
                    rb.rows[1] = rb.per_tile == 2 * pack ? rows : 0;
                    rb.row0_b = (int32_t)r0;
                    rb.head_b = pack;
                    rb.end[0] = rb.steps;
                    rb.end[1] = rb.rows[1] > 0 ? rb.steps : 0;
                } else {
                    rb.pack = 1;
                    rb.per_tile = 1;
                    rb.rows[0] = WPP_HALF_M;
                    rb.rows[1] = rows - WPP_HALF_M;
                    rb.row0_b = (int32_t)r0 + WPP_HALF_M;
                    rb.head_b = 0;
                    rb.end[0] = steps_for(P + r0 + WPP_HALF_M);
                    rb.end[1] = rb.steps;
                }
                n_tiles += Hq / rb.per_tile;
                rbs.push_back(rb);
            }
        }
        rb_first[(size_t)R] = (int32_t)rbs.size();
        return n_tiles;
    };
    int TM = o.tile_m;
    int64_t n_base = build_rows(TM);
    if (auto_tile_m && TM == 256 && n_base < o.max_ctas) {   // few tiles: prefer more, smaller ones
        TM = 128;
        n_base = build_rows(TM);
    }
    if (n_base > 0x3fffffff) return WPP_ERR_INVALID_ARG;
    // cost of key steps [a, b) of a tile = 128x128 steps over its halves, each cut at its own causal end
    auto cost_of = [](const RowBlock& t, int32_t a, int32_t b) -> int32_t {
        return std::max(0, std::min(b, t.end[0]) - a) + std::max(0, std::min(b, t.end[1]) - a);
    };

    // ---- order of execution.  The persistent CTAs take tiles in this order at run time (a counter in the
    //      workspace), so tiles adjacent in the order run at the same time on different SMs.
    //      order 0 (default), "stream order": KV head major, then requests (longest first), then row blocks and
    //      heads.  All tiles that read one (request, KV head) stream start together and walk its pages in step,
    //      so a page comes from DRAM once and is then hit in L2 by the other tiles; a prefix shared by many
    //      requests stays L2-resident while its KV head is being worked on.
    //      order 1: longest tile first (best balance, no regard for which tiles run together).
    struct Tile { int32_t rb, head; };          // row block and first head
    std::vector<Tile> tiles;
    tiles.reserve((size_t)n_base);
    if (o.order == 1) {
        for (int32_t k = 0; k < (int32_t)rbs.size(); ++k)
            for (int h = 0; h < Hq; h += rbs[(size_t)k].per_tile) tiles.push_back({k, h});
        std::stable_sort(tiles.begin(), tiles.end(),
                         [&](const Tile& a, const Tile& b) { return rbs[(size_t)a.rb].cost() > rbs[(size_t)b.rb].cost(); });
    } else {
        std::vector<int64_t> req_cost((size_t)std::max(R, 1), 0);
        for (const RowBlock& rb : rbs) req_cost[(size_t)rb.request] += (int64_t)rb.cost() * (Hq / rb.per_tile);
        std::vector<int32_t> by_cost((size_t)R);
        for (int i = 0; i < R; ++i) by_cost[(size_t)i] = i;
        std::stable_sort(by_cost.begin(), by_cost.end(),
                         [&](int32_t a, int32_t b) { return req_cost[(size_t)a] > req_cost[(size_t)b]; });
        for (int kvh = 0; kvh < d.num_kv_heads; ++kvh)
            for (int rank = 0; rank < R; ++rank) {
                const int i = by_cost[(size_t)rank];
                for (int32_t k = rb_first[(size_t)i]; k < rb_first[(size_t)i + 1]; ++k)
                    for (int h = kvh * G; h < (kvh + 1) * G; h += rbs[(size_t)k].per_tile) tiles.push_back({k, h});
            }
    }

    // ---- split decision: into how many key ranges each tile is cut (1 = not at all)
    int32_t few_want = 0;          // fewer tiles than CTAs: every tile is cut so that all CTAs have work (>= 2 steps per part)
    int64_t tail = 0;              // tiles of a partly filled last round ...
    int32_t tail_parts = 1;        // ... and the number of key ranges each of them is cut into
    if (o.force_kv_splits == 0 && n_base > 0 && n_base < o.max_ctas) {
        few_want = (int32_t)((o.max_ctas + n_base - 1) / n_base);
    } else if (o.force_kv_splits == 0 && n_base % o.max_ctas != 0 && n_base < kTailSplitMaxRounds * (int64_t)o.max_ctas) {
        // A few rounds of long tiles: the last, partly filled round leaves CTAs idle for a whole tile.  Cutting the
        // tiles of that round into p key ranges each fills it.  The candidates are compared on a model of the run
        // (tiles handed out in order to the CTA that is free first; a tile costs its key steps plus a fixed start
        // and end, a part a little more, the combine pass a constant).  The model flatters the cut: SMs of a partly
        // filled round run faster than those of a full one (more of the power budget and of L2 each), so that a
        // modelled gain of 12 % measured as 5-6 % and one of 8 % as a small loss; a cut is made from 10 % up.
        const int64_t n_tail = n_base % o.max_ctas;
        int32_t min_steps = 0x7fffffff;
        for (int64_t k = n_base - n_tail; k < n_base; ++k) min_steps = std::min(min_steps, rbs[(size_t)tiles[(size_t)k].rb].steps);
        if (min_steps >= 2 * kTailSplitMinSteps) {
            using MinHeap = std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>>;
            MinHeap before_tail;                 // when each CTA is free once the full rounds have been handed out
            for (int c = 0; c < o.max_ctas; ++c) before_tail.push(0);
            int64_t end_before = 0;
            for (int64_t k = 0; k < n_base - n_tail; ++k) {
                const int64_t done = before_tail.top() + rbs[(size_t)tiles[(size_t)k].rb].cost() + kTileFixedCost;
                before_tail.pop();
                before_tail.push(done);
                end_before = std::max(end_before, done);
            }
            auto makespan = [&](int32_t p) -> int64_t {
                MinHeap free_at = before_tail;
                int64_t end = end_before;
                for (int64_t k = n_base - n_tail; k < n_base; ++k) {
                    const RowBlock& t = rbs[(size_t)tiles[(size_t)k].rb];
                    for (int32_t q = 0; q < p; ++q) {
                        const int32_t a = (int32_t)((int64_t)t.steps * q / p), b = (int32_t)((int64_t)t.steps * (q + 1) / p);
                        const int64_t done = free_at.top() + cost_of(t, a, b) + kTileFixedCost + (p > 1 ? kPartExtraCost : 0);
                        free_at.pop();
                        free_at.push(done);
                        end = std::max(end, done);
                    }
                }
                return end + (p > 1 ? kCombineCost : 0);
            };
            const int64_t whole = makespan(1);
            int64_t best = whole;
            for (int32_t p = 2; p <= kTailSplitMaxParts && min_steps >= p * kTailSplitMinSteps; ++p) {
                const int64_t m = makespan(p);
                if (m < best) { best = m; tail_parts = p; }
            }
            if (tail_parts > 1 && best * 100 <= whole * (100 - kTailSplitMinGainPct)) tail = n_tail;
            else tail_parts = 1;
        }
    }

    // ---- the plan: header, row offsets, the spans the plan is made for, units, combine records
    WppPlanHeader hd;
    std::memset(&hd, 0, sizeof(hd));
    size_t off = sizeof(WppPlanHeader);
    hd.off_q_offsets = (uint32_t)off;
    off += align_up(sizeof(int32_t) * (size_t)(R + 1), 16);
    hd.off_prefix = (uint32_t)off;
    off += align_up(sizeof(int32_t) * (size_t)(R + 1), 16);
    hd.off_units = (uint32_t)off;
    char* p = static_cast<char*>(plan_host);
    std::memset(p, 0, off);
    const int64_t unit_cap = ((int64_t)plan_host_bytes - (int64_t)off) / (int64_t)sizeof(WppUnit);
    WppUnit* us = reinterpret_cast<WppUnit*>(p + hd.off_units);
    std::vector<WppCombine> combines;
    int32_t slots = 0;
    int64_t n_units = 0, key_steps = 0, n_split_units = 0, nonempty_halves = 0;
    for (int64_t k = 0; k < n_base; ++k) {
        const RowBlock& t = rbs[(size_t)tiles[(size_t)k].rb];
        const int32_t h = tiles[(size_t)k].head;
        int32_t parts = 1;
        if (o.force_kv_splits >= 2) parts = std::max(1, std::min(o.force_kv_splits, t.steps));
        else if (few_want > 1) parts = std::max(1, std::min(few_want, t.steps / 2));
        else if (k >= n_base - tail) parts = tail_parts;
        if (n_units + parts > unit_cap) return WPP_ERR_PLAN_MISMATCH;
        WppUnit u;
        u.request = t.request;
        u.row0[0] = t.r0; u.row0[1] = t.row0_b;
        u.rows[0] = t.rows[0]; u.rows[1] = t.rows[1];
        u.head[0] = h; u.head[1] = h + t.head_b;
        u.pack = t.pack;
        nonempty_halves += (int64_t)parts * ((t.rows[0] > 0) + (t.rows[1] > 0));
        if (parts == 1) {
            u.kv_begin = 0; u.kv_end = t.steps; u.split_slot = -1; u.cost = t.cost();
            us[n_units++] = u;
            key_steps += u.cost;
        } else {
            for (int hf = 0; hf < 2; ++hf)
                for (int kk = 0; kk < t.pack && t.rows[hf] > 0; ++kk)
                    combines.push_back({t.request, u.row0[hf], t.rows[hf], u.head[hf] + kk, slots, parts, hf,
                                        kk * (WPP_HALF_M / t.pack)});
            for (int32_t q = 0; q < parts; ++q) {
                u.kv_begin = (int32_t)((int64_t)t.steps * q / parts);
                u.kv_end = (int32_t)((int64_t)t.steps * (q + 1) / parts);
                u.split_slot = slots + q;
                u.cost = cost_of(t, u.kv_begin, u.kv_end);
                us[n_units++] = u;
                key_steps += u.cost;
                ++n_split_units;
            }
            slots += parts;
        }
    }
    if (n_units > 0x3fffffff) return WPP_ERR_INVALID_ARG;
    // ---- kernel shape: short tiles (few key steps per half) go to the small CTAs, two per SM, where the start and end of
    //      one tile hide under the other CTA's steps; long tiles to the SM-wide CTA whose two halves overlap each other
    int shape = o.shape;
    if (shape == 0) shape = (key_steps <= WPP_SMALL_SHAPE_MAX_STEPS * nonempty_halves) ? 2 : 1;
    const int num_ctas = shape == 2 ? (int)std::max<int64_t>(1, std::min<int64_t>(2 * (int64_t)o.max_ctas, 2 * n_units))
                                    : (int)std::max<int64_t>(1, std::min<int64_t>(o.max_ctas, n_units));
    off += sizeof(WppUnit) * (size_t)n_units;
    hd.off_combine = (uint32_t)off;
    off += sizeof(WppCombine) * combines.size();
    hd.plan_bytes = align_up(off, 16);
    if (hd.plan_bytes > plan_host_bytes) return WPP_ERR_PLAN_MISMATCH;
    if (!combines.empty())
        std::memcpy(p + hd.off_combine, combines.data(), sizeof(WppCombine) * combines.size());
    std::memset(p + off, 0, hd.plan_bytes - off);

    hd.magic = WPP_PLAN_MAGIC;
    hd.version = WPP_PLAN_VERSION;
    hd.desc_hash = wpp_desc_hash(&d);
    hd.num_requests = R;
    hd.num_ctas = num_ctas;
    hd.num_units = (int32_t)n_units;
    hd.num_combine = (int32_t)combines.size();
    hd.num_split_slots = slots;
    hd.tile_m = TM;
    hd.tile_n = WPP_TILE_N;
    hd.head_dim = d.head_dim;
    hd.shape = shape;
    hd.nonempty_halves = (int32_t)std::min<int64_t>(nonempty_halves, 0x7fffffff);
    hd.total_new_tokens = T;
    hd.key_steps = key_steps;
    hd.flops = 4 * (int64_t)d.head_dim * Hq * pairs;
    hd.workspace_bytes = WPP_WS_HEADER_BYTES + align_up((size_t)slots * 2 * WPP_HALF_M * (d.head_dim + 1) * sizeof(float), 256);
    std::memcpy(p, &hd, sizeof(hd));
    int32_t* qo = reinterpret_cast<int32_t*>(p + hd.off_q_offsets);
    qo[0] = 0;
    for (int i = 0; i < R; ++i) qo[i + 1] = qo[i] + chunk_lens[i];
    int32_t* pp = reinterpret_cast<int32_t*>(p + hd.off_prefix);
    for (int i = 0; i < R; ++i) pp[i] = prefix_lens[i];

    info->num_tiles = n_units;
    info->num_split_tiles = n_split_units;
    info->num_combine_tiles = (int64_t)combines.size();
    info->num_ctas = num_ctas;
    info->total_new_tokens = T;
    info->key_steps = key_steps;
    info->flops = hd.flops;
    info->shape = shape;
    info->workspace_bytes = hd.workspace_bytes;
    info->plan_bytes = hd.plan_bytes;
    return WPP_OK;
}

// Check a host plan against a description; returns the header on success.
int wpp_check_plan(const void* plan_host, const wpp_batch_desc* resolved, const WppPlanHeader** out) {
    if (!plan_host) return WPP_ERR_INVALID_ARG;
    const WppPlanHeader* h = static_cast<const WppPlanHeader*>(plan_host);
    if (h->magic != WPP_PLAN_MAGIC || h->version != WPP_PLAN_VERSION) return WPP_ERR_PLAN_MISMATCH;
    if (h->desc_hash != wpp_desc_hash(resolved) || h->num_requests != resolved->num_requests ||
        h->head_dim != resolved->head_dim)
        return WPP_ERR_PLAN_MISMATCH;
    *out = h;
    return WPP_OK;
}

int wpp_validate_batch(const wpp_batch_desc* desc, const int32_t* bt, const int32_t* prefix_lens,
                       const int32_t* chunk_lens) {
    wpp_batch_desc d;
    int rc = wpp_resolve_desc(desc, &d);
    if (rc != WPP_OK) return rc;
    const int R = d.num_requests, B = d.page_size;
    if (R > 0 && (!bt || !prefix_lens || !chunk_lens)) return WPP_ERR_INVALID_ARG;
    // written slot -> writer; read ranges per page -> max readable slots by a non-writer
    std::unordered_map<int64_t, int32_t> writer;   // page*B+slot -> request
    for (int i = 0; i < R; ++i) {
        const int64_t P = prefix_lens[i], C = chunk_lens[i];
        if (P < 0 || C < 0) return WPP_ERR_INVALID_ARG;
        const int64_t n = P + C;
        if (C > 0 && (n + B - 1) / B > d.max_blocks_per_req) return WPP_ERR_BOUNDS;
        if (C == 0) continue;
        for (int64_t j = 0; j < (n + B - 1) / B; ++j) {
            const int32_t page = bt[(int64_t)i * d.max_blocks_per_req + j];
            if (page < 0 || page >= d.num_pages) return WPP_ERR_BOUNDS;
        }
        for (int64_t pos = P; pos < n; ++pos) {
            const int64_t key = (int64_t)bt[(int64_t)i * d.max_blocks_per_req + pos / B] * B + pos % B;
            if (!writer.emplace(key, i).second) return WPP_ERR_ALIASED_APPEND;
        }
    }
    for (int i = 0; i < R; ++i) {
        if (chunk_lens[i] == 0) continue;
        const int64_t P = prefix_lens[i];
        for (int64_t pos = 0; pos < P; ++pos) {
            const int64_t key = (int64_t)bt[(int64_t)i * d.max_blocks_per_req + pos / B] * B + pos % B;
            if (writer.count(key)) return WPP_ERR_ALIASED_APPEND;   // someone writes what this request reads
        }
    }
    return WPP_OK;
}
