// Chunked-prefill attention for waves of SHORT tiles (few key steps per tile): a second kernel shape.
//
// The main kernel (wpp_attention.cu) owns an SM: 193 KB of shared memory and all of tensor memory per CTA, two
// 128-row halves in flight.  On tiles of one to eight key steps its pipeline never fills: the start of a tile (tile
// hand-out, unit and page-id reads, Q load, first S, first softmax) and its end (epilogue) take longer than the
// steps in between and nothing of the next tile overlaps them.  This kernel turns the trade round: a CTA is small
// - ONE 128-row half, key steps of 64 keys, 97 KB of shared memory, 256 columns of tensor memory, 192 threads - so
// that TWO CTAs share an SM and one CTA's tile start and end hide under the other's steps.  Inside a CTA the roles
// are the main kernel's, minus the second half: warps 0-3 softmax and epilogue (thread = query row = tensor-memory
// lane), warp 4 producer (tile hand-out, page gather, TMA), warp 5 one thread issuing S = Q K^T and O += P V.
// S(j+1) is issued as soon as the softmax warps have copied S(j) out, so the exponentials of step j overlap the next
// score product.
//
// A work item is one half of a planner tile, (unit, half); the CTAs take items from the counter in the workspace
// in the planner's order.  Arithmetic, masking, lazy rescaling, head packing, split-KV partials and the bounded
// waits are those of the main kernel.
// Tensor memory: S [0, 64)   P [64, 96) (packed bf16)   O [128, 128 + D).
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "wpp_device.h"
#include "wpp_plan_format.h"
#include "wpp_ptx.cuh"

namespace wpp {
namespace small {

constexpr int kThreads = 192;
constexpr int kKeys = 64;                 // keys per step
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColP = 64, kColO = 128;
constexpr float kRefSlack = 16.f;         // a row keeps its reference while its scores stay below reference + 16 (log2)
constexpr int kRescaleCols = 16;

// What every role derives from an item, identically.  A request whose span on the device differs from the plan's
// gets no key steps (see the main kernel).
struct ItemView {
    int P, kv_len, q_off;
    int step0, n;          // first 64-key step (absolute) and number of steps
    bool mismatch;
};
// What the producer hands to the other roles with an item: the unit and everything derived from it, so that no
// consumer repeats the dependent global reads (unit, then the request's lengths) at the start of every item.
struct ItemRec {
    WppUnit un;
    int32_t it;            // item index (2 * unit + half), < 0: no more items
    int32_t P, kv_len, q_off, step0, n, mismatch, pad;
};
template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzled column blocks
    static constexpr int kQBytes = 128 * D * 2;            // the 128-row Q tile
    static constexpr int kQHalfBytes = 128 * 128;
    static constexpr int kKVBytes = kKeys * D * 2;         // one K or V step
    static constexpr int kKVHalfBytes = kKeys * 128;
    static constexpr int kSlots = 2;                       // ring slots for K and for V
    static constexpr int kOffK = kQBytes;
    static constexpr int kOffV = kOffK + kSlots * kKVBytes;
    static constexpr int kOffBars = kOffV + kSlots * kKVBytes;
    static constexpr int kTileQ = 2;
    static constexpr int kNumBars = 2 + 4 * kSlots + 5 + 2 * kTileQ;
    static constexpr int kOffStage = (kOffBars + 8 * kNumBars + 15) / 16 * 16;   // 4 x 2 KB: the warps' store staging
    static constexpr int kOffMisc = kOffStage + 4 * 2048;
    static constexpr int kUsedBytes = kOffMisc + 16 + (int)sizeof(ItemRec) * kTileQ + 8;
    static constexpr int kSmemBytes = kUsedBytes + 1024;   // 105.4 KB at D = 128
};

struct Ring {
    uint32_t stage, phase;
    __device__ __forceinline__ void advance(uint32_t n) {
        if (++stage == n) { stage = 0; phase ^= 1u; }
    }
};

__device__ __forceinline__ ItemView view_of(const WppUnit& un, int hf, const AttnParams& p, const int32_t* q_offsets,
                                            const int32_t* plan_prefix) {
    ItemView v;
    v.P = p.prefix_lens[un.request];
    const int C = p.chunk_lens[un.request];
    v.kv_len = v.P + C;
    v.q_off = q_offsets[un.request];
    v.mismatch = (v.P != plan_prefix[un.request]) || (C != q_offsets[un.request + 1] - v.q_off);
    v.step0 = 2 * un.kv_begin;
    const int end_keys = min(un.kv_end * 128, v.P + un.row0[hf] + un.rows[hf]);        // keys [.., end_keys) can be visible
    v.n = (un.rows[hf] > 0 && !v.mismatch) ? max(0, (end_keys + kKeys - 1) / kKeys - v.step0) : 0;
    return v;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
wpp_attn_small_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_q64,
                      const __grid_constant__ CUtensorMap tm_q32, const __grid_constant__ CUtensorMap tm_q16,
                      const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                      const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base, sK = smem_base + C::kOffK, sV = smem_base + C::kOffV;
    const uint32_t bars = smem_base + C::kOffBars;
    const uint32_t bQFull = bars, bQEmpty = bars + 8;
    const uint32_t bKFull = bars + 16, bKEmpty = bKFull + 8 * C::kSlots;
    const uint32_t bVFull = bKEmpty + 8 * C::kSlots, bVEmpty = bVFull + 8 * C::kSlots;
    // s_full: S landed; s_free: the 128 rows have copied it out; p_ready: P written (and O rescaled if a reference
    // moved); p_free: O += P V landed (P may be replaced, O may be rescaled); o_final: the item's last product landed
    const uint32_t bSFull = bVEmpty + 8 * C::kSlots, bSFree = bSFull + 8, bPReady = bSFull + 16, bPFree = bSFull + 24,
                   bOFinal = bSFull + 32;
    const uint32_t bTileFull = bSFull + 40, bTileEmpty = bTileFull + 8 * C::kTileQ;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile ItemRec* item_q = reinterpret_cast<volatile ItemRec*>(tmem_slot + 4);        // [kTileQ]
    constexpr uint32_t kTileConsumers = 1 + 128;   // the issuing thread and the softmax threads

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(bQFull, 1); mbar_init(bQEmpty, 1);
        for (int s = 0; s < C::kSlots; ++s) {
            mbar_init(bKFull + 8 * s, 1); mbar_init(bKEmpty + 8 * s, 1);
            mbar_init(bVFull + 8 * s, 1); mbar_init(bVEmpty + 8 * s, 1);
        }
        mbar_init(bSFull, 1); mbar_init(bSFree, 128); mbar_init(bPReady, 128); mbar_init(bPFree, 1); mbar_init(bOFinal, 1);
        for (int i = 0; i < C::kTileQ; ++i) { mbar_init(bTileFull + 8 * i, 1); mbar_init(bTileEmpty + 8 * i, kTileConsumers); }
        *abort_flag = 0u;
        fence_barrier_init();
    }
    if (warp == 5) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_q64); prefetch_tensormap(&tm_q32); prefetch_tensormap(&tm_q16);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const char* plan = static_cast<const char*>(p.plan);
    const WppPlanHeader* hd = reinterpret_cast<const WppPlanHeader*>(plan);
    const int32_t* q_offsets = reinterpret_cast<const int32_t*>(plan + hd->off_q_offsets);
    const int32_t* plan_prefix = reinterpret_cast<const int32_t*>(plan + hd->off_prefix);
    const WppUnit* units = reinterpret_cast<const WppUnit*>(plan + hd->off_units);
    const int num_items = 2 * hd->num_units;
    Ring tile_ring = {0, 0};
    // the next item for a consuming role; returns false when the wait was abandoned (rec.it < 0: no more items)
    auto next_item = [&](WppUnit& un, int& hf, ItemView& v, int& it) -> bool {
        if (!mbar_wait(bTileFull + 8 * tile_ring.stage, tile_ring.phase, abort_flag)) return false;
        volatile ItemRec& r = item_q[tile_ring.stage];
        it = r.it;
        if (it >= 0) {
            un.request = r.un.request; un.kv_begin = r.un.kv_begin; un.kv_end = r.un.kv_end; un.split_slot = r.un.split_slot;
            un.row0[0] = r.un.row0[0]; un.row0[1] = r.un.row0[1]; un.rows[0] = r.un.rows[0]; un.rows[1] = r.un.rows[1];
            un.head[0] = r.un.head[0]; un.head[1] = r.un.head[1]; un.cost = r.un.cost; un.pack = r.un.pack;
            hf = it & 1;
            v.P = r.P; v.kv_len = r.kv_len; v.q_off = r.q_off; v.step0 = r.step0; v.n = r.n; v.mismatch = r.mismatch != 0;
        }
        mbar_arrive(bTileEmpty + 8 * tile_ring.stage);
        tile_ring.advance(C::kTileQ);
        return true;
    };
    const int B = p.page_size;
    const int rows_box = B < kKeys ? B : kKeys;       // rows of one K/V box (the maps are built with this box)

    if (warp == 4) {
        // ================================================================ producer
        Ring ring_k = {0, 0}, ring_v = {0, 0};
        uint32_t q_phase = 0;
        bool dead = false;
        // item ids are taken one ahead: the atomic's round trip overlaps the previous item's load issue
        int it_next = 0;
        if (lane == 0) it_next = (int)atomicAdd(p.tile_counter, 1u);
        while (!dead) {
            int it = __shfl_sync(0xffffffffu, it_next, 0);
            if (it >= num_items) it = -1;
            if (it >= 0 && lane == 0) it_next = (int)atomicAdd(p.tile_counter, 1u);
            WppUnit un;
            ItemView v;
            int hf = 0;
            if (it >= 0) {
                un = units[it >> 1];
                hf = it & 1;
                v = view_of(un, hf, p, q_offsets, plan_prefix);
            }
            {
                const bool ok = mbar_wait(bTileEmpty + 8 * tile_ring.stage, tile_ring.phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) break;
                if (lane == 0) {
                    volatile ItemRec& r = item_q[tile_ring.stage];
                    r.it = it;
                    if (it >= 0) {
                        r.un.request = un.request; r.un.kv_begin = un.kv_begin; r.un.kv_end = un.kv_end; r.un.split_slot = un.split_slot;
                        r.un.row0[0] = un.row0[0]; r.un.row0[1] = un.row0[1]; r.un.rows[0] = un.rows[0]; r.un.rows[1] = un.rows[1];
                        r.un.head[0] = un.head[0]; r.un.head[1] = un.head[1]; r.un.cost = un.cost; r.un.pack = un.pack;
                        r.P = v.P; r.kv_len = v.kv_len; r.q_off = v.q_off; r.step0 = v.step0; r.n = v.n; r.mismatch = v.mismatch;
                    }
                    mbar_arrive(bTileFull + 8 * tile_ring.stage);
                }
                tile_ring.advance(C::kTileQ);
            }
            if (it < 0) break;
            if (v.mismatch && lane == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_PLAN_MISMATCH);
            if (v.n == 0) continue;
            const int kvh = un.head[hf] / p.group;
            const int32_t* bt = p.block_tables + (int64_t)un.request * p.max_blocks;
            // one ring slot: the K or the V tile of step j; box b of the step and its column block h go to lane
            // b * kHalves + h
            auto load_tile = [&](const CUtensorMap* tm, int j, Ring& ring, uint32_t s_base, uint32_t full0, uint32_t empty0) -> bool {
                const int key0 = (v.step0 + j) * kKeys;
                const int keys = min(kKeys, v.kv_len - key0);                 // keys of the step that exist
                const int cnt = (keys + rows_box - 1) / rows_box;             // boxes to fetch
                const int bx = lane / C::kHalves, h = lane % C::kHalves;
                const int key_b = key0 + bx * rows_box;
                int pid = 0;
                if (bx < cnt) pid = bt[key_b / B];
                if (pid < 0 || pid >= p.num_pages) {
                    if (p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                    pid = 0;
                }
                const bool ok = mbar_wait(empty0 + 8 * ring.stage, ring.phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) return false;
                const uint32_t full = full0 + 8 * ring.stage;
                if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)cnt * rows_box * D * 2);
                __syncwarp();
                if (bx < cnt)
                    tma_load_4d(s_base + ring.stage * C::kKVBytes + bx * rows_box * 128 + h * C::kKVHalfBytes, tm, full,
                                h * 64, key_b % B, kvh, pid);
                ring.advance(C::kSlots);
                return true;
            };
            auto load_q = [&]() -> bool {
                const bool ok = mbar_wait(bQEmpty, q_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) return false;
                q_phase ^= 1u;
                if (lane == 0) mbar_arrive_expect_tx(bQFull, C::kQBytes);
                __syncwarp();
                // head k of the half lands in tensor rows [k*rph, (k+1)*rph): one box of rph rows per head and
                // 64-column block; box b = (head, column block) is issued by lane b (at most 8 x 2)
                const int rph = 128 / un.pack;
                const CUtensorMap* qm = un.pack == 1 ? &tm_q : un.pack == 2 ? &tm_q64 : un.pack == 4 ? &tm_q32 : &tm_q16;
                if (lane < un.pack * C::kHalves) {
                    const int k = lane / C::kHalves, h = lane % C::kHalves;
                    tma_load_3d(sQ + h * C::kQHalfBytes + k * rph * 128, qm, bQFull, h * 64, un.head[hf] + k,
                                v.q_off + un.row0[hf]);
                }
                return true;
            };
            // the queries need no page ids: they go first when their buffer is free already (the usual case after a
            // short item), else the first K tile goes while the previous item still holds the Q buffer
            const bool q_first = __all_sync(0xffffffffu, mbar_test(bQEmpty, q_phase ^ 1u) != 0u);
            if (q_first && !load_q()) { dead = true; break; }
            if (!load_tile(&tm_k, 0, ring_k, sK, bKFull, bKEmpty)) { dead = true; break; }
            if (!q_first && !load_q()) { dead = true; break; }
            __syncwarp();
            for (int j = 0; j < v.n && !dead; ++j) {
                if (!load_tile(&tm_v, j, ring_v, sV, bVFull, bVEmpty)) dead = true;
                if (!dead && j + 1 < v.n && !load_tile(&tm_k, j + 1, ring_k, sK, bKFull, bKEmpty)) dead = true;
            }
        }
    } else if (warp == 5 && lane == 0) {
        // ================================================================ issuer of S = Q K^T and O += P V (one thread)
        Ring ring_k = {0, 0}, ring_v = {0, 0};
        uint32_t q_phase = 0, sfree_phase = 0, pready_phase = 0;
        constexpr uint32_t idesc_qk = idesc_bf16(kKeys, 0, 0), idesc_pv = idesc_bf16(D, 0, 1);
        const uint64_t q_desc = smem_desc_sw128(sQ, 16, 1024);
        const uint64_t k_desc0 = smem_desc_sw128(sK, 16, 1024);                      // + stage * (kKVBytes >> 4)
        const uint64_t v_desc0 = smem_desc_sw128(sV, C::kKVHalfBytes, 1024);
        const uint32_t tS = tmem + kColS, tP = tmem + kColP, tO = tmem + kColO;
        bool dead = false;
        auto issue_s = [&](int) -> bool {
            if (!mbar_wait(bKFull + 8 * ring_k.stage, ring_k.phase, abort_flag)) return false;
            if (!mbar_wait(bSFree, sfree_phase ^ 1u, abort_flag)) return false;       // the landing buffer was copied out
            sfree_phase ^= 1u;
            tc_fence_after();
            const uint64_t kd = k_desc0 + (uint64_t)(ring_k.stage * (C::kKVBytes >> 4));
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint64_t qoff = (uint64_t)(((kk >> 2) * C::kQHalfBytes + (kk & 3) * 32) >> 4);
                const uint64_t koff = (uint64_t)(((kk >> 2) * C::kKVHalfBytes + (kk & 3) * 32) >> 4);
                if (kk == 0) mma_ss_overwrite(tS, q_desc + qoff, kd + koff, idesc_qk);
                else mma_ss_accumulate(tS, q_desc + qoff, kd + koff, idesc_qk);
            }
            mma_commit(bSFull);
            mma_commit(bKEmpty + 8 * ring_k.stage);
            ring_k.advance(C::kSlots);
            return true;
        };
        while (!dead) {
            WppUnit un;
            ItemView v;
            int hf = 0, it = -1;
            if (!next_item(un, hf, v, it) || it < 0) break;
            if (v.n == 0) continue;
            if (!mbar_wait(bQFull, q_phase, abort_flag)) break;
            q_phase ^= 1u;
            if (!issue_s(0)) break;
            for (int j = 0; j < v.n; ++j) {
                if (j + 1 < v.n) { if (!issue_s(j + 1)) { dead = true; break; } }
                else mma_commit(bQEmpty);                   // every S of the item has been issued: Q may be replaced
                if (!mbar_wait(bVFull + 8 * ring_v.stage, ring_v.phase, abort_flag)) { dead = true; break; }
                const int valid = v.kv_len - (v.step0 + j) * kKeys;      // keys of this step that exist
                if (valid < kKeys) {
                    // rows past the end of the sequence may hold anything (stale slots, boxes never fetched): zero
                    // them so that 0 * garbage cannot reach O
                    uint8_t* vg = smem_gen + C::kOffV + ring_v.stage * C::kKVBytes;
                    for (int h = 0; h < C::kHalves; ++h)
                        for (int i = valid * 8; i < kKeys * 8; ++i)
                            *reinterpret_cast<uint4*>(vg + h * C::kKVHalfBytes + i * 16) = make_uint4(0, 0, 0, 0);
                    fence_proxy_async_smem();
                }
                if (!mbar_wait(bPReady, pready_phase, abort_flag)) { dead = true; break; }      // P written, O fixed
                pready_phase ^= 1u;
                tc_fence_after();
                const uint64_t vd = v_desc0 + (uint64_t)(ring_v.stage * (C::kKVBytes >> 4));
                if (j > 0) mma_ts_accumulate(tO, tP, vd, idesc_pv); else mma_ts_overwrite(tO, tP, vd, idesc_pv);
#pragma unroll
                for (int kk = 1; kk < kKeys / 16; ++kk) mma_ts_accumulate(tO, tP + kk * 8, vd + (uint64_t)(kk * 128), idesc_pv);
                mma_commit(bPFree);
                if (j + 1 == v.n) mma_commit(bOFinal);
                mma_commit(bVEmpty + 8 * ring_v.stage);
                ring_v.advance(C::kSlots);
            }
        }
    } else if (warp < 4) {
        // ================================================================ softmax and epilogue (thread = query row)
        const int r = threadIdx.x;
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        uint32_t s_phase = 0, pf_phase = 0, of_phase = 0;
        const float c = p.scale_log2;
        const uint64_t c2 = pack2(c, c);
        bool dead = false;
        while (!dead) {
            WppUnit un;
            ItemView v;
            int hf = 0, it = -1;
            const bool got = next_item(un, hf, v, it);
            if (!__all_sync(0xffffffffu, got) || it < 0) break;
            if (un.rows[hf] == 0) continue;
            const int rph = 128 / un.pack, rr = r & (rph - 1);           // row inside its head's block
            const int head = un.head[hf] + r / rph;
            const bool row_ok = rr < un.rows[hf];
            const int64_t tok = (int64_t)v.q_off + un.row0[hf] + rr;
            const int64_t prow = ((int64_t)un.split_slot * 2 + hf) * 128 + r;
            if (v.n == 0) {
                // a split part that lies wholly above this half's diagonal (or a refused request): no key is visible
                if (un.split_slot >= 0 && row_ok) p.ws_lse[prow] = -INFINITY;
                continue;
            }
            const int first_pos = v.P + un.row0[hf];          // last key visible to row 0 of this half
            const int row_last = min(first_pos + rr, v.kv_len - 1);
            float m_ref = -INFINITY, l_run = 0.f, nmc = 0.f;
            for (int j = 0; j < v.n; ++j) {
                {
                    const bool ok = mbar_wait(bSFull, s_phase, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                }
                s_phase ^= 1u;
                tc_fence_after();
                float s[kKeys];
                tmem_ld32(lane_addr + kColS, reinterpret_cast<uint32_t*>(s));
                tmem_ld32(lane_addr + kColS + 32, reinterpret_cast<uint32_t*>(s) + 32);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bSFree);
                const int key0 = (v.step0 + j) * kKeys;
                if (key0 + kKeys - 1 > first_pos) {           // only steps that touch the diagonal are masked
                    const int limit = row_last - key0;
#pragma unroll
                    for (int i = 0; i < kKeys; ++i) s[i] = (i > limit) ? -INFINITY : s[i];
                }
                float mx[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) mx[k] = fmaxf(s[2 * k], s[2 * k + 1]);
#pragma unroll
                for (int i = 16; i < kKeys; i += 16) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) mx[k] = fmax3(mx[k], s[i + 2 * k], s[i + 2 * k + 1]);
                }
                const float mxx = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmaxf(fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                bool waited = false;
                const bool move = (m_ref == -INFINITY) || !(fmaf(mxx, c, nmc) <= kRefSlack);
                if (__any_sync(0xffffffffu, move)) {
                    const float m_new = fmaxf(m_ref, mxx);
                    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
                    const float nmc_new = -m_safe * c;
                    const float alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(nmc_new - nmc);
                    nmc = nmc_new;
                    m_ref = m_new;
                    l_run *= alpha;
                    if (j > 0) {
                        // O may only be touched once the O += P V of step j-1 has landed
                        const bool okp = mbar_wait(bPFree, pf_phase, abort_flag);
                        if (!__all_sync(0xffffffffu, okp)) { dead = true; break; }
                        pf_phase ^= 1u;
                        waited = true;
                        tc_fence_after();
                        if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
                            for (int q0 = 0; q0 < D; q0 += kRescaleCols) {
                                float o[kRescaleCols];
#pragma unroll
                                for (int c8 = 0; c8 < kRescaleCols; c8 += 8)
                                    tmem_ld8(lane_addr + kColO + q0 + c8, reinterpret_cast<uint32_t*>(o) + c8);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < kRescaleCols; ++i) o[i] *= alpha;
#pragma unroll
                                for (int c8 = 0; c8 < kRescaleCols; c8 += 8)
                                    tmem_st8(lane_addr + kColO + q0 + c8, reinterpret_cast<uint32_t*>(o) + c8);
                            }
                        }
                    }
                }
                // p = 2^(s*c - m_ref*c) for the whole row: bf16 pairs for the tensor cores, fp32 row sum
                uint32_t* pk = reinterpret_cast<uint32_t*>(s);
                {
                    const uint64_t nm2 = pack2(nmc, nmc);
                    uint64_t sum2a = pack2(0.f, 0.f), sum2b = pack2(0.f, 0.f);
#pragma unroll
                    for (int i0 = 0; i0 < kKeys / 2; i0 += 8) {
                        uint64_t x2[8];
                        float e[16];
#pragma unroll
                        for (int k = 0; k < 8; ++k) x2[k] = ffma2(pack2(s[2 * (i0 + k)], s[2 * (i0 + k) + 1]), c2, nm2);
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            float x0, x1;
                            unpack2(x2[k], x0, x1);
                            e[2 * k] = fast_exp2(x0);
                            e[2 * k + 1] = fast_exp2(x1);
                        }
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            if (k & 1) sum2b = fadd2(sum2b, pack2(e[2 * k], e[2 * k + 1]));
                            else sum2a = fadd2(sum2a, pack2(e[2 * k], e[2 * k + 1]));
                            pk[i0 + k] = pack_bf16x2(e[2 * k], e[2 * k + 1]);
                        }
                    }
                    float t0, t1;
                    unpack2(fadd2(sum2a, sum2b), t0, t1);
                    l_run += t0 + t1;
                }
                if (!waited && j > 0) {
                    // P(j-1) must have been consumed before P(j) replaces it
                    const bool okp = mbar_wait(bPFree, pf_phase, abort_flag);
                    if (!__all_sync(0xffffffffu, okp)) { dead = true; break; }
                    pf_phase ^= 1u;
                    tc_fence_after();
                }
#pragma unroll
                for (int c8 = 0; c8 < kKeys / 2; c8 += 8) tmem_st8(lane_addr + kColP + c8, pk + c8);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bPReady);
            }
            if (dead) break;
            // ---- epilogue: the item's last product has landed (which also consumes the last p_free phase)
            {
                bool ok = mbar_wait(bOFinal, of_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) break;
                of_phase ^= 1u;
                ok = mbar_wait(bPFree, pf_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) break;
                pf_phase ^= 1u;
            }
            tc_fence_after();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const float lse2 = (l_run > 0.f) ? (-nmc + log2f(l_run)) : -INFINITY;
            uint8_t* stage = smem_gen + C::kOffStage + warp * 2048;
            if (un.split_slot < 0) {
                const __nv_bfloat16* dst = p.out + tok * p.o_token_stride + (int64_t)head * p.o_head_stride;
#pragma unroll 1
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    float o[32];
                    tmem_ld32(lane_addr + kColO + q4 * 32, reinterpret_cast<uint32_t*>(o));
                    tmem_wait_ld();
                    uint4 w[4];
#pragma unroll
                    for (int w4 = 0; w4 < 4; ++w4) {
                        w[w4].x = pack_bf16x2(o[8 * w4 + 0] * inv_l, o[8 * w4 + 1] * inv_l);
                        w[w4].y = pack_bf16x2(o[8 * w4 + 2] * inv_l, o[8 * w4 + 3] * inv_l);
                        w[w4].z = pack_bf16x2(o[8 * w4 + 4] * inv_l, o[8 * w4 + 5] * inv_l);
                        w[w4].w = pack_bf16x2(o[8 * w4 + 6] * inv_l, o[8 * w4 + 7] * inv_l);
                    }
                    warp_store_rows64(stage, lane, w, dst, row_ok, q4 * 64);
                }
                if (p.lse && row_ok) p.lse[tok * p.num_q_heads + head] = lse2 * 0.6931471805599453f;
            } else {
                const float* dst = p.ws_o + prow * D;
#pragma unroll 1
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    float o[32];
                    tmem_ld32(lane_addr + kColO + q4 * 32, reinterpret_cast<uint32_t*>(o));
                    tmem_wait_ld();
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {
                        uint4 w[4];
#pragma unroll
                        for (int w4 = 0; w4 < 4; ++w4) {
                            w[w4].x = __float_as_uint(o[16 * h2 + 4 * w4 + 0] * inv_l);
                            w[w4].y = __float_as_uint(o[16 * h2 + 4 * w4 + 1] * inv_l);
                            w[w4].z = __float_as_uint(o[16 * h2 + 4 * w4 + 2] * inv_l);
                            w[w4].w = __float_as_uint(o[16 * h2 + 4 * w4 + 3] * inv_l);
                        }
                        warp_store_rows64(stage, lane, w, dst, row_ok, q4 * 128 + h2 * 64);
                    }
                }
                if (row_ok) p.ws_lse[prow] = lse2;
            }
            tc_fence_before();
        }
    }

    // ---- teardown: every loop above is bounded, so every thread gets here
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) { }     // let copies and tensor-core work in flight land
        if (threadIdx.x == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

template <int D>
static cudaError_t launch(const CUtensorMap* tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                          int num_ctas, cudaStream_t stream) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(wpp_attn_small_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg<D>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    wpp_attn_small_kernel<D><<<num_ctas, kThreads, Cfg<D>::kSmemBytes, stream>>>(tq[0], tq[1], tq[2], tq[3], tk, tv, p);
    return cudaGetLastError();
}

}  // namespace small
}  // namespace wpp

// tq: four maps of q with boxes of 128, 64, 32 and 16 rows; tk, tv: maps whose boxes have min(page_size, 64) rows
extern "C" int wpp_launch_attention_small(int head_dim, const CUtensorMap* tq, const CUtensorMap* tk, const CUtensorMap* tv,
                                          const wpp::AttnParams* p, int num_ctas, void* stream) {
    if (head_dim == 128) return (int)wpp::small::launch<128>(tq, *tk, *tv, *p, num_ctas, (cudaStream_t)stream);
    if (head_dim == 64) return (int)wpp::small::launch<64>(tq, *tk, *tv, *p, num_ctas, (cudaStream_t)stream);
    return (int)cudaErrorInvalidValue;
}
