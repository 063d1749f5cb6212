// Persistent chunked-prefill attention kernel for sm_100a.
//
// One CTA per SM walks the list of work tiles the host planner gave it.  A work tile is two 128-row query
// "halves" (A, B) that share one K/V stream, against key steps [kv_begin, kv_end) of 128 keys each.
// 16 warps, specialised by warpgroup:
//   warps 0-3   softmax of half A: thread r owns query row r (TMEM lane r): row max / row sum need no shuffles
//   warps 4-7   softmax of half B
//   warps 8-11  epilogue: O / l -> bf16 -> global (or fp32 partials for split tiles), overlapping the next tile
//   warps 12,14 tensor-core issuers, one thread per half: S = Q K^T and O += P V with tcgen05.mma (fp32 accumulators
//               in TMEM; P is read from TMEM where the softmax warps wrote it as packed bf16 over S; V is an
//               MN-major operand).  They issue strictly in turns (A, B, A, ...), which keeps the halves in anti-phase
//               while one half's barrier waits never hold up the other half's MMAs.
//   warp 13     producer: reads the block table and issues TMA tile loads (Q once per tile; per key step one box
//               per (page, 64-wide half of head_dim) for K and for V, 128-byte swizzle).  V(j) and K(j+1) are used
//               in the same issuer iteration, so they travel as one ring item with one barrier.
// The two halves ping-pong: while the softmax warps of A work on S_A(j+1), the tensor cores run O_B += P_B V(j)
// and S_B(j+1).  Rescaling is lazy: a row keeps its reference maximum, and does not even compute the maximum of
// a step, as long as the step's row sum shows that no score rose far above the reference; only then (and on the
// first step of a tile) the softmax warps take the true maximum and rescale O and l themselves.
// Tensor memory (512 columns): S_A [0,128)  S_B [128,256)  O_A [256,256+D)  O_B [384,384+D); P aliases the first
// 64 columns of its S.
// All mbarrier waits are bounded; on expiry the CTA raises its abort flag, every role drains, TMEM is freed and
// WPP_ERR_TIMEOUT is written to the status word.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "wpp_device.h"
#include "wpp_plan_format.h"
#include "wpp_ptx.cuh"

namespace wpp {

constexpr int kThreads = 512;
constexpr uint32_t kTmemCols = 512;
__host__ __device__ constexpr uint32_t col_s(int hf) { return 128u * hf; }          // S (and P) of half hf
__host__ __device__ constexpr uint32_t col_o(int hf) { return 256u + 128u * hf; }   // O of half hf
constexpr float kFastPathSumLimit = 65536.f;  // row sum of p below which the old reference was safe to keep
#ifndef WPP_EMU_PAIRS_OF_4
#define WPP_EMU_PAIRS_OF_4 0
#endif
constexpr int kEmuPairsOf4 = WPP_EMU_PAIRS_OF_4;  // of every 4 score pairs, how many take exp2 on the FMA pipes

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzled column blocks
    static constexpr int kTileBytes = 128 * D * 2;         // one 128-row Q half, or one K or V step
    static constexpr int kHalfBytes = 128 * 128;           // 128 rows x 128 bytes
    static constexpr int kItems = (D == 128) ? 2 : 4;      // ring of items {V(j), K(j+1)}
    static constexpr int kItemBytes = 2 * kTileBytes;      // V part, then K part
    static constexpr int kOffKV = 2 * kTileBytes;
    static constexpr int kOffBars = kOffKV + kItems * kItemBytes;
    static constexpr int kNumBars = 2 + 2 * kItems + 5 * 2;
    static constexpr int kOffFinal = kOffBars + 8 * kNumBars;          // float2 (m, l)[2][128]
    static constexpr int kOffMisc = kOffFinal + 2 * 128 * 8;           // tmem ptr, abort flag
    static constexpr int kSmemBytes = kOffMisc + 16 + 1024;            // + alignment slack
};

// Optional timeline instrumentation for tuning (compiled out unless WPP_TRACE is defined): CTA 0 records the
// low 32 bits of clock64 at a few points of its first key steps into p.trace[role][step][event].
#ifdef WPP_TRACE
#define WPP_TRACE_EVENTS 8
#define WPP_TRACE_STEPS 64
#define TRACE(role, step, ev)                                                                              \
    do {                                                                                                   \
        if (p.trace && blockIdx.x == 0 && (threadIdx.x & 127) == 0 && (step) < WPP_TRACE_STEPS)            \
            p.trace[((role) * WPP_TRACE_STEPS + (step)) * WPP_TRACE_EVENTS + (ev)] = (uint32_t)clock64(); \
    } while (0)
#else
#define TRACE(role, step, ev) do { } while (0)
#endif

struct Ring {
    uint32_t stage, phase;
    __device__ __forceinline__ void advance(uint32_t n) {
        if (++stage == n) { stage = 0; phase ^= 1u; }
    }
};

// What every role derives from a unit, identically.
struct UnitView {
    int request, kv_begin, n_steps;      // n_steps = max over halves
    int n[2];                            // key steps of each half (0: nothing to compute)
    int P, kv_len, q_off;
};
__device__ __forceinline__ UnitView view_of(const WppUnit& un, const AttnParams& p, const int32_t* q_offsets) {
    UnitView v;
    v.request = un.request;
    v.kv_begin = un.kv_begin;
    v.P = p.prefix_lens[un.request];
    v.kv_len = v.P + p.chunk_lens[un.request];
    v.q_off = q_offsets[un.request];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int end = un.rows[h] > 0 ? (v.P + un.row0[h] + un.rows[h] + 127) / 128 : 0;
        v.n[h] = max(0, min(un.kv_end, end) - un.kv_begin);
    }
    v.n_steps = max(v.n[0], v.n[1]);
    return v;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
wpp_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_q64,
                const __grid_constant__ CUtensorMap tm_q32, const __grid_constant__ CUtensorMap tm_q16,
                const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;                       // two halves, kTileBytes each
    const uint32_t sKV = smem_base + C::kOffKV;          // kItems x {V tile, K tile}
    const uint32_t bars = smem_base + C::kOffBars;
    const uint32_t bQFull = bars, bQEmpty = bars + 8;
    const uint32_t bItemFull = bars + 16, bItemEmpty = bItemFull + 8 * C::kItems;
    // Per half: s_full (S = Q K^T landed; it also proves the previous O += P V landed, the tensor pipe being in
    // order), p_ready (P written, and O rescaled if the row reference moved, by the 128 softmax threads),
    // final_ready (end-of-tile (m, l) are in smem), o_final (last O += P V landed), o_free (the epilogue threads
    // have read O out, the next tile may overwrite it).  A thread never arrives twice on one barrier without a
    // wait in between that implies the earlier phase completed.
    const uint32_t bHalf = bItemEmpty + 8 * C::kItems;
    auto bSFull = [&](int h) { return bHalf + 40 * h; };
    auto bPReady = [&](int h) { return bHalf + 40 * h + 8; };
    auto bFinalReady = [&](int h) { return bHalf + 40 * h + 16; };
    auto bOFinal = [&](int h) { return bHalf + 40 * h + 24; };
    auto bOFree = [&](int h) { return bHalf + 40 * h + 32; };
    float2* s_final = reinterpret_cast<float2*>(smem_gen + C::kOffFinal);     // [2][128] (reference in log2 units, l)
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* turn = tmem_slot + 2;             // which half's issuer may issue next

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wg = warp >> 2;

    if (threadIdx.x == 0) {
        mbar_init(bQFull, 1); mbar_init(bQEmpty, 2);
        for (int s = 0; s < C::kItems; ++s) { mbar_init(bItemFull + 8 * s, 1); mbar_init(bItemEmpty + 8 * s, 2); }
        for (int h = 0; h < 2; ++h) {
            mbar_init(bSFull(h), 1); mbar_init(bPReady(h), 128);
            mbar_init(bFinalReady(h), 128); mbar_init(bOFinal(h), 1); mbar_init(bOFree(h), 128);
        }
        *abort_flag = 0u;
        *turn = 0u;
        fence_barrier_init();
    }
    if (warp == 12) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 13 && lane == 0) {
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
    const int32_t* cta_begin = reinterpret_cast<const int32_t*>(plan + hd->off_cta_begin);
    const WppUnit* units = reinterpret_cast<const WppUnit*>(plan + hd->off_units);
    const int u_begin = cta_begin[blockIdx.x], u_end = cta_begin[blockIdx.x + 1];
    const int B = p.page_size, ppt = 128 / B;   // pages per key step

    if (wg == 3) {
        setmaxnreg_dec<96>();
        if (warp == 13) {
            // ================================================================ producer
            Ring ring = {0, 0};
            uint32_t q_phase = 0;
            bool dead = false;
            for (int u = u_begin; u < u_end && !dead; ++u) {
                const WppUnit un = units[u];
                const UnitView v = view_of(un, p, q_offsets);
                if (v.n_steps == 0) continue;
                const int n_pages = (v.kv_len + B - 1) / B;
                const int kvh = un.head[0] / p.group;
                const int32_t* bt = p.block_tables + (int64_t)un.request * p.max_blocks;
                // one ring item: V of step jv (if jv >= 0) and K of step jk (if jk < n_steps); lane l moves
                // page l of each step
                auto load_item = [&](int jv, int jk) -> bool {
                    const bool has_v = jv >= 0, has_k = jk < v.n_steps;
                    const int page_v = (v.kv_begin + jv) * ppt, page_k = (v.kv_begin + jk) * ppt;
                    const int cnt_v = has_v ? min(ppt, n_pages - page_v) : 0;
                    const int cnt_k = has_k ? min(ppt, n_pages - page_k) : 0;
                    int pid_v = 0, pid_k = 0;
                    if (lane < cnt_v) pid_v = bt[page_v + lane];
                    if (lane < cnt_k) pid_k = bt[page_k + lane];
                    if (pid_v < 0 || pid_v >= p.num_pages || pid_k < 0 || pid_k >= p.num_pages) {
                        if (p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                        pid_v = (pid_v < 0 || pid_v >= p.num_pages) ? 0 : pid_v;
                        pid_k = (pid_k < 0 || pid_k >= p.num_pages) ? 0 : pid_k;
                    }
                    const bool ok = mbar_wait(bItemEmpty + 8 * ring.stage, ring.phase ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) return false;
                    const uint32_t full = bItemFull + 8 * ring.stage;
                    if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)(cnt_v + cnt_k) * B * D * 2);
                    __syncwarp();
                    const uint32_t dst = sKV + ring.stage * C::kItemBytes + lane * B * 128;
                    if (lane < cnt_v) {
#pragma unroll
                        for (int h = 0; h < C::kHalves; ++h)
                            tma_load_4d(dst + h * C::kHalfBytes, &tm_v, full, h * 64, 0, kvh, pid_v);
                    }
                    if (lane < cnt_k) {
#pragma unroll
                        for (int h = 0; h < C::kHalves; ++h)
                            tma_load_4d(dst + C::kTileBytes + h * C::kHalfBytes, &tm_k, full, h * 64, 0, kvh, pid_k);
                    }
                    ring.advance(C::kItems);
                    return true;
                };
                // K(0) only needs a ring slot, which frees up before the previous tile's Q does
                if (!load_item(-1, 0)) { dead = true; break; }
                const bool ok = mbar_wait(bQEmpty, q_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                q_phase ^= 1u;
                if (lane == 0) {
                    const int nq = (v.n[0] > 0) + (v.n[1] > 0);
                    mbar_arrive_expect_tx(bQFull, nq * C::kTileBytes);
                    // head k of a half lands in tensor rows [k*rph, (k+1)*rph): one box of rph rows per head
                    const int rph = 128 / un.pack;
                    const CUtensorMap* qm = un.pack == 1 ? &tm_q : un.pack == 2 ? &tm_q64 : un.pack == 4 ? &tm_q32 : &tm_q16;
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        if (v.n[hf] == 0) continue;
                        for (int k = 0; k < un.pack; ++k) {
#pragma unroll
                            for (int h = 0; h < C::kHalves; ++h)
                                tma_load_3d(sQ + hf * C::kTileBytes + h * C::kHalfBytes + k * rph * 128, qm, bQFull, h * 64,
                                            un.head[hf] + k, v.q_off + un.row0[hf]);
                        }
                    }
                }
                __syncwarp();
                for (int j = 0; j < v.n_steps; ++j)
                    if (!load_item(j, j + 1)) { dead = true; break; }
            }
        } else if ((warp == 12 || warp == 14) && lane == 0) {
            // ================================================================ tensor-core issuers (one thread per half)
            // Each half has its own issuing thread, so one half's barrier waits and bookkeeping never hold up the
            // other half's MMAs.  A turn word makes them issue strictly in turns (A, B, A, B, ...): that keeps the
            // two halves in anti-phase - while the softmax warps of A own the exp units, the tensor pipe works for
            // B - which two free-running issuers lose (measured).  Both walk the same item ring; an item and the Q
            // buffer are released by both (barrier count 2), and a release is only signalled after the item's
            // "full" barrier was seen, so neither issuer can run a whole ring turn ahead of the other.
            const int hf = (warp == 12) ? 0 : 1;
            Ring ring = {0, 0};
            uint32_t q_phase = 0, p_phase = 0, of_phase = 0;
            int tstep = 0;
            (void)tstep;
            constexpr uint32_t idesc_qk = idesc_bf16(128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(D, 0, 1);
            const uint64_t q_desc = smem_desc_sw128(sQ + hf * C::kTileBytes, 16, 1024);
            const uint64_t k_desc0 = smem_desc_sw128(sKV + C::kTileBytes, 16, 1024);   // + item * (kItemBytes >> 4)
            const uint64_t v_desc0 = smem_desc_sw128(sKV, C::kHalfBytes, 1024);
            const uint32_t tS = tmem + col_s(hf), tO = tmem + col_o(hf);
            bool dead = false;
            auto issue_qk = [&](uint32_t item) {     // S = Q K^T over head_dim in chunks of 16
                const uint64_t kd = k_desc0 + (uint64_t)(item * (C::kItemBytes >> 4));
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * C::kHalfBytes + (kk & 3) * 32) >> 4);
                    if (kk == 0) mma_ss_overwrite(tS, q_desc + off, kd + off, idesc_qk);
                    else mma_ss_accumulate(tS, q_desc + off, kd + off, idesc_qk);
                }
                mma_commit(bSFull(hf));
            };
            // bounded spin on the turn word (shared memory, written by the other issuer)
            auto take_turn = [&]() -> bool {
                if (*turn == (uint32_t)hf) return true;
                const long long t0 = clock64();
                uint32_t n = 0;
                while (*turn != (uint32_t)hf) {
                    if ((++n & 255u) == 0u) {
                        if (*abort_flag) return false;
                        if (clock64() - t0 > WPP_WAIT_LIMIT) { *abort_flag = 1u; return false; }
                    }
                }
                return true;
            };
            auto pass_turn = [&]() {
                __threadfence_block();
                *turn = (uint32_t)(hf ^ 1);
            };
            for (int u = u_begin; u < u_end && !dead; ++u) {
                const WppUnit un = units[u];
                const UnitView v = view_of(un, p, q_offsets);
                if (v.n_steps == 0) continue;
                const int n = v.n[hf];
                // K(0), Q
                if (!mbar_wait(bItemFull + 8 * ring.stage, ring.phase, abort_flag)) break;
                if (!mbar_wait(bQFull, q_phase, abort_flag)) break;
                q_phase ^= 1u;
                tc_fence_after();
                if (!take_turn()) break;
                if (n > 0) issue_qk(ring.stage);
                pass_turn();
                mma_commit(bItemEmpty + 8 * ring.stage);
                if (n <= 1) mma_commit(bQEmpty);              // this half issues no further S for this tile
                ring.advance(C::kItems);
                for (int j = 0; j < v.n_steps; ++j) {
                    // item {V(j), K(j+1)}
                    if (!mbar_wait(bItemFull + 8 * ring.stage, ring.phase, abort_flag)) { dead = true; break; }
                    const uint32_t item = ring.stage;
                    const bool active = j < n;
                    if (active) {
                        const int valid = v.kv_len - (v.kv_begin + j) * 128;      // keys of this step that exist
                        if (valid < 128) {
                            // rows past the end of the sequence may hold anything (stale slots, never-loaded
                            // pages): zero them so that 0 * garbage cannot reach O (both issuers write the same zeros)
                            uint8_t* vg = smem_gen + C::kOffKV + item * C::kItemBytes;
                            for (int h = 0; h < C::kHalves; ++h)
                                for (int i = valid * 8; i < 128 * 8; ++i)
                                    *reinterpret_cast<uint4*>(vg + h * C::kHalfBytes + i * 16) = make_uint4(0, 0, 0, 0);
                            fence_proxy_async_smem();
                        }
                        if (!mbar_wait(bPReady(hf), p_phase, abort_flag)) { dead = true; break; }   // P written, O fixed
                        p_phase ^= 1u;
                        if (j == 0) {
                            // the first product of a tile overwrites O: the previous tile's epilogue must have read it
                            if (!mbar_wait(bOFree(hf), of_phase ^ 1u, abort_flag)) { dead = true; break; }
                            of_phase ^= 1u;
                        }
                        tc_fence_after();
                    }
                    if (!take_turn()) { dead = true; break; }
                    if (active) {
                        const uint64_t vd = v_desc0 + (uint64_t)(item * (C::kItemBytes >> 4));
                        if (j > 0) mma_ts_accumulate(tO, tS, vd, idesc_pv); else mma_ts_overwrite(tO, tS, vd, idesc_pv);
#pragma unroll
                        for (int kk = 1; kk < 8; ++kk) mma_ts_accumulate(tO, tS + kk * 8, vd + (uint64_t)(kk * 128), idesc_pv);
                        if (j + 1 < n) issue_qk(item);            // its commit also covers the O += P V above
                        else mma_commit(bOFinal(hf));
                    }
                    pass_turn();
                    mma_commit(bItemEmpty + 8 * item);
                    if (j + 2 == n) mma_commit(bQEmpty);           // the last S of this half has been issued
                    ring.advance(C::kItems);
                    ++tstep;
                }
            }
        }
    } else if (wg == 2) {
        // ================================================================ epilogue (one thread per output row)
        setmaxnreg_dec<80>();
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t o_phase[2] = {0, 0}, f_phase[2] = {0, 0};
        bool dead = false;
        for (int u = u_begin; u < u_end && !dead; ++u) {
            const WppUnit un = units[u];
            const UnitView v = view_of(un, p, q_offsets);
            // ---- epilogue of both halves
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                if (un.rows[hf] == 0) continue;
                const int rph = 128 / un.pack, rr = r & (rph - 1);       // row inside its head's block
                const int head = un.head[hf] + r / rph;
                const bool row_ok = rr < un.rows[hf];
                const int64_t tok = (int64_t)v.q_off + un.row0[hf] + rr;
                const int64_t prow = ((int64_t)un.split_slot * 2 + hf) * 128 + r;
                if (v.n[hf] == 0) {
                    // a split part that lies wholly above this half's diagonal: no key is visible
                    if (un.split_slot >= 0 && row_ok) p.ws_lse[prow] = -INFINITY;
                    continue;
                }
                bool ok = mbar_wait(bFinalReady(hf), f_phase[hf], abort_flag);      // final (m, l) are in smem
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                f_phase[hf] ^= 1u;
                ok = mbar_wait(bOFinal(hf), o_phase[hf], abort_flag);               // last O += P V has landed
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                o_phase[hf] ^= 1u;
                tc_fence_after();
                const float2 ml = s_final[hf * 128 + r];
                const float inv_l = (ml.y > 0.f) ? 1.f / ml.y : 0.f;
                const float lse2 = (ml.y > 0.f) ? (ml.x + log2f(ml.y)) : -INFINITY;
                if (un.split_slot < 0) {
                    __nv_bfloat16* dst = p.out + tok * p.o_token_stride + (int64_t)head * p.o_head_stride;
#pragma unroll
                    for (int q4 = 0; q4 < D / 32; ++q4) {
                        float o[32];
                        tmem_ld32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
                        tmem_wait_ld();
                        if (row_ok) {
#pragma unroll
                            for (int w4 = 0; w4 < 4; ++w4) {
                                uint4 w;
                                w.x = pack_bf16x2(o[8 * w4 + 0] * inv_l, o[8 * w4 + 1] * inv_l);
                                w.y = pack_bf16x2(o[8 * w4 + 2] * inv_l, o[8 * w4 + 3] * inv_l);
                                w.z = pack_bf16x2(o[8 * w4 + 4] * inv_l, o[8 * w4 + 5] * inv_l);
                                w.w = pack_bf16x2(o[8 * w4 + 6] * inv_l, o[8 * w4 + 7] * inv_l);
                                *reinterpret_cast<uint4*>(dst + q4 * 32 + w4 * 8) = w;
                            }
                        }
                    }
                    if (p.lse && row_ok) p.lse[tok * p.num_q_heads + head] = lse2 * 0.6931471805599453f;
                } else {
                    float* dst = p.ws_o + prow * D;
#pragma unroll
                    for (int q4 = 0; q4 < D / 32; ++q4) {
                        float o[32];
                        tmem_ld32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
                        tmem_wait_ld();
                        if (row_ok) {
#pragma unroll
                            for (int w4 = 0; w4 < 8; ++w4)
                                *reinterpret_cast<float4*>(dst + q4 * 32 + w4 * 4) =
                                    make_float4(o[4 * w4] * inv_l, o[4 * w4 + 1] * inv_l, o[4 * w4 + 2] * inv_l,
                                                o[4 * w4 + 3] * inv_l);
                        }
                    }
                    if (row_ok) p.ws_lse[prow] = lse2;
                }
                tc_fence_before();
                mbar_arrive(bOFree(hf));
            }
        }
    } else {
        // ================================================================ softmax (thread = query row of half `hf`)
        setmaxnreg_inc<168>();
        const int hf = wg;
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t colS = col_s(hf);
        uint32_t s_phase = 0, fin_phase = 0;
        int tstep = 0;      // steps since kernel start (trace index only)
        (void)tstep;
        const float c = p.scale_log2;
        const uint64_t c2 = pack2(c, c);
        bool dead = false;
        for (int u = u_begin; u < u_end && !dead; ++u) {
            const WppUnit un = units[u];
            const UnitView v = view_of(un, p, q_offsets);
            const int n = v.n[hf];
            if (n == 0) continue;
            const int first_pos = v.P + un.row0[hf];          // last key visible to row 0 of this half
            // last key this thread's row may see: its own position (rows of packed heads repeat every 128/pack
            // tensor rows), never past the end of the sequence
            const int row_last = min(first_pos + (r & (128 / un.pack - 1)), v.kv_len - 1);
            // m_ref: reference of the row (raw score units); nmc = -(m_ref * c) rounded once.  Every p of the row is
            // 2^(s*c + nmc) with that same nmc, and a change of reference rescales by 2^(nmc_new - nmc_old) of the two
            // stored numbers, so old and new terms stay consistent even for scores around 1e8.
            float m_ref = -INFINITY, l_run = 0.f, nmc = 0.f;
            for (int j = 0; j < n; ++j) {
                TRACE(hf, tstep, 0);
                const bool ok = mbar_wait(bSFull(hf), s_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                s_phase ^= 1u;
                tc_fence_after();
                TRACE(hf, tstep, 1);
#ifdef WPP_EXPERIMENT_NO_SOFTMAX
                // tuning experiment: how fast is the tile loop when the softmax costs nothing (results are garbage)
                tc_fence_before();
                mbar_arrive(bPReady(hf));
                continue;
#endif
                float s[128];
                const int key0 = (v.kv_begin + j) * 128;
                const bool masked = key0 + 127 > first_pos;    // only steps that touch the diagonal are masked
                const int limit = row_last - key0;
                auto load_scores = [&]() {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        tmem_ld32(lane_addr + colS + q4 * 32, reinterpret_cast<uint32_t*>(s) + q4 * 32);
                    tmem_wait_ld();
                    if (masked) {
#pragma unroll
                        for (int i = 0; i < 128; ++i) s[i] = (i > limit) ? -INFINITY : s[i];
                    }
                };
                // p = 2^(s*c - m_ref*c) for the whole row: bf16 pairs for the tensor cores, fp32 row sum
                uint32_t pk[64];
                auto exp_pass = [&](float neg_mc) -> float {
                    const uint64_t nm2 = pack2(neg_mc, neg_mc);
                    uint64_t sum2a = pack2(0.f, 0.f), sum2b = pack2(0.f, 0.f);
#pragma unroll
                    for (int i = 0; i < 64; ++i) {
                        const uint64_t x2 = ffma2(pack2(s[2 * i], s[2 * i + 1]), c2, nm2);
                        float e0, e1;
                        if ((i & 3) < kEmuPairsOf4) {
                            exp2_poly2(x2, e0, e1);
                        } else {
                            float x0, x1;
                            unpack2(x2, x0, x1);
#ifdef WPP_EXPERIMENT_CHEAP_EXP
                            // tuning experiment: the same loop without the special-function unit (results are garbage)
                            e0 = __saturatef(x0 * 0.01f + 0.5f);
                            e1 = __saturatef(x1 * 0.01f + 0.5f);
#else
                            e0 = fast_exp2(x0);
                            e1 = fast_exp2(x1);
#endif
                        }
                        if (i & 1) sum2b = fadd2(sum2b, pack2(e0, e1)); else sum2a = fadd2(sum2a, pack2(e0, e1));
                        pk[i] = pack_bf16x2(e0, e1);
                    }
                    float t0, t1;
                    unpack2(fadd2(sum2a, sum2b), t0, t1);
                    return t0 + t1;
                };
                load_scores();
                TRACE(hf, tstep, 2);
                // Fast path: keep the row's reference m_ref and skip the row maximum altogether.  The row sum tells
                // whether that was safe: every p <= row sum, so a sum below 2^16 means no score rose more than 16
                // (log2 units) above the reference and nothing can overflow.  Otherwise (or when a row has no
                // reference yet) the warp takes the slow path: true maximum, new reference, O and l rescaled.
                bool slow = __any_sync(0xffffffffu, m_ref == -INFINITY);
                float row_sum = 0.f;
                if (!slow) {
                    row_sum = exp_pass(nmc);
                    slow = __any_sync(0xffffffffu, !(row_sum <= kFastPathSumLimit));
                    if (slow) load_scores();          // S is still intact in tensor memory
                }
                TRACE(hf, tstep, 3);
                if (slow) {
                    float mx[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) mx[k] = fmaxf(s[2 * k], s[2 * k + 1]);
#pragma unroll
                    for (int i = 16; i < 128; i += 16) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) mx[k] = fmax3(mx[k], s[i + 2 * k], s[i + 2 * k + 1]);
                    }
                    const float mxx = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmaxf(fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                    const float m_new = fmaxf(m_ref, mxx);
                    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
                    const float nmc_new = -m_safe * c;
                    const float alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(nmc_new - nmc);
                    nmc = nmc_new;
                    m_ref = m_new;
                    l_run *= alpha;
                    if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                        // S(j) has landed, so the O += P V of step j-1 has too: O may be rescaled in place
#pragma unroll
                        for (int q4 = 0; q4 < D / 32; ++q4) {
                            float o[32];
                            tmem_ld32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= alpha;
                            tmem_st32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
                        }
                    }
                    row_sum = exp_pass(nmc);
                }
                l_run += row_sum;
                TRACE(hf, tstep, 4);
                tmem_st32(lane_addr + colS, pk);
                tmem_st32(lane_addr + colS + 32, pk + 32);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bPReady(hf));
                TRACE(hf, tstep, 5);
                ++tstep;
            }
            if (dead) break;
            {
                // the end-of-tile slot (and its barrier) may only be reused once the epilogue threads have consumed
                // the previous tile's values; for tiles of a single key step nothing else orders the two
                const bool ok = mbar_wait(bOFree(hf), fin_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) break;
                fin_phase ^= 1u;
            }
            s_final[hf * 128 + r] = make_float2(-nmc, l_run);
            mbar_arrive(bFinalReady(hf));
        }
    }

    // ---- teardown: every loop above is bounded, so every thread gets here
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) { }     // let copies and tensor-core work in flight land
        if (threadIdx.x == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 12) {
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
        cudaError_t e = cudaFuncSetAttribute(wpp_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg<D>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    wpp_attn_kernel<D><<<num_ctas, kThreads, Cfg<D>::kSmemBytes, stream>>>(tq[0], tq[1], tq[2], tq[3], tk, tv, p);
    return cudaGetLastError();
}

}  // namespace wpp

// tq: four maps of q with boxes of 128, 64, 32 and 16 rows
extern "C" int wpp_launch_attention(int head_dim, const CUtensorMap* tq, const CUtensorMap* tk, const CUtensorMap* tv,
                                    const wpp::AttnParams* p, int num_ctas, void* stream) {
    if (head_dim == 128) return (int)wpp::launch<128>(tq, *tk, *tv, *p, num_ctas, (cudaStream_t)stream);
    if (head_dim == 64) return (int)wpp::launch<64>(tq, *tk, *tv, *p, num_ctas, (cudaStream_t)stream);
    return (int)cudaErrorInvalidValue;
}
