// Persistent chunked-prefill attention kernel for sm_100a.
//
// One CTA per SM walks the list of work tiles the host planner gave it.  A work tile is two 128-row query
// "halves" (A, B) that share one K/V stream, against key steps [kv_begin, kv_end) of 128 keys each.
// 16 warps, specialised by warpgroup:
//   warps 0-3   softmax of half A: thread r owns query row r (TMEM lane r): row max / row sum need no shuffles
//   warps 4-7   softmax of half B
//   warps 8-11  correction: rescales the O accumulators in TMEM when a running maximum moved, and runs the
//               epilogue (O / l -> bf16 -> global, or fp32 partials for split tiles)
//   warp 12     tensor-core issuer: S = Q K^T and O += P V with tcgen05.mma (fp32 accumulators in TMEM; P is
//               read from TMEM where the softmax warps wrote it as packed bf16 over S; V is an MN-major operand)
//   warp 13     producer: reads the block table and issues TMA tile loads (Q once per tile; per key step one box
//               per (page, 64-wide half of head_dim) for K and for V, 128-byte swizzle, 4-deep ring)
// The two halves ping-pong: while the softmax warps of A work on S_A(j+1), the tensor cores run O_B += P_B V(j)
// and S_B(j+1).  Rescaling is lazy: the reference maximum of a row only moves when the new maximum exceeds it by
// more than 2^8, so the correction warps rarely touch O after the first steps.
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
constexpr float kRescaleThreshold = 8.0f;     // log2 units

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzled column blocks
    static constexpr int kTileBytes = 128 * D * 2;         // one 128-row Q half, or one K or V step
    static constexpr int kHalfBytes = 128 * 128;           // 128 rows x 128 bytes
    static constexpr int kStages = 4;                      // K/V ring (K(j), V(j), K(j+1), V(j+1))
    static constexpr int kOffKV = 2 * kTileBytes;
    static constexpr int kOffBars = kOffKV + kStages * kTileBytes;
    static constexpr int kNumBars = 2 + 2 * kStages + 6 * 2;
    static constexpr int kOffScale = kOffBars + 8 * kNumBars;          // float alpha[2][128]
    static constexpr int kOffFinal = kOffScale + 2 * 128 * 4;          // float2 (m, l)[2][128]
    static constexpr int kOffMisc = kOffFinal + 2 * 128 * 8;           // tmem ptr, abort flag
    static constexpr int kSmemBytes = kOffMisc + 16 + 1024;            // + alignment slack
};

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
wpp_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;                       // two halves, kTileBytes each
    const uint32_t sKV = smem_base + C::kOffKV;
    const uint32_t bars = smem_base + C::kOffBars;
    const uint32_t bQFull = bars, bQEmpty = bars + 8;
    const uint32_t bKVFull = bars + 16, bKVEmpty = bKVFull + 8 * C::kStages;
    // per half: s_full, p_full, o_full, corr_ready, corr_done, final_ready.  A thread never arrives twice on one
    // barrier without a wait in between that implies the earlier phase completed; that is why the end-of-tile
    // hand-over of (m, l) has a barrier of its own instead of reusing corr_ready.
    const uint32_t bHalf = bKVEmpty + 8 * C::kStages;
    auto bSFull = [&](int h) { return bHalf + 48 * h; };
    auto bPFull = [&](int h) { return bHalf + 48 * h + 8; };
    auto bOFull = [&](int h) { return bHalf + 48 * h + 16; };
    auto bCorrReady = [&](int h) { return bHalf + 48 * h + 24; };
    auto bCorrDone = [&](int h) { return bHalf + 48 * h + 32; };
    auto bFinalReady = [&](int h) { return bHalf + 48 * h + 40; };
    float* s_alpha = reinterpret_cast<float*>(smem_gen + C::kOffScale);       // [2][128]
    float2* s_final = reinterpret_cast<float2*>(smem_gen + C::kOffFinal);     // [2][128] (m_ref, l)
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wg = warp >> 2;

    if (threadIdx.x == 0) {
        mbar_init(bQFull, 1); mbar_init(bQEmpty, 1);
        for (int s = 0; s < C::kStages; ++s) { mbar_init(bKVFull + 8 * s, 1); mbar_init(bKVEmpty + 8 * s, 1); }
        for (int h = 0; h < 2; ++h) {
            mbar_init(bSFull(h), 1); mbar_init(bPFull(h), 128); mbar_init(bOFull(h), 1);
            mbar_init(bCorrReady(h), 128); mbar_init(bCorrDone(h), 128); mbar_init(bFinalReady(h), 128);
        }
        *abort_flag = 0u;
        fence_barrier_init();
    }
    if (warp == 12) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 13 && lane == 0) {
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
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
        setmaxnreg_dec<56>();
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
                // K(j) then V(j) into consecutive ring slots; lane l moves page (j*ppt + l) of the step
                auto load_step = [&](int j) -> bool {
                    const int page0 = (v.kv_begin + j) * ppt;
                    const int cnt = min(ppt, n_pages - page0);
                    int pid = 0;
                    if (lane < cnt) {
                        pid = bt[page0 + lane];
                        if (pid < 0 || pid >= p.num_pages) {
                            if (p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                            pid = 0;
                        }
                    }
                    const uint32_t bytes = (uint32_t)cnt * B * D * 2;
#pragma unroll
                    for (int kv = 0; kv < 2; ++kv) {
                        const bool ok = mbar_wait(bKVEmpty + 8 * ring.stage, ring.phase ^ 1u, abort_flag);
                        if (!__all_sync(0xffffffffu, ok)) return false;
                        const uint32_t full = bKVFull + 8 * ring.stage;
                        if (lane == 0) mbar_arrive_expect_tx(full, bytes);
                        __syncwarp();
                        if (lane < cnt) {
                            const uint32_t dst = sKV + ring.stage * C::kTileBytes + lane * B * 128;
#pragma unroll
                            for (int h = 0; h < C::kHalves; ++h)
                                tma_load_4d(dst + h * C::kHalfBytes, kv == 0 ? &tm_k : &tm_v, full, h * 64, 0, kvh, pid);
                        }
                        ring.advance(C::kStages);
                    }
                    return true;
                };
                // the first step's K/V only needs ring slots, which free up before the previous tile's Q does
                if (!load_step(0)) { dead = true; break; }
                const bool ok = mbar_wait(bQEmpty, q_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                q_phase ^= 1u;
                if (lane == 0) {
                    const int nq = (v.n[0] > 0) + (v.n[1] > 0);
                    mbar_arrive_expect_tx(bQFull, nq * C::kTileBytes);
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        if (v.n[hf] == 0) continue;
#pragma unroll
                        for (int h = 0; h < C::kHalves; ++h)
                            tma_load_3d(sQ + hf * C::kTileBytes + h * C::kHalfBytes, &tm_q, bQFull, h * 64, un.head[hf],
                                        v.q_off + un.row0[hf]);
                    }
                }
                __syncwarp();
                for (int j = 1; j < v.n_steps; ++j)
                    if (!load_step(j)) { dead = true; break; }
            }
        } else if (warp == 12) {
            // ================================================================ tensor-core issuer
            Ring ring = {0, 0};
            uint32_t q_phase = 0, p_phase[2] = {0, 0}, c_phase[2] = {0, 0};
            constexpr uint32_t idesc_qk = idesc_bf16(128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(D, 0, 1);
            bool dead = false;
            auto issue_qk = [&](int hf, uint32_t kb) {
                if (lane == 0) {
                    const uint32_t qb = sQ + hf * C::kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * C::kHalfBytes + (kk & 3) * 32;
                        mma_ss(tmem + col_s(hf), smem_desc_sw128(qb + off, 16, 1024), smem_desc_sw128(kb + off, 16, 1024),
                               idesc_qk, kk > 0);
                    }
                    mma_commit(bSFull(hf));
                }
                __syncwarp();
            };
            for (int u = u_begin; u < u_end && !dead; ++u) {
                const WppUnit un = units[u];
                const UnitView v = view_of(un, p, q_offsets);
                if (v.n_steps == 0) continue;
                // K(0)
                bool ok = mbar_wait(bKVFull + 8 * ring.stage, ring.phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                ok = mbar_wait(bQFull, q_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                q_phase ^= 1u;
                tc_fence_after();
                uint32_t k_stage = ring.stage;
                ring.advance(C::kStages);
                if (v.n[0] > 0) issue_qk(0, sKV + k_stage * C::kTileBytes);
                if (v.n[1] > 0) issue_qk(1, sKV + k_stage * C::kTileBytes);
                if (lane == 0) {
                    mma_commit(bKVEmpty + 8 * k_stage);
                    if (v.n_steps == 1) mma_commit(bQEmpty);
                }
                __syncwarp();
                for (int j = 0; j < v.n_steps; ++j) {
                    // V(j)
                    ok = mbar_wait(bKVFull + 8 * ring.stage, ring.phase, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                    const uint32_t v_stage = ring.stage;
                    ring.advance(C::kStages);
                    const uint32_t vb = sKV + v_stage * C::kTileBytes;
                    const int valid = v.kv_len - (v.kv_begin + j) * 128;      // keys of this step that exist
                    if (valid < 128) {
                        // rows past the end of the sequence may hold anything (stale slots, never-loaded pages):
                        // zero them so that 0 * garbage cannot reach O
                        uint8_t* vg = smem_gen + (vb - smem_base);
                        const int rows = 128 - valid;
                        for (int i = lane; i < rows * 8 * C::kHalves; i += 32) {
                            const int h = i / (rows * 8), rem = i % (rows * 8);
                            *reinterpret_cast<uint4*>(vg + h * C::kHalfBytes + (valid + rem / 8) * 128 + (rem % 8) * 16) =
                                make_uint4(0, 0, 0, 0);
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                    }
                    // K(j+1)
                    const bool more = j + 1 < v.n_steps;
                    if (more) {
                        ok = mbar_wait(bKVFull + 8 * ring.stage, ring.phase, abort_flag);
                        if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                        k_stage = ring.stage;
                        ring.advance(C::kStages);
                    }
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        if (j >= v.n[hf]) continue;
                        ok = mbar_wait(bPFull(hf), p_phase[hf], abort_flag);
                        if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                        p_phase[hf] ^= 1u;
                        ok = mbar_wait(bCorrDone(hf), c_phase[hf], abort_flag);
                        if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                        c_phase[hf] ^= 1u;
                        tc_fence_after();
                        if (lane == 0) {
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)
                                mma_ts(tmem + col_o(hf), tmem + col_s(hf) + kk * 8,
                                       smem_desc_sw128(vb + kk * 2048, C::kHalfBytes, 1024), idesc_pv, (j > 0) || (kk > 0));
                            mma_commit(bOFull(hf));
                        }
                        __syncwarp();
                        if (j + 1 < v.n[hf]) issue_qk(hf, sKV + k_stage * C::kTileBytes);
                    }
                    if (dead) break;
                    if (lane == 0) {
                        mma_commit(bKVEmpty + 8 * v_stage);
                        if (more) mma_commit(bKVEmpty + 8 * k_stage);
                        if (j + 2 == v.n_steps) mma_commit(bQEmpty);   // the last S of this tile has been issued
                    }
                    __syncwarp();
                }
            }
        }
    } else if (wg == 2) {
        // ================================================================ correction + epilogue
        setmaxnreg_dec<88>();
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t cr_phase[2] = {0, 0}, o_phase[2] = {0, 0}, f_phase[2] = {0, 0};
        bool dead = false;
        for (int u = u_begin; u < u_end && !dead; ++u) {
            const WppUnit un = units[u];
            const UnitView v = view_of(un, p, q_offsets);
            for (int j = 0; j < v.n_steps && !dead; ++j) {
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (j >= v.n[hf]) continue;
                    bool ok = mbar_wait(bCorrReady(hf), cr_phase[hf], abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                    cr_phase[hf] ^= 1u;
                    const float alpha = s_alpha[hf * 128 + r];
                    if (j > 0) {
                        ok = mbar_wait(bOFull(hf), o_phase[hf], abort_flag);     // O += P V of step j-1 has landed
                        if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                        o_phase[hf] ^= 1u;
                        if (__any_sync(0xffffffffu, alpha != 1.f)) {
                            tc_fence_after();
#pragma unroll
                            for (int q4 = 0; q4 < D / 32; ++q4) {
                                float o[32];
                                tmem_ld32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; ++i) o[i] *= alpha;
                                tmem_st32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
                            }
                            tmem_wait_st();
                            tc_fence_before();
                        }
                    }
                    mbar_arrive(bCorrDone(hf));
                }
            }
            if (dead) break;
            // ---- epilogue of both halves
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                if (un.rows[hf] == 0) continue;
                const bool row_ok = r < un.rows[hf];
                const int64_t tok = (int64_t)v.q_off + un.row0[hf] + r;
                const int64_t prow = ((int64_t)un.split_slot * 2 + hf) * 128 + r;
                if (v.n[hf] == 0) {
                    // a split part that lies wholly above this half's diagonal: no key is visible
                    if (un.split_slot >= 0 && row_ok) p.ws_lse[prow] = -INFINITY;
                    continue;
                }
                bool ok = mbar_wait(bFinalReady(hf), f_phase[hf], abort_flag);      // final (m, l) are in smem
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                f_phase[hf] ^= 1u;
                ok = mbar_wait(bOFull(hf), o_phase[hf], abort_flag);                // last O += P V has landed
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                o_phase[hf] ^= 1u;
                tc_fence_after();
                const float2 ml = s_final[hf * 128 + r];
                const float inv_l = (ml.y > 0.f) ? 1.f / ml.y : 0.f;
                const float lse2 = (ml.y > 0.f) ? (ml.x * p.scale_log2 + log2f(ml.y)) : -INFINITY;
                if (un.split_slot < 0) {
                    __nv_bfloat16* dst = p.out + tok * p.o_token_stride + (int64_t)un.head[hf] * p.o_head_stride;
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
                    if (p.lse && row_ok) p.lse[tok * p.num_q_heads + un.head[hf]] = lse2 * 0.6931471805599453f;
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
            }
        }
    } else {
        // ================================================================ softmax (thread = query row of half `hf`)
        setmaxnreg_inc<184>();
        const int hf = wg;
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t colS = col_s(hf);
        uint32_t s_phase = 0;
        const float c = p.scale_log2;
        bool dead = false;
        for (int u = u_begin; u < u_end && !dead; ++u) {
            const WppUnit un = units[u];
            const UnitView v = view_of(un, p, q_offsets);
            const int n = v.n[hf];
            if (n == 0) continue;
            const int first_pos = v.P + un.row0[hf];          // last key visible to row 0 of this half
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n; ++j) {
                const bool ok = mbar_wait(bSFull(hf), s_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                s_phase ^= 1u;
                tc_fence_after();
                float s[128];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(lane_addr + colS + q4 * 32, reinterpret_cast<uint32_t*>(s) + q4 * 32);
                tmem_wait_ld();
                const int key0 = (v.kv_begin + j) * 128;
                if (key0 + 127 > first_pos) {               // only steps that touch the diagonal are masked
                    const int limit = first_pos + r - key0;
#pragma unroll
                    for (int i = 0; i < 128; ++i) s[i] = (i > limit) ? -INFINITY : s[i];
                }
                float mx0 = fmaxf(s[0], s[1]), mx1 = fmaxf(s[2], s[3]);
#pragma unroll
                for (int i = 4; i < 128; i += 4) {
                    mx0 = fmaxf(mx0, fmaxf(s[i], s[i + 1]));
                    mx1 = fmaxf(mx1, fmaxf(s[i + 2], s[i + 3]));
                }
                const float mx = fmaxf(mx0, mx1);
                // lazy rescale: keep the old reference unless the new maximum is far above it
                float alpha = 1.f;
                if ((mx - m_ref) * c > kRescaleThreshold || m_ref == -INFINITY) {
                    const float m_new = fmaxf(m_ref, mx);
                    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
                    alpha = fast_exp2((m_ref - m_safe) * c);        // 0 when there was no reference yet
                    m_ref = m_new;
                    l_run *= alpha;
                }
                s_alpha[hf * 128 + r] = (j == 0) ? 1.f : alpha;
                mbar_arrive(bCorrReady(hf));
                const float neg_mc = (m_ref == -INFINITY) ? 0.f : -m_ref * c;
                float sum0 = 0.f, sum1 = 0.f;
                uint32_t pk[64];
#pragma unroll
                for (int i = 0; i < 64; ++i) {
                    const float a = fast_exp2(fmaf(s[2 * i], c, neg_mc));
                    const float b = fast_exp2(fmaf(s[2 * i + 1], c, neg_mc));
                    sum0 += a;
                    sum1 += b;
                    pk[i] = pack_bf16x2(a, b);
                }
                l_run += sum0 + sum1;
                tmem_st32(lane_addr + colS, pk);
                tmem_st32(lane_addr + colS + 32, pk + 32);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bPFull(hf));
            }
            if (dead) break;
            s_final[hf * 128 + r] = make_float2(m_ref, l_run);
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
static cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
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
    wpp_attn_kernel<D><<<num_ctas, kThreads, Cfg<D>::kSmemBytes, stream>>>(tq, tk, tv, p);
    return cudaGetLastError();
}

}  // namespace wpp

extern "C" int wpp_launch_attention(int head_dim, const CUtensorMap* tq, const CUtensorMap* tk, const CUtensorMap* tv,
                                    const wpp::AttnParams* p, int num_ctas, void* stream) {
    if (head_dim == 128) return (int)wpp::launch<128>(*tq, *tk, *tv, *p, num_ctas, (cudaStream_t)stream);
    if (head_dim == 64) return (int)wpp::launch<64>(*tq, *tk, *tv, *p, num_ctas, (cudaStream_t)stream);
    return (int)cudaErrorInvalidValue;
}
