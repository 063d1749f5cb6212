// Persistent chunked-prefill attention kernel for sm_100a.
//
// One CTA per SM walks the list of work tiles the host planner gave it.  A work tile is 128 query rows of one
// request and one query head against key steps [kv_begin, kv_end) of 128 keys each.  Roles:
//   warps 0-3  softmax + epilogue: thread r owns query row r (TMEM lane r), so row max / row sum need no shuffles
//   warp 4     producer: reads the block table and issues TMA tile loads (Q once per tile; per key step the K and
//              V pages of that step, one TMA box per (page, 64-wide half of head_dim), 128-byte swizzle)
//   warp 5     tensor-core issuer: S = Q K^T (tcgen05.mma, operands from shared memory, fp32 accumulator in
//              TMEM), then O += P V with P read from TMEM (bf16, written by the softmax warps over S) and V from
//              shared memory as an MN-major operand
// Tensor memory: columns [0,128) S (P aliases the first 64 as packed bf16), columns [128, 128+D) O.
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

constexpr int kSoftmaxThreads = 128;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColP = 0, kColO = 128;

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzled column blocks
    static constexpr int kTileBytes = 128 * D * 2;         // one Q, K or V tile
    static constexpr int kHalfBytes = 128 * 128;           // 128 rows x 128 bytes
    static constexpr int kStages = (D == 128) ? 3 : 4;
    static constexpr int kBarOff = kTileBytes * (1 + 2 * kStages);
    static constexpr int kNumBars = 5 + 4 * kStages;
    static constexpr int kSmemBytes = kBarOff + 8 * kNumBars + 16 + 1024;  // + tmem ptr/abort + alignment slack
};

struct Ring {
    uint32_t stage, phase;
    __device__ __forceinline__ void advance(uint32_t n) {
        if (++stage == n) { stage = 0; phase ^= 1u; }
    }
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
wpp_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + C::kTileBytes;
    const uint32_t sV = sK + C::kStages * C::kTileBytes;
    const uint32_t bars = smem_base + C::kBarOff;
    // barrier indices
    const uint32_t bQFull = bars, bQEmpty = bars + 8, bSFull = bars + 16, bPFull = bars + 24, bOFull = bars + 32;
    const uint32_t bKFull = bars + 40, bKEmpty = bKFull + 8 * C::kStages, bVFull = bKEmpty + 8 * C::kStages,
                   bVEmpty = bVFull + 8 * C::kStages;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::kBarOff + 8 * C::kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(bQFull, 1); mbar_init(bQEmpty, 1); mbar_init(bSFull, 1); mbar_init(bPFull, kSoftmaxThreads);
        mbar_init(bOFull, 1);
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(bKFull + 8 * s, 1); mbar_init(bKEmpty + 8 * s, 1);
            mbar_init(bVFull + 8 * s, 1); mbar_init(bVEmpty + 8 * s, 1);
        }
        *abort_flag = 0u;
        fence_barrier_init();
    }
    if (warp == 5) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
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
    const int tile_m = hd->tile_m;

    const int B = p.page_size, ppt = 128 / B;   // pages per key step

    if (warp == 4) {
        // ================================================================ producer
        Ring k_ring = {0, 0}, v_ring = {0, 0};
        uint32_t q_phase = 0;
        for (int u = u_begin; u < u_end; ++u) {
            const WppUnit un = units[u];
            if (un.kv_end <= un.kv_begin) continue;       // never planned; all roles skip it alike
            const int P = p.prefix_lens[un.request], Cn = p.chunk_lens[un.request];
            const int kv_len = P + Cn;
            const int n_pages = (kv_len + B - 1) / B;
            const int kvh = un.q_head / p.group;
            const int32_t* bt = p.block_tables + (int64_t)un.request * p.max_blocks;
            bool ok = mbar_wait(bQEmpty, q_phase ^ 1u, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(bQFull, C::kTileBytes);
                for (int h = 0; h < C::kHalves; ++h)
                    tma_load_3d(sQ + h * C::kHalfBytes, &tm_q, bQFull, h * 64, un.q_head,
                                q_offsets[un.request] + un.q_row0);
            }
            q_phase ^= 1u;
            bool dead = false;
            for (int j = un.kv_begin; j < un.kv_end; ++j) {
                const int page0 = j * ppt;
                const int cnt = min(ppt, n_pages - page0);
                // lane l holds the physical id of page page0 + l of this step
                int pid = 0;
                if (lane < cnt) {
                    pid = bt[page0 + lane];
                    if (pid < 0 || pid >= p.num_pages) {
                        if (p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                        pid = 0;
                    }
                }
                const uint32_t bytes = (uint32_t)cnt * B * D * 2;
                ok = mbar_wait(bKEmpty + 8 * k_ring.stage, k_ring.phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                if (lane == 0) mbar_arrive_expect_tx(bKFull + 8 * k_ring.stage, bytes);
                __syncwarp();
                if (lane < cnt) {
                    for (int h = 0; h < C::kHalves; ++h)
                        tma_load_4d(sK + k_ring.stage * C::kTileBytes + h * C::kHalfBytes + lane * B * 128, &tm_k,
                                    bKFull + 8 * k_ring.stage, h * 64, 0, kvh, pid);
                }
                k_ring.advance(C::kStages);
                ok = mbar_wait(bVEmpty + 8 * v_ring.stage, v_ring.phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                if (lane == 0) mbar_arrive_expect_tx(bVFull + 8 * v_ring.stage, bytes);
                __syncwarp();
                if (lane < cnt) {
                    for (int h = 0; h < C::kHalves; ++h)
                        tma_load_4d(sV + v_ring.stage * C::kTileBytes + h * C::kHalfBytes + lane * B * 128, &tm_v,
                                    bVFull + 8 * v_ring.stage, h * 64, 0, kvh, pid);
                }
                v_ring.advance(C::kStages);
            }
            if (dead) break;
        }
    } else if (warp == 5) {
        // ================================================================ tensor-core issuer
        Ring k_ring = {0, 0}, v_ring = {0, 0};
        uint32_t q_phase = 0, p_phase = 0;
        constexpr uint32_t idesc_qk = idesc_bf16(128, 0, 0);
        constexpr uint32_t idesc_pv = idesc_bf16(D, 0, 1);
        for (int u = u_begin; u < u_end; ++u) {
            const WppUnit un = units[u];
            if (un.kv_end <= un.kv_begin) continue;
            const int kv_len = p.prefix_lens[un.request] + p.chunk_lens[un.request];
            bool ok = mbar_wait(bQFull, q_phase, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            q_phase ^= 1u;
            bool dead = false;
            for (int j = un.kv_begin; j < un.kv_end; ++j) {
                // ---- S = Q K^T
                ok = mbar_wait(bKFull + 8 * k_ring.stage, k_ring.phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t kb = sK + k_ring.stage * C::kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * C::kHalfBytes + (kk & 3) * 32;
                        mma_ss(tmem + kColS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(kb + off, 16, 1024),
                               idesc_qk, kk > 0);
                    }
                    mma_commit(bSFull);
                    mma_commit(bKEmpty + 8 * k_ring.stage);
                }
                __syncwarp();
                k_ring.advance(C::kStages);
                // ---- O += P V
                ok = mbar_wait(bPFull, p_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                p_phase ^= 1u;
                ok = mbar_wait(bVFull + 8 * v_ring.stage, v_ring.phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                const uint32_t vb = sV + v_ring.stage * C::kTileBytes;
                const int valid = kv_len - j * 128;       // keys of this step that exist
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
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        mma_ts(tmem + kColO, tmem + kColP + kk * 8,
                               smem_desc_sw128(vb + kk * 2048, C::kHalfBytes, 1024), idesc_pv,
                               (j > un.kv_begin) || (kk > 0));
                    }
                    mma_commit(bOFull);
                    mma_commit(bVEmpty + 8 * v_ring.stage);
                    if (j == un.kv_end - 1) mma_commit(bQEmpty);
                }
                __syncwarp();
                v_ring.advance(C::kStages);
            }
            if (dead) break;
        }
    } else {
        // ================================================================ softmax + epilogue (thread = query row)
        const int r = threadIdx.x;
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        uint32_t s_phase = 0, o_phase = 0;
        const float c = p.scale_log2;
        for (int u = u_begin; u < u_end; ++u) {
            const WppUnit un = units[u];
            if (un.kv_end <= un.kv_begin) continue;
            const int P = p.prefix_lens[un.request];
            const int row_pos = P + un.q_row0 + r;          // last key this row may see
            float m_run = -INFINITY, l_run = 0.f;
            bool dead = false;
            for (int j = un.kv_begin; j < un.kv_end; ++j) {
                bool ok = mbar_wait(bSFull, s_phase, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                s_phase ^= 1u;
                tc_fence_after();
                float s[128];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(lane_addr + kColS + q4 * 32, reinterpret_cast<uint32_t*>(s) + q4 * 32);
                tmem_wait_ld();
                if (j * 128 + 127 > P + un.q_row0) {      // only steps that touch the diagonal are masked
                    const int limit = row_pos - j * 128;
#pragma unroll
                    for (int i = 0; i < 128; ++i) s[i] = (i > limit) ? -INFINITY : s[i];
                }
                float mx = s[0];
#pragma unroll
                for (int i = 1; i < 128; ++i) mx = fmaxf(mx, s[i]);
                const float m_new = fmaxf(m_run, mx);
                const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = fast_exp2((m_run - m_safe) * c);
                const float neg_mc = -m_safe * c;
                float sum = 0.f;
#pragma unroll
                for (int i = 0; i < 128; ++i) {
                    s[i] = fast_exp2(fmaf(s[i], c, neg_mc));
                    sum += s[i];
                }
                l_run = l_run * alpha + sum;
                m_run = m_new;
                if (j > un.kv_begin) {
                    ok = mbar_wait(bOFull, o_phase, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                    o_phase ^= 1u;
                    tc_fence_after();
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                        for (int q4 = 0; q4 < D / 32; ++q4) {
                            float o[32];
                            tmem_ld32(lane_addr + kColO + q4 * 32, reinterpret_cast<uint32_t*>(o));
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= alpha;
                            tmem_st32(lane_addr + kColO + q4 * 32, reinterpret_cast<uint32_t*>(o));
                        }
                    }
                }
                uint32_t pk[64];
#pragma unroll
                for (int i = 0; i < 64; ++i) pk[i] = pack_bf16x2(s[2 * i], s[2 * i + 1]);
                tmem_st32(lane_addr + kColP, pk);
                tmem_st32(lane_addr + kColP + 32, pk + 32);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bPFull);
            }
            if (dead) break;
            // ---- epilogue
            bool ok = mbar_wait(bOFull, o_phase, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            o_phase ^= 1u;
            tc_fence_after();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const bool row_ok = r < un.num_rows;
            const int64_t tok = (int64_t)q_offsets[un.request] + un.q_row0 + r;
            if (un.split_slot < 0) {
                __nv_bfloat16* dst = p.out + tok * p.o_token_stride + (int64_t)un.q_head * p.o_head_stride;
#pragma unroll
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    float o[32];
                    tmem_ld32(lane_addr + kColO + q4 * 32, reinterpret_cast<uint32_t*>(o));
                    tmem_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 w;
                            w.x = pack_bf16x2(o[8 * v + 0] * inv_l, o[8 * v + 1] * inv_l);
                            w.y = pack_bf16x2(o[8 * v + 2] * inv_l, o[8 * v + 3] * inv_l);
                            w.z = pack_bf16x2(o[8 * v + 4] * inv_l, o[8 * v + 5] * inv_l);
                            w.w = pack_bf16x2(o[8 * v + 6] * inv_l, o[8 * v + 7] * inv_l);
                            *reinterpret_cast<uint4*>(dst + q4 * 32 + v * 8) = w;
                        }
                    }
                }
                if (p.lse && row_ok)
                    p.lse[tok * p.num_q_heads + un.q_head] =
                        (l_run > 0.f) ? (m_run * c + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            } else {
                float* dst = p.ws_o + ((int64_t)un.split_slot * tile_m + r) * D;
#pragma unroll
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    float o[32];
                    tmem_ld32(lane_addr + kColO + q4 * 32, reinterpret_cast<uint32_t*>(o));
                    tmem_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            *reinterpret_cast<float4*>(dst + q4 * 32 + v * 4) =
                                make_float4(o[4 * v] * inv_l, o[4 * v + 1] * inv_l, o[4 * v + 2] * inv_l,
                                            o[4 * v + 3] * inv_l);
                    }
                }
                if (row_ok)
                    p.ws_lse[(int64_t)un.split_slot * tile_m + r] =
                        (l_run > 0.f) ? (m_run * c + log2f(l_run)) : -INFINITY;
            }
            tc_fence_before();
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
    if (warp == 5) {
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
