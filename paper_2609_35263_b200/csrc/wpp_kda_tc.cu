// Recurrent-state (KDA) layer of a chunk in its chunk-parallel form, on the tensor cores (Section 3.1 update, Section
// 3.2 snapshots).  Per request and head the update
//     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,     o_t = S_t^T q_t
// is rewritten over a block of tokens [a, b) that starts from the state S_0.  With S_0' = Diag(alpha_a) S_0 and the
// decay products G_t = prod_{a < r <= t} alpha_r (G_a = 1):
//     u_t  = beta_t (v_t - (Diag(alpha_t) S_{t-1})^T k_t)                       so that S_t = Diag(alpha_t) S_{t-1} + k_t u_t^T
//     S_t  = Diag(G_t) S_0' + sum_{s <= t} Diag(G_t / G_s) k_s u_s^T
// and, with Kt = K o G (rows k_t o G_t), Kh = K / G, Qt = Q o G, Kb = Kh o G_{b-1}:
//     A = tril(diag(beta) Kt Kh^T, -1),   (I + A) U = diag(beta) (V - Kt S_0'),   i.e.  U = T (V - Kt S_0'),  T = (I + A)^-1 diag(beta)
//     O = Qt S_0' + tril(Qt Kh^T) U,       S_b = Diag(G_{b-1}) S_0' + Kb^T U.
// Everything that does not involve the state is computed for all blocks in parallel by the PREPARATION kernel
// (one CTA per 64-token block and head: decay products, Kt, Kh, Qt, Kb, the products Kt Kh^T and Qt Kh^T on the tensor
// cores, the inverse of the unit lower triangular 64 x 64 matrix on CUDA cores) and left in a workspace; the CHAIN
// kernel (one CTA per request and head) then walks the blocks in order with five tensor-core products per block
// (Kt S_0', T (V - W), Qt S_0', M U, Kb^T U) and the 128 x 128 fp32 state resident in tensor memory.
//
// Precision.  The state must stay within 1e-4 of its largest element, which single bf16 operands (8 significant
// bits) cannot give.  Every operand is therefore split into two bf16 terms, x = hi + lo with hi = bf16(x) and lo =
// bf16(x - hi) (16 significant bits together), and every product is three MMAs: hi*hi + hi*lo + lo*hi (the dropped
// lo*lo term is below 2^-17 relative); accumulation is fp32 in tensor memory.
//
// Blocks are 64 consecutive sequence positions, aligned to absolute multiples of 64 (so a chunk split at such a
// position reproduces the unsplit result bit for bit).  A block is cut into sub-blocks, processed as steps of
// their own, wherever the state is needed (a periodic snapshot) and wherever a channel's decay product inside the
// block would fall below 2^-40: the token that causes it starts a new sub-block, where its own alpha is applied to
// the state directly instead of through a quotient G_t / G_s.  Decays of exactly 0 are therefore exact.
//
// Orientation on the tensor cores: everything is kept transposed, with the value dimension d_v = 128 on the 128
// rows (tensor-memory lanes): S^T [d_v x d_k], W^T = S_0'^T Kt^T [d_v x 64], U^T = (V - W)^T T^T, O^T = S_0'^T Qt^T +
// U^T M^T, S_b^T = Diag-scaled S_0'^T + U^T Kb.  Thread r of the chain warps owns row r: column r of the state.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/wpp.h"
#include "wpp_device.h"
#include "wpp_ptx.cuh"

namespace wpp {
namespace kdatc {

constexpr int kL = 64;                 // tokens per block
constexpr int kD = 128;                // d_k = d_v
constexpr float kMinGamma = 9.094947e-13f;   // 2^-40: smallest decay product a sub-block may contain
constexpr int kTileBytes = kL * 128;   // one 64-row x 128-byte swizzled tile (8 KB)

// hi/lo split of two fp32 values into two packed bf16 pairs (element 0 in the low half)
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    hi = pack_bf16x2(x0, x1);
    const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
    lo = pack_bf16x2(x0 - h0, x1 - h1);
}

// byte offset of 16-byte chunk j of row t inside a 128-byte-swizzled tile of 128-byte rows
__device__ __forceinline__ uint32_t sw_off(int t, int j) { return (uint32_t)(t * 128 + ((j ^ (t & 7)) << 4)); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
// plain (untiled) bulk copy global -> shared; both addresses and the size are multiples of 16 bytes
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void named_bar(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// The sub-block a token belongs to, from the block's cut mask (bit t set: token t starts a sub-block).
__device__ __forceinline__ int sub_start(uint64_t mask, int t) {
    const uint64_t below = mask & ((t >= 63) ? ~0ull : ((2ull << t) - 1ull));
    return 63 - __clzll((long long)below);
}
__device__ __forceinline__ int sub_end(uint64_t mask, int t, int hi) {     // exclusive
    const uint64_t above = (t >= 63) ? 0ull : (mask & ~((2ull << t) - 1ull));
    return above ? min(hi, __ffsll((long long)above) - 1) : hi;
}

// Geometry of a request's blocks.  Blocks are aligned to absolute sequence positions.
struct ReqBlocks {
    int64_t row0;       // first row of the request in the packed arrays
    int P, C;           // tokens already folded into the resumed state; chunk length
    int first_block;    // P / 64
    int n_blocks;
};
__device__ __forceinline__ ReqBlocks req_blocks(const KdaTcParams& p, int req) {
    ReqBlocks g;
    g.row0 = p.row_offsets[req];
    g.C = (int)(p.row_offsets[req + 1] - g.row0);
    g.P = p.prefix_lens ? p.prefix_lens[req] : 0;
    g.first_block = g.P / kL;
    g.n_blocks = g.C > 0 ? (g.P + g.C + kL - 1) / kL - g.first_block : 0;
    return g;
}

// ---------------------------------------------------------------------------------------------------------------
// Set-up: exclusive scan of the requests' block counts (one CTA).
__global__ void __launch_bounds__(1024) kda_tc_setup_kernel(const KdaTcParams p) {
    __shared__ int part[1024];
    const int R = p.num_requests, tid = threadIdx.x;
    const int per = (R + 1023) / 1024;
    const int i0 = min(R, tid * per), i1 = min(R, i0 + per);
    int sum = 0;
    for (int i = i0; i < i1; ++i) sum += req_blocks(p, i).n_blocks;
    part[tid] = sum;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
        const int v = tid >= o ? part[tid - o] : 0;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
    }
    int run = part[tid] - sum;
    for (int i = i0; i < i1; ++i) {
        p.blk_off[i] = run;
        run += req_blocks(p, i).n_blocks;
    }
    if (tid == 1023) p.blk_off[R] = part[1023];
}

// ---------------------------------------------------------------------------------------------------------------
// Preparation: one CTA (128 threads) per (block, head).
struct PrepSmem {
    static constexpr int kOffG = 0;                          // fp32 [64][128]: alpha, then decay products
    static constexpr int kOffA = kOffG + kL * kD * 4;        // Kt (later Qt) as MMA operand: hi0 hi1 lo0 lo1 tiles
    static constexpr int kOffB = kOffA + 4 * kTileBytes;     // Kh: hi0 hi1 lo0 lo1; later the triangular matrix (fp32)
    static constexpr int kOffMisc = kOffB + 4 * kTileBytes;  // beta[64], barrier, tmem slot, reduction scratch
    static constexpr int kBytes = kOffMisc + 1024 + 1024;    // + alignment slack
};

__global__ void __launch_bounds__(128) kda_tc_prep_kernel(const KdaTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    float* G = reinterpret_cast<float*>(sm + PrepSmem::kOffG);
    uint8_t* tileA = sm + PrepSmem::kOffA;
    uint8_t* tileB = sm + PrepSmem::kOffB;
    float* s_beta = reinterpret_cast<float*>(sm + PrepSmem::kOffMisc);              // [64]
    int* s_red = reinterpret_cast<int*>(sm + PrepSmem::kOffMisc + 256);             // [4]
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + PrepSmem::kOffMisc + 512);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    const uint32_t bar = base + PrepSmem::kOffMisc + 528;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.y, H = p.num_heads, R = p.num_requests;
    const int gb = blockIdx.x;
    if (gb >= p.blk_off[R]) return;
    int lo_r = 0, hi_r = R;                 // request: largest i with blk_off[i] <= gb (empty requests share offsets)
    while (hi_r - lo_r > 1) {
        const int mid = (lo_r + hi_r) >> 1;
        if (p.blk_off[mid] <= gb) lo_r = mid; else hi_r = mid;
    }
    const int req = lo_r;
    const ReqBlocks g = req_blocks(p, req);
    const int blk = g.first_block + (gb - p.blk_off[req]);
    const int t_lo = max(0, g.P - blk * kL), t_hi = min(kL, g.P + g.C - blk * kL);     // active tokens [t_lo, t_hi)
    const int64_t row_t0 = g.row0 + ((int64_t)blk * kL - g.P);                         // row of token 0 (may be < 0)
    const size_t bh = (size_t)gb * H + head;

    if (tid == 0) {
        mbar_init(bar, 1);
        *abort_flag = 0u;
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 128);
        tmem_relinquish();
    }
    // ---- alpha and beta of the block (inactive tokens: alpha 1, beta 0)
    for (int it = 0; it < 16; ++it) {
        const int item = it * 128 + tid, t = item >> 5, c4 = (item & 31) * 4;
        float4 a = make_float4(1.f, 1.f, 1.f, 1.f);
        if (t >= t_lo && t < t_hi) a = *reinterpret_cast<const float4*>(p.alpha + ((row_t0 + t) * H + head) * kD + c4);
        *reinterpret_cast<float4*>(G + t * kD + c4) = a;
    }
    if (tid < kL) s_beta[tid] = (tid >= t_lo && tid < t_hi) ? p.beta[(row_t0 + tid) * H + head] : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // ---- cuts.  A sub-block starts at the first active token, after every token that completes a periodic
    //      snapshot position, and at every token whose alpha would push a channel's decay product below 2^-40.
    uint64_t mask = 1ull << t_lo;
    if (p.snap_interval > 0) {
        for (int t = t_lo; t + 1 < t_hi; ++t)
            if (((int64_t)blk * kL + t + 1) % p.snap_interval == 0) mask |= 1ull << (t + 1);
    }
    for (int round = 0; round < kL; ++round) {
        // thread c follows channel c: the first token whose decay product (from its sub-block's start) is too small
        int first_bad = kL;
        float gacc = 1.f;
        for (int t = t_lo + 1; t < t_hi; ++t) {
            if ((mask >> t) & 1ull) { gacc = 1.f; continue; }
            gacc *= G[t * kD + tid];
            if (gacc < kMinGamma) { first_bad = t; break; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) first_bad = min(first_bad, __shfl_xor_sync(0xffffffffu, first_bad, o));
        if (lane == 0) s_red[warp] = first_bad;
        __syncthreads();
        first_bad = min(min(s_red[0], s_red[1]), min(s_red[2], s_red[3]));
        __syncthreads();
        if (first_bad >= kL) break;
        mask |= 1ull << first_bad;
    }
    // decay products in place of alpha; the last row of every sub-block goes to the workspace (the chain scales
    // the state by it)
    {
        float gacc = 1.f;
        for (int t = 0; t < kL; ++t) {
            if (t < t_lo || t >= t_hi) { G[t * kD + tid] = 1.f; continue; }
            gacc = ((mask >> t) & 1ull) ? 1.f : gacc * G[t * kD + tid];
            G[t * kD + tid] = gacc;
            if (t + 1 == t_hi || ((mask >> (t + 1)) & 1ull)) p.ws_e[(bh * kL + t) * kD + tid] = gacc;
        }
    }
    if (tid == 0) p.ws_mask[bh] = mask;
    __syncthreads();

    // ---- Kt = k G, Kh = k / G, Kb = Kh G_end as hi/lo bf16: Kt and Kh to shared memory (MMA operands), Kt and Kb
    //      to the workspace.  A thread handles 8 consecutive channels of a token at a time.
    const size_t tile_elems = (size_t)kL * kD;
    for (int it = 0; it < 8; ++it) {
        const int item = it * 128 + tid, t = item >> 4, ch = item & 15, c0 = ch * 8;
        const bool active = t >= t_lo && t < t_hi;
        uint4 kt_h = make_uint4(0, 0, 0, 0), kt_l = kt_h, kh_h = kt_h, kh_l = kt_h, kb_h = kt_h, kb_l = kt_h;
        if (active) {
            const uint4 raw = *reinterpret_cast<const uint4*>(p.k + ((row_t0 + t) * H + head) * kD + c0);
            const int e_t = sub_end(mask, t, t_hi) - 1;
            const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t o[6][4];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float k0 = __uint_as_float(rw[w] << 16), k1 = __uint_as_float(rw[w] & 0xffff0000u);
                const float g0 = G[t * kD + c0 + 2 * w], g1 = G[t * kD + c0 + 2 * w + 1];
                const float e0 = G[e_t * kD + c0 + 2 * w], e1 = G[e_t * kD + c0 + 2 * w + 1];
                split2(k0 * g0, k1 * g1, o[0][w], o[1][w]);
                split2(k0 / g0, k1 / g1, o[2][w], o[3][w]);
                split2(k0 * (e0 / g0), k1 * (e1 / g1), o[4][w], o[5][w]);
            }
            kt_h = make_uint4(o[0][0], o[0][1], o[0][2], o[0][3]); kt_l = make_uint4(o[1][0], o[1][1], o[1][2], o[1][3]);
            kh_h = make_uint4(o[2][0], o[2][1], o[2][2], o[2][3]); kh_l = make_uint4(o[3][0], o[3][1], o[3][2], o[3][3]);
            kb_h = make_uint4(o[4][0], o[4][1], o[4][2], o[4][3]); kb_l = make_uint4(o[5][0], o[5][1], o[5][2], o[5][3]);
        }
        const uint32_t off = (uint32_t)((ch >> 3) * kTileBytes) + sw_off(t, ch & 7);
        *reinterpret_cast<uint4*>(tileA + off) = kt_h;
        *reinterpret_cast<uint4*>(tileA + 2 * kTileBytes + off) = kt_l;
        *reinterpret_cast<uint4*>(tileB + off) = kh_h;
        *reinterpret_cast<uint4*>(tileB + 2 * kTileBytes + off) = kh_l;
        const size_t go = bh * tile_elems + (size_t)t * kD + c0;
        *reinterpret_cast<uint4*>(p.ws_kt_h + go) = kt_h;
        *reinterpret_cast<uint4*>(p.ws_kt_l + go) = kt_l;
        *reinterpret_cast<uint4*>(p.ws_kb_h + go) = kb_h;
        *reinterpret_cast<uint4*>(p.ws_kb_l + go) = kb_l;
    }
    fence_proxy_async_smem();
    __syncthreads();

    // D[128 x 64] (rows 64.. are never read: the A tiles have 64 rows, the rows after them are whatever follows in
    // shared memory) = A (hi + lo) x B (hi + lo)^T without the lo x lo term
    constexpr uint32_t idesc = idesc_bf16(64, 0, 0);
    auto issue_product = [&](uint32_t d_col) {
        const uint32_t a_hi = base + PrepSmem::kOffA, a_lo = a_hi + 2 * kTileBytes;
        const uint32_t b_hi = base + PrepSmem::kOffB, b_lo = b_hi + 2 * kTileBytes;
        const uint32_t aa[3] = {a_hi, a_hi, a_lo}, bb[3] = {b_hi, b_lo, b_hi};
        bool first = true;
#pragma unroll
        for (int term = 0; term < 3; ++term) {
            const uint64_t ad = smem_desc_sw128(aa[term], 16, 1024), bd = smem_desc_sw128(bb[term], 16, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint64_t off = (uint64_t)(((kk >> 2) * kTileBytes + (kk & 3) * 32) >> 4);
                mma_ss(tmem + d_col, ad + off, bd + off, idesc, first ? 0u : 1u);
                first = false;
            }
        }
        mma_commit(bar);
    };
    if (tid == 0) {
        tc_fence_after();
        issue_product(0);
    }
    bool ok = mbar_wait(bar, 0, abort_flag);

    // ---- Qt = q G over the Kt tiles (the first product has completed), also to the workspace
    for (int it = 0; it < 8 && ok; ++it) {
        const int item = it * 128 + tid, t = item >> 4, ch = item & 15, c0 = ch * 8;
        uint4 q_h = make_uint4(0, 0, 0, 0), q_l = q_h;
        if (t >= t_lo && t < t_hi) {
            const uint4 raw = *reinterpret_cast<const uint4*>(p.q + ((row_t0 + t) * H + head) * kD + c0);
            const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t o[2][4];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float q0 = __uint_as_float(rw[w] << 16), q1 = __uint_as_float(rw[w] & 0xffff0000u);
                split2(q0 * G[t * kD + c0 + 2 * w], q1 * G[t * kD + c0 + 2 * w + 1], o[0][w], o[1][w]);
            }
            q_h = make_uint4(o[0][0], o[0][1], o[0][2], o[0][3]);
            q_l = make_uint4(o[1][0], o[1][1], o[1][2], o[1][3]);
        }
        const uint32_t off = (uint32_t)((ch >> 3) * kTileBytes) + sw_off(t, ch & 7);
        *reinterpret_cast<uint4*>(tileA + off) = q_h;
        *reinterpret_cast<uint4*>(tileA + 2 * kTileBytes + off) = q_l;
        const size_t go = bh * tile_elems + (size_t)t * kD + c0;
        *reinterpret_cast<uint4*>(p.ws_qt_h + go) = q_h;
        *reinterpret_cast<uint4*>(p.ws_qt_l + go) = q_l;
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) {
        tc_fence_after();
        issue_product(64);
    }
    ok = ok && mbar_wait(bar, 1, abort_flag);
    tc_fence_after();

    // ---- rows of the two products (thread t < 64 owns token t = tensor-memory lane t).  The triangular matrix goes
    //      to shared memory (over the Kh tiles: both products have completed), M = tril(Qt Kh^T) to the workspace.
    float* Amat = reinterpret_cast<float*>(tileB);          // [64][64] fp32: beta_t (Kt Kh^T)[t][s] for s < t in the sub-block
    if (warp < 2 && ok) {
        const int t = tid;
        const bool active = t >= t_lo && t < t_hi;
        const int s0 = active ? sub_start(mask, t) : kL;    // columns [s0, t) (and t itself for M) count
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        const float bt = s_beta[t];
        float x[32];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            tmem_ld32(lane_addr + half * 32, reinterpret_cast<uint32_t*>(x));
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int s = half * 32 + i;
                Amat[t * kL + s] = (active && s >= s0 && s < t) ? bt * x[i] : 0.f;
            }
        }
        __nv_bfloat16* mh = p.ws_m_h + (bh * kL + t) * kL;
        __nv_bfloat16* ml = p.ws_m_l + (bh * kL + t) * kL;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            tmem_ld32(lane_addr + 64 + half * 32, reinterpret_cast<uint32_t*>(x));
            tmem_wait_ld();
            uint32_t oh[16], ol[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int s = half * 32 + 2 * i;
                const float m0 = (active && s >= s0 && s <= t) ? x[2 * i] : 0.f;
                const float m1 = (active && s + 1 >= s0 && s + 1 <= t) ? x[2 * i + 1] : 0.f;
                split2(m0, m1, oh[i], ol[i]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                *reinterpret_cast<uint4*>(mh + half * 32 + i * 8) = make_uint4(oh[4 * i], oh[4 * i + 1], oh[4 * i + 2], oh[4 * i + 3]);
                *reinterpret_cast<uint4*>(ml + half * 32 + i * 8) = make_uint4(ol[4 * i], ol[4 * i + 1], ol[4 * i + 2], ol[4 * i + 3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, 128);
    }
    if (!ok) {
        if (tid == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_TIMEOUT);
        return;
    }
    // ---- T = (I + A)^-1 diag(beta) by forward substitution: thread c owns column c (T[t][c] = 0 for t < c)
    if (tid < kL) {
        const int c = tid;
        float Tc[kL];
#pragma unroll
        for (int t = 0; t < kL; ++t) {
            float acc = (t == c) ? s_beta[t] : 0.f;
            const float4* arow = reinterpret_cast<const float4*>(Amat + t * kL);
#pragma unroll
            for (int s4 = 0; s4 < (t + 3) / 4; ++s4) {
                const float4 a = arow[s4];
                if (4 * s4 + 0 < t) acc = fmaf(-a.x, Tc[4 * s4 + 0], acc);
                if (4 * s4 + 1 < t) acc = fmaf(-a.y, Tc[4 * s4 + 1], acc);
                if (4 * s4 + 2 < t) acc = fmaf(-a.z, Tc[4 * s4 + 2], acc);
                if (4 * s4 + 3 < t) acc = fmaf(-a.w, Tc[4 * s4 + 3], acc);
            }
            Tc[t] = acc;
        }
        __nv_bfloat16* th = p.ws_t_h + bh * kL * kL + c;
        __nv_bfloat16* tl = p.ws_t_l + bh * kL * kL + c;
#pragma unroll
        for (int t = 0; t < kL; ++t) {
            const __nv_bfloat16 h = __float2bfloat16_rn(Tc[t]);
            th[t * kL] = h;
            tl[t * kL] = __float2bfloat16_rn(Tc[t] - __bfloat162float(h));
        }
    }
}

// ---------------------------------------------------------------------------------------------------------------
// Chain: one CTA per (request, head).  Warps 0-3: the state's rows (thread r = tensor-memory lane r = column r of S);
// warps 4-7: output epilogue; warp 8: producer (TMA loads of the block's operands, step records); warp 9: one thread
// issues the MMAs.
constexpr int kStepRing = 4;
struct Ring {
    uint32_t stage, phase;
    __device__ __forceinline__ void advance(uint32_t n) {
        if (++stage == n) { stage = 0; phase ^= 1u; }
    }
};
struct StepRec {
    int a, b;            // tokens [a, b) of the block; a < 0: no more steps
    int first, last;     // first / last step of its block (operand buffers are acquired / released there)
    int store_slot;      // state slot to write after the step (periodic snapshot or the chunk's end), or -1
    int pad[3];
    int64_t row_t0;      // row of the block's token 0 in the packed arrays
};
struct ChainSmem {
    // operand tiles of one block, each a pair (hi, lo); 128-channel operands have two 64-column tiles per part
    static constexpr int kOffKt = 0;                          // hi0 hi1 lo0 lo1
    static constexpr int kOffQt = kOffKt + 4 * kTileBytes;
    static constexpr int kOffKb = kOffQt + 4 * kTileBytes;
    static constexpr int kOffT = kOffKb + 4 * kTileBytes;     // hi lo
    static constexpr int kOffM = kOffT + 2 * kTileBytes;
    static constexpr int kOffV = kOffM + 2 * kTileBytes;      // two 64-column tiles
    static constexpr int kOffVec = kOffV + 2 * kTileBytes;    // per ring slot: alpha of the step's first token, decay product at its end
    static constexpr int kOffRec = kOffVec + kStepRing * 2 * kD * 4;
    static constexpr int kOffBars = kOffRec + kStepRing * (int)sizeof(StepRec);
    static constexpr int kNumBars = 2 * kStepRing + 12 + 8;
    static constexpr int kOffMisc = kOffBars + 8 * kNumBars;
    static constexpr int kBytes = kOffMisc + 64 + 1024;
};
// tensor-memory columns
constexpr uint32_t kColS = 0, kColShl = 128, kColWU = 256, kColRU = 320, kColO = 384;

__global__ void __launch_bounds__(320, 1)
kda_tc_chain_kernel(const __grid_constant__ CUtensorMap tm_kt_h, const __grid_constant__ CUtensorMap tm_kt_l,
                    const __grid_constant__ CUtensorMap tm_qt_h, const __grid_constant__ CUtensorMap tm_qt_l,
                    const __grid_constant__ CUtensorMap tm_kb_h, const __grid_constant__ CUtensorMap tm_kb_l,
                    const __grid_constant__ CUtensorMap tm_t_h, const __grid_constant__ CUtensorMap tm_t_l,
                    const __grid_constant__ CUtensorMap tm_m_h, const __grid_constant__ CUtensorMap tm_m_l,
                    const __grid_constant__ CUtensorMap tm_v, const KdaTcParams p) {
    using CS = ChainSmem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + CS::kOffBars;
    auto bStepFull = [&](int s) { return bars + 8 * s; };
    auto bStepEmpty = [&](int s) { return bars + 8 * (kStepRing + s); };
    const uint32_t b0 = bars + 16 * kStepRing;
    // operand buffers (one block in flight each): full / empty
    const uint32_t bKtFull = b0, bKtEmpty = b0 + 8, bQtFull = b0 + 16, bQtEmpty = b0 + 24, bKbFull = b0 + 32,
                   bKbEmpty = b0 + 40, bTFull = b0 + 48, bTEmpty = b0 + 56, bMFull = b0 + 64, bMEmpty = b0 + 72,
                   bVFull = b0 + 80, bVEmpty = b0 + 88;
    const uint32_t b1 = b0 + 96;
    const uint32_t bShlReady = b1, bWReady = b1 + 8, bRhsReady = b1 + 16, bUReady = b1 + 24, bUhlReady = b1 + 32,
                   bSReady = b1 + 40, bOReady = b1 + 48, bOFree = b1 + 56;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + CS::kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* s_vec = reinterpret_cast<float*>(sm + CS::kOffVec);
    volatile StepRec* s_rec = reinterpret_cast<volatile StepRec*>(sm + CS::kOffRec);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.x, req = blockIdx.y, H = p.num_heads;
    const ReqBlocks g = req_blocks(p, req);

    // slot ids: anything outside [-1, num_slots) is reported and treated as -1
    int slot_in = p.state_in[req], slot_out = p.state_out[req];
    if (slot_in < -1 || slot_in >= p.num_slots || slot_out < -1 || slot_out >= p.num_slots) {
        if (p.status && tid == 0) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
        if (slot_in < -1 || slot_in >= p.num_slots) slot_in = -1;
        if (slot_out < -1 || slot_out >= p.num_slots) slot_out = -1;
    }
    const size_t head_floats = (size_t)kD * kD;
    if (g.C == 0) {
        // an empty chunk copies the state
        if (slot_out >= 0 && slot_out != slot_in) {
            float4* dst = reinterpret_cast<float4*>(p.state_pool + ((size_t)slot_out * H + head) * head_floats);
            const float4* src = slot_in >= 0
                ? reinterpret_cast<const float4*>(p.state_pool + ((size_t)slot_in * H + head) * head_floats) : nullptr;
            for (int i = tid; i < (int)(head_floats / 4); i += blockDim.x) dst[i] = src ? src[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        return;
    }

    if (tid == 0) {
        for (int s = 0; s < kStepRing; ++s) { mbar_init(bStepFull(s), 1); mbar_init(bStepEmpty(s), 128 + 128 + 1); }
        for (int i = 0; i < 5; ++i) { mbar_init(b0 + 16 * i, 1); mbar_init(b0 + 16 * i + 8, 1); }
        mbar_init(bVFull, 1);
        mbar_init(bVEmpty, 128);          // the value tile is released by the 128 row threads
        mbar_init(bShlReady, 128); mbar_init(bWReady, 1); mbar_init(bRhsReady, 128); mbar_init(bUReady, 1);
        mbar_init(bUhlReady, 128); mbar_init(bSReady, 1); mbar_init(bOReady, 1); mbar_init(bOFree, 128);
        *abort_flag = 0u;
        fence_barrier_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int gb0 = p.blk_off[req];

    if (warp == 8) {
        // ================================================================ producer
        uint32_t ph_e[6] = {0, 0, 0, 0, 0, 0};      // parity of the operand buffers' empty barriers (Kt Qt Kb T M V)
        Ring step = {0, 0};
        bool dead = false;
        // periodic snapshots: next sequence position at which one is due
        const int interval = p.snap_interval;
        int64_t next_snap = interval > 0 ? ((int64_t)g.P / interval + 1) * interval : -1;
        int n_snap = 0;
        for (int b = 0; b <= g.n_blocks && !dead; ++b) {
            if (b == g.n_blocks) {      // terminal record
                const bool okw = mbar_wait(bStepEmpty(step.stage), step.phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, okw)) break;
                if (lane == 0) {
                    s_rec[step.stage].a = -1;
                    mbar_arrive(bStepFull(step.stage));
                }
                break;
            }
            const int blk = g.first_block + b;
            const size_t bh = (size_t)(gb0 + b) * H + head;
            const int t_lo = max(0, g.P - blk * kL), t_hi = min(kL, g.P + g.C - blk * kL);
            const int64_t row_t0 = g.row0 + ((int64_t)blk * kL - g.P);
            // ---- operand loads of the block: each waits for its buffer (lanes 0..5 own one buffer each)
            {
                bool okw = true;
                if (lane < 6) okw = mbar_wait(b0 + 16 * lane + 8, ph_e[lane] ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, okw)) { dead = true; break; }
#pragma unroll
                for (int i = 0; i < 6; ++i) ph_e[i] ^= 1u;
                const int row = (int)(bh * kL);
                if (lane == 0) {
                    mbar_arrive_expect_tx(bKtFull, 4 * kTileBytes);
                    tma_load_2d(base + CS::kOffKt, &tm_kt_h, bKtFull, 0, row);
                    tma_load_2d(base + CS::kOffKt + kTileBytes, &tm_kt_h, bKtFull, 64, row);
                    tma_load_2d(base + CS::kOffKt + 2 * kTileBytes, &tm_kt_l, bKtFull, 0, row);
                    tma_load_2d(base + CS::kOffKt + 3 * kTileBytes, &tm_kt_l, bKtFull, 64, row);
                } else if (lane == 1) {
                    mbar_arrive_expect_tx(bQtFull, 4 * kTileBytes);
                    tma_load_2d(base + CS::kOffQt, &tm_qt_h, bQtFull, 0, row);
                    tma_load_2d(base + CS::kOffQt + kTileBytes, &tm_qt_h, bQtFull, 64, row);
                    tma_load_2d(base + CS::kOffQt + 2 * kTileBytes, &tm_qt_l, bQtFull, 0, row);
                    tma_load_2d(base + CS::kOffQt + 3 * kTileBytes, &tm_qt_l, bQtFull, 64, row);
                } else if (lane == 2) {
                    mbar_arrive_expect_tx(bKbFull, 4 * kTileBytes);
                    tma_load_2d(base + CS::kOffKb, &tm_kb_h, bKbFull, 0, row);
                    tma_load_2d(base + CS::kOffKb + kTileBytes, &tm_kb_h, bKbFull, 64, row);
                    tma_load_2d(base + CS::kOffKb + 2 * kTileBytes, &tm_kb_l, bKbFull, 0, row);
                    tma_load_2d(base + CS::kOffKb + 3 * kTileBytes, &tm_kb_l, bKbFull, 64, row);
                } else if (lane == 3) {
                    mbar_arrive_expect_tx(bTFull, 2 * kTileBytes);
                    tma_load_2d(base + CS::kOffT, &tm_t_h, bTFull, 0, row);
                    tma_load_2d(base + CS::kOffT + kTileBytes, &tm_t_l, bTFull, 0, row);
                } else if (lane == 4) {
                    mbar_arrive_expect_tx(bMFull, 2 * kTileBytes);
                    tma_load_2d(base + CS::kOffM, &tm_m_h, bMFull, 0, row);
                    tma_load_2d(base + CS::kOffM + kTileBytes, &tm_m_l, bMFull, 0, row);
                } else if (lane == 5) {
                    mbar_arrive_expect_tx(bVFull, 2 * kTileBytes);
                    tma_load_3d(base + CS::kOffV, &tm_v, bVFull, 0, head, (int)row_t0);
                    tma_load_3d(base + CS::kOffV + kTileBytes, &tm_v, bVFull, 64, head, (int)row_t0);
                }
            }
            // ---- the block's steps
            uint64_t mask = 0;
            if (lane == 0) mask = p.ws_mask[bh];
            mask = __shfl_sync(0xffffffffu, mask, 0);
            int a = t_lo;
            while (a < t_hi && !dead) {
                const int e = sub_end(mask, a, t_hi);
                const bool okw = mbar_wait(bStepEmpty(step.stage), step.phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, okw)) { dead = true; break; }
                if (lane == 0) {
                    volatile StepRec& r = s_rec[step.stage];
                    r.a = a; r.b = e; r.first = (a == t_lo); r.last = (e == t_hi); r.row_t0 = row_t0;
                    int store = -1;
                    const int64_t pos_end = (int64_t)blk * kL + e;            // tokens folded into S after the step
                    if (interval > 0 && pos_end == next_snap) {
                        if (p.snap_slots && n_snap < p.max_snaps) {
                            const int slot = p.snap_slots[(size_t)req * p.max_snaps + n_snap];
                            if (slot >= 0 && slot < p.num_slots) store = slot;
                            else if (slot != -1 && p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                        }
                        ++n_snap;
                        next_snap += interval;
                    }
                    r.store_slot = store;
                    // the step's two vectors: alpha of its first token, the decay product at its last token
                    mbar_arrive_expect_tx(bStepFull(step.stage), 2 * kD * 4);
                    const uint32_t dst = base + CS::kOffVec + step.stage * 2 * kD * 4;
                    bulk_load(dst, p.alpha + ((row_t0 + a) * H + head) * kD, kD * 4, bStepFull(step.stage));
                    bulk_load(dst + kD * 4, p.ws_e + (bh * kL + (e - 1)) * kD, kD * 4, bStepFull(step.stage));
                }
                step.advance(kStepRing);
                a = e;
            }
        }
    } else if (warp == 9 && lane == 0) {
        // ================================================================ MMA issuer
        Ring step = {0, 0};
        uint32_t ph_kt = 0, ph_qt = 0, ph_kb = 0, ph_t = 0, ph_m = 0;
        uint32_t ph_shl = 0, ph_rhs = 0, ph_uhl = 0, ph_ofree = 0;
        constexpr uint32_t idesc64 = idesc_bf16(64, 0, 0), idesc128mn = idesc_bf16(128, 0, 1);
        const uint32_t tS = tmem + kColS, tShl = tmem + kColShl, tWU = tmem + kColWU, tRU = tmem + kColRU, tO = tmem + kColO;
        // A (hi + lo, in tensor memory, `acols` columns per part) x B^T (hi + lo tiles in shared memory, K-major)
        auto product_k = [&](uint32_t d, uint32_t a_tm, uint32_t acols, uint32_t b_hi, uint32_t b_lo, int ksteps, bool overwrite) {
            const uint32_t aa[3] = {a_tm, a_tm, a_tm + acols}, bb[3] = {b_hi, b_lo, b_hi};
            bool first = overwrite;
            for (int term = 0; term < 3; ++term) {
                const uint64_t bd = smem_desc_sw128(bb[term], 16, 1024);
                for (int kk = 0; kk < ksteps; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * kTileBytes + (kk & 3) * 32) >> 4);
                    mma_ts(d, aa[term] + kk * 8, bd + off, idesc64, first ? 0u : 1u);
                    first = false;
                }
            }
        };
        bool dead = false;
        bool first_step = true;
        while (!dead) {
            if (!mbar_wait(bStepFull(step.stage), step.phase, abort_flag)) break;
            const int a = s_rec[step.stage].a;
            const bool first = s_rec[step.stage].first, last = s_rec[step.stage].last;
            mbar_arrive(bStepEmpty(step.stage));
            step.advance(kStepRing);
            if (a < 0) break;
            // ---- W^T = S_0'^T Kt^T
            if (!mbar_wait(bShlReady, ph_shl, abort_flag)) break;
            ph_shl ^= 1u;
            if (first) { if (!mbar_wait(bKtFull, ph_kt, abort_flag)) break; ph_kt ^= 1u; }
            tc_fence_after();
            product_k(tWU, tShl, 64, base + CS::kOffKt, base + CS::kOffKt + 2 * kTileBytes, 8, true);
            mma_commit(bWReady);
            if (last) mma_commit(bKtEmpty);
            // ---- U^T = (V - W)^T T^T
            if (!mbar_wait(bRhsReady, ph_rhs, abort_flag)) break;
            ph_rhs ^= 1u;
            if (first) { if (!mbar_wait(bTFull, ph_t, abort_flag)) break; ph_t ^= 1u; }
            tc_fence_after();
            product_k(tWU, tRU, 32, base + CS::kOffT, base + CS::kOffT + kTileBytes, 4, true);
            mma_commit(bUReady);
            if (last) mma_commit(bTEmpty);
            // ---- O^T = S_0'^T Qt^T (the previous step's output must have been read out)
            if (!first_step) { if (!mbar_wait(bOFree, ph_ofree, abort_flag)) break; ph_ofree ^= 1u; }
            first_step = false;
            if (first) { if (!mbar_wait(bQtFull, ph_qt, abort_flag)) break; ph_qt ^= 1u; }
            tc_fence_after();
            product_k(tO, tShl, 64, base + CS::kOffQt, base + CS::kOffQt + 2 * kTileBytes, 8, true);
            // ---- S_b^T += U^T Kb   (the accumulator was preset to the decayed S_0'),   O^T += U^T M^T
            if (!mbar_wait(bUhlReady, ph_uhl, abort_flag)) break;
            ph_uhl ^= 1u;
            if (first) { if (!mbar_wait(bKbFull, ph_kb, abort_flag)) break; ph_kb ^= 1u; }
            tc_fence_after();
            {
                const uint32_t kb_hi = base + CS::kOffKb, kb_lo = kb_hi + 2 * kTileBytes;
                const uint32_t aa[3] = {tRU, tRU, tRU + 32}, bb[3] = {kb_hi, kb_lo, kb_hi};
                for (int term = 0; term < 3; ++term) {
                    const uint64_t bd = smem_desc_sw128(bb[term], kTileBytes, 1024);      // MN-major: 64-column halves kTileBytes apart
                    for (int kk = 0; kk < 4; ++kk) mma_ts(tS, aa[term] + kk * 8, bd + (uint64_t)(kk * 128), idesc128mn, 1u);
                }
            }
            mma_commit(bSReady);
            if (last) mma_commit(bKbEmpty);
            if (first) { if (!mbar_wait(bMFull, ph_m, abort_flag)) break; ph_m ^= 1u; }
            product_k(tO, tRU, 32, base + CS::kOffM, base + CS::kOffM + kTileBytes, 4, false);
            mma_commit(bOReady);
            if (last) { mma_commit(bQtEmpty); mma_commit(bMEmpty); }
        }
    } else if (warp >= 4 && warp < 8) {
        // ================================================================ output epilogue (thread = value column r)
        const int r = tid - 128;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        Ring step = {0, 0};
        uint32_t ph_o = 0;
        while (true) {
            const bool okw = mbar_wait(bStepFull(step.stage), step.phase, abort_flag);
            if (!__all_sync(0xffffffffu, okw)) break;
            const int a = s_rec[step.stage].a, b = s_rec[step.stage].b;
            const int64_t row_t0 = s_rec[step.stage].row_t0;
            mbar_arrive(bStepEmpty(step.stage));
            step.advance(kStepRing);
            if (a < 0) break;
            const bool oko = mbar_wait(bOReady, ph_o, abort_flag);
            if (!__all_sync(0xffffffffu, oko)) break;
            ph_o ^= 1u;
            tc_fence_after();
            float o[64];
            tmem_ld32(lane_addr + kColO, reinterpret_cast<uint32_t*>(o));
            tmem_ld32(lane_addr + kColO + 32, reinterpret_cast<uint32_t*>(o) + 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bOFree);
#pragma unroll
            for (int t = 0; t < kL; ++t)
                if (t >= a && t < b) p.out[((row_t0 + t) * H + head) * kD + r] = __float2bfloat16_rn(o[t]);
        }
    } else if (warp < 4) {
        // ================================================================ the state's rows (thread r = column r of S)
        const int r = tid;
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        // initial state: S[c][r] for all c
        {
            const float* src = slot_in >= 0 ? p.state_pool + ((size_t)slot_in * H + head) * head_floats + r : nullptr;
#pragma unroll 1
            for (int c0 = 0; c0 < kD; c0 += 32) {
                float x[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) x[i] = src ? src[(size_t)(c0 + i) * kD] : 0.f;
                tmem_st32(lane_addr + kColS + c0, reinterpret_cast<const uint32_t*>(x));
            }
            tmem_wait_st();
        }
        auto store_state = [&](int slot) {
            float* dst = p.state_pool + ((size_t)slot * H + head) * head_floats + r;
#pragma unroll 1
            for (int c0 = 0; c0 < kD; c0 += 32) {
                float x[32];
                tmem_ld32(lane_addr + kColS + c0, reinterpret_cast<uint32_t*>(x));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) dst[(size_t)(c0 + i) * kD] = x[i];
            }
        };
        Ring step = {0, 0};
        uint32_t ph_w = 0, ph_u = 0, ph_s = 0, ph_v = 0;
        bool s_pending = false;          // an S_b product is in flight: wait for it before touching S
        bool dead = false;
        const uint8_t* vt = sm + CS::kOffV + (r >> 6) * kTileBytes;
        const int vj = (r & 63) >> 3, vb = (r & 7) * 2;
        while (!dead) {
            const bool okw = mbar_wait(bStepFull(step.stage), step.phase, abort_flag);
            if (!__all_sync(0xffffffffu, okw)) { dead = true; break; }
            const int slot_ring = step.stage;
            const int a = s_rec[slot_ring].a, b = s_rec[slot_ring].b;
            const bool first = s_rec[slot_ring].first, last = s_rec[slot_ring].last;
            const int store_slot = s_rec[slot_ring].store_slot;
            if (a < 0) { mbar_arrive(bStepEmpty(slot_ring)); break; }
            const float* v_alpha = s_vec + slot_ring * 2 * kD;
            const float* v_end = v_alpha + kD;
            // ---- S_0' = alpha_a o S_0 as the hi/lo operand, and Diag(G_end) S_0' as the accumulator of S_b
            if (s_pending) {
                const bool oks = mbar_wait(bSReady, ph_s, abort_flag);
                if (!__all_sync(0xffffffffu, oks)) { dead = true; break; }
                ph_s ^= 1u;
                s_pending = false;
            }
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < kD; c0 += 32) {
                float x[32];
                uint32_t hi[16], lo[16];
                tmem_ld32(lane_addr + kColS + c0, reinterpret_cast<uint32_t*>(x));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float y0 = x[2 * i] * v_alpha[c0 + 2 * i], y1 = x[2 * i + 1] * v_alpha[c0 + 2 * i + 1];
                    split2(y0, y1, hi[i], lo[i]);
                    x[2 * i] = y0 * v_end[c0 + 2 * i];
                    x[2 * i + 1] = y1 * v_end[c0 + 2 * i + 1];
                }
                tmem_st32(lane_addr + kColS + c0, reinterpret_cast<const uint32_t*>(x));
                tmem_st8(lane_addr + kColShl + c0 / 2, hi);
                tmem_st8(lane_addr + kColShl + c0 / 2 + 8, hi + 8);
                tmem_st8(lane_addr + kColShl + 64 + c0 / 2, lo);
                tmem_st8(lane_addr + kColShl + 64 + c0 / 2 + 8, lo + 8);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bShlReady);
            mbar_arrive(bStepEmpty(slot_ring));      // the record and its vectors have been consumed
            // ---- (V - W)^T for the step's tokens, zero elsewhere
            if (first) {
                const bool okv = mbar_wait(bVFull, ph_v, abort_flag);
                if (!__all_sync(0xffffffffu, okv)) { dead = true; break; }
                ph_v ^= 1u;
            }
            {
                const bool okw2 = mbar_wait(bWReady, ph_w, abort_flag);
                if (!__all_sync(0xffffffffu, okw2)) { dead = true; break; }
                ph_w ^= 1u;
            }
            tc_fence_after();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float x[32];
                uint32_t hi[16], lo[16];
                tmem_ld32(lane_addr + kColWU + half * 32, reinterpret_cast<uint32_t*>(x));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float rr[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int t = half * 32 + 2 * i + e;
                        const float vv = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vt + sw_off(t, vj) + vb));
                        rr[e] = (t >= a && t < b) ? vv - x[2 * i + e] : 0.f;
                    }
                    split2(rr[0], rr[1], hi[i], lo[i]);
                }
                tmem_st8(lane_addr + kColRU + half * 16, hi);
                tmem_st8(lane_addr + kColRU + half * 16 + 8, hi + 8);
                tmem_st8(lane_addr + kColRU + 32 + half * 16, lo);
                tmem_st8(lane_addr + kColRU + 32 + half * 16 + 8, lo + 8);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bRhsReady);
            if (last) mbar_arrive(bVEmpty);
            // ---- U^T as the hi/lo operand
            {
                const bool oku = mbar_wait(bUReady, ph_u, abort_flag);
                if (!__all_sync(0xffffffffu, oku)) { dead = true; break; }
                ph_u ^= 1u;
            }
            tc_fence_after();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float x[32];
                uint32_t hi[16], lo[16];
                tmem_ld32(lane_addr + kColWU + half * 32, reinterpret_cast<uint32_t*>(x));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) split2(x[2 * i], x[2 * i + 1], hi[i], lo[i]);
                tmem_st8(lane_addr + kColRU + half * 16, hi);
                tmem_st8(lane_addr + kColRU + half * 16 + 8, hi + 8);
                tmem_st8(lane_addr + kColRU + 32 + half * 16, lo);
                tmem_st8(lane_addr + kColRU + 32 + half * 16 + 8, lo + 8);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bUhlReady);
            s_pending = true;
            step.advance(kStepRing);
            if (store_slot >= 0) {
                const bool oks = mbar_wait(bSReady, ph_s, abort_flag);
                if (!__all_sync(0xffffffffu, oks)) { dead = true; break; }
                ph_s ^= 1u;
                s_pending = false;
                tc_fence_after();
                store_state(store_slot);
            }
        }
        if (!dead && slot_out >= 0) {
            bool oks = true;
            if (s_pending) oks = mbar_wait(bSReady, ph_s, abort_flag);
            if (__all_sync(0xffffffffu, oks)) {
                tc_fence_after();
                store_state(slot_out);
            }
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) { }
        if (tid == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 9) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace kdatc
}  // namespace wpp

extern "C" int wpp_launch_kda_tc(const wpp::KdaTcParams* p, const CUtensorMap* maps, int max_blocks, void* stream) {
    using namespace wpp::kdatc;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kda_tc_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PrepSmem::kBytes);
        if (e != cudaSuccess) return (int)e;
        e = cudaFuncSetAttribute(kda_tc_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ChainSmem::kBytes);
        if (e != cudaSuccess) return (int)e;
        attr_set[dev] = true;
    }
    cudaStream_t st = (cudaStream_t)stream;
    kda_tc_setup_kernel<<<1, 1024, 0, st>>>(*p);
    if (max_blocks > 0) {
        dim3 grid_a((unsigned)max_blocks, (unsigned)p->num_heads);
        kda_tc_prep_kernel<<<grid_a, 128, PrepSmem::kBytes, st>>>(*p);
    }
    dim3 grid_b((unsigned)p->num_heads, (unsigned)p->num_requests);
    kda_tc_chain_kernel<<<grid_b, 320, ChainSmem::kBytes, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], maps[6],
                                                               maps[7], maps[8], maps[9], maps[10], *p);
    return (int)cudaGetLastError();
}
