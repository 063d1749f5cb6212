// Recurrent-state (KDA) layer of a chunk in its chunk-parallel form, on the tensor cores (Section 3.1 update, Section
// 3.2 snapshots).  Per request and head the update
//     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,     o_t = S_t^T q_t
// is rewritten over a block of tokens [a, b) that starts from the state S_0.  With S_0' = Diag(alpha_a) S_0 and the
// decay products G_t = prod_{a < r <= t} alpha_r (G_a = 1):
//     u_t  = beta_t (v_t - (Diag(alpha_t) S_{t-1})^T k_t)                       so that S_t = Diag(alpha_t) S_{t-1} + k_t u_t^T
//     S_t  = Diag(G_t) S_0' + sum_{s <= t} Diag(G_t / G_s) k_s u_s^T
// and, with Kt = K o G (rows k_t o G_t), Kh = K / G, Qt = Q o G, Kb = Kh o G_{b-1}:
//     A = tril(diag(beta) Kt Kh^T, -1),   (I + A) U = diag(beta) (V - Kt S_0'),   T = (I + A)^-1 diag(beta),
//     U = U0 - W0 S_0'   with   U0 = T V,  W0 = T Kt   (neither depends on the state),
//     O = Qt S_0' + M U  with   M = tril(Qt Kh^T),       S_b = Diag(G_{b-1}) S_0' + Kb^T U.
// Everything that does not involve the state is computed for all blocks in parallel by the PREPARATION kernel (one
// CTA per 64-token block and head: decay products, Kt, Kh, Qt, Kb, the products Kt Kh^T, Qt Kh^T, T Kt and T V on the
// tensor cores, the inverse of the unit lower triangular 64 x 64 matrix on CUDA cores) and left in a workspace; the
// CHAIN kernel (one CTA per request and head) then walks the blocks in order with four tensor-core products per
// block (W0 S_0', Qt S_0', M U, Kb^T U) and the 128 x 128 fp32 state resident in tensor memory.  Per block the
// chain from state to state is: scale and split the state, one product, form and split U, one product.
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
// the state directly instead of through a quotient G_t / G_s.  Decays of exactly 0 are therefore exact.  (T and M
// are block diagonal over the sub-blocks, so one set of operands serves all steps of a block; a step zeroes the
// rows of U outside its own tokens.)
//
// Orientation on the tensor cores: everything is kept transposed, with the value dimension d_v = 128 on the 128
// rows (tensor-memory lanes): S^T [d_v x d_k], X^T = S_0'^T W0^T [d_v x 64], O^T = S_0'^T Qt^T + U^T M^T,
// S_b^T = Diag-scaled S_0'^T + U^T Kb.  Thread r of a row warpgroup owns row r: column r of the state.
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
    const float2 d = __fadd2_rn(make_float2(x0, x1), make_float2(-__uint_as_float(hi << 16), -__uint_as_float(hi & 0xffff0000u)));
    lo = pack_bf16x2(d.x, d.y);
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
// Preparation: persistent CTAs (256 threads, two per SM), each taking (block, head) items in turn.  Inputs arrive by
// TMA a phase ahead of their use and results leave by TMA stores from swizzled staging tiles, so that no warp waits
// on a global load and no store instruction touches 32 rows at once.  Shared memory:
//   RA (64 KB): four slabs of 16 KB, slab s = 2 * term + khalf (term 0 = hi, 1 = lo; khalf = channels [64 khalf, +64)).
//       Each slab is a Kt tile (64 tokens x 128 bytes, swizzled) followed by an 8 KB slot, so that the A operand of a
//       128-row MMA that starts at the Kt tile has the slot as its rows 64..127.
//       Kt tiles, in turn: the raw keys (in the hi tiles) and queries (in the lo tiles) as they arrive; Kt (a thread
//       replaces the 16 bytes it read); staging of U0 on the way out.
//       Slots, in turn: alpha and then the decay products G (fp32, 32 channels per slot, 16-byte chunks swizzled like a
//       tile's); the Qt tiles (rows 64..127 of the first product's A operand: one MMA forms Kt Kh^T on lanes 0..63 and
//       Qt Kh^T on lanes 64..127; the same tiles are the source of the Qt stores); then the triangular matrix (fp32,
//       32 rows per slot, slots 0 and 1) and the V tiles (slots 2 and 3).
//   R2 (32 KB): the Kh tiles (same order as the slabs, 8 KB each); then staging of M (16 KB) and the inverse (16 KB);
//       then T as an A operand whose rows 64..127 repeat rows 0..63 (hi tile twice, lo tile twice), so that all 128
//       lanes of the second products carry results and all eight warps read them out; then staging of W0.
// fp32 arrays (alpha, U0) go through bf16 tensor maps with twice the elements per row: the copies move bytes.
struct PrepSmem {
    static constexpr int kSlab = 2 * kTileBytes;
    static constexpr int kOffRA = 0;
    static constexpr int kOffR2 = kOffRA + 4 * kSlab;
    static constexpr int kOffTmp = kOffR2 + 4 * kTileBytes;   // a 32 x 32 fp32 block (products of the inverse)
    static constexpr int kOffMisc = kOffTmp + 4 * 1024;       // beta[64], reduction scratch, tmem slot, barriers
    static constexpr int kBytes = kOffMisc + 1024 + 1024;     // + alignment slack
};

constexpr int kPrepThreads = 256;

__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(src), "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

struct PrepMaps {
    CUtensorMap w0_h, w0_l, qt_h, qt_l, m_h, m_l, u0;     // workspace arrays (stores)
    CUtensorMap q, k, v, alpha;                            // inputs (loads): (channel, head, row)
};

// The (block, head) item `item` of the wave: its request's geometry and the block's place in it.
struct PrepItem {
    int gb, head, blk, t_lo, t_hi;
    int64_t row_t0;
};
__device__ __forceinline__ PrepItem prep_item(const KdaTcParams& p, int item) {
    PrepItem it;
    const int H = p.num_heads, R = p.num_requests;
    it.gb = item / H;
    it.head = item - it.gb * H;
    int lo_r = 0, hi_r = R;                 // request: largest i with blk_off[i] <= gb (empty requests share offsets)
    while (hi_r - lo_r > 1) {
        const int mid = (lo_r + hi_r) >> 1;
        if (p.blk_off[mid] <= it.gb) lo_r = mid; else hi_r = mid;
    }
    const ReqBlocks g = req_blocks(p, lo_r);
    it.blk = g.first_block + (it.gb - p.blk_off[lo_r]);
    it.t_lo = max(0, g.P - it.blk * kL);                                    // active tokens [t_lo, t_hi)
    it.t_hi = min(kL, g.P + g.C - it.blk * kL);
    it.row_t0 = g.row0 + ((int64_t)it.blk * kL - g.P);                      // row of token 0 (may be < 0)
    return it;
}

__global__ void __launch_bounds__(kPrepThreads, 2)
kda_tc_prep_kernel(const __grid_constant__ PrepMaps maps, const KdaTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    uint8_t* r2 = sm + PrepSmem::kOffR2;
    float* Tmp = reinterpret_cast<float*>(sm + PrepSmem::kOffTmp);
    float* s_beta = reinterpret_cast<float*>(sm + PrepSmem::kOffMisc);              // [64]
    float* s_red = reinterpret_cast<float*>(sm + PrepSmem::kOffMisc + 256);         // [8]
    int* s_redi = reinterpret_cast<int*>(sm + PrepSmem::kOffMisc + 320);            // [4]
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + PrepSmem::kOffMisc + 512);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    const uint32_t bar = base + PrepSmem::kOffMisc + 528;           // MMA completions (two per item)
    const uint32_t bAlpha = bar + 8, bKQ = bar + 16, bV = bar + 24; // input arrivals (one each per item)
    const uint32_t a0 = base + PrepSmem::kOffRA, a2 = base + PrepSmem::kOffR2;
    constexpr int kSlab = PrepSmem::kSlab;
    // element (t, c) of the decay products; row t of the triangular matrix
    auto Gp = [&](int t, int c) -> float* {
        return reinterpret_cast<float*>(sm + (c >> 5) * kSlab + kTileBytes + t * 128 + ((((c & 31) >> 2) ^ (t & 7)) << 4) +
                                        (c & 3) * 4);
    };
    // (rows of 64 floats; the 16-byte chunks of a row are XOR-swizzled by the row so that a column walk across rows
    // and row-per-lane stores spread over the banks); the inverse X is laid out the same way
    auto Ap = [&](int t, int c) -> float* {
        return reinterpret_cast<float*>(sm + (t >> 5) * kSlab + kTileBytes + (t & 31) * 256) + ((((c >> 2) ^ (t & 7)) << 2) | (c & 3));
    };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int H = p.num_heads;
    const int n_items = p.blk_off[p.num_requests] * H;
    if ((int)blockIdx.x >= n_items) return;
    const size_t tile_elems = (size_t)kL * kD;

    // alpha into the slots and the raw keys and queries into the Kt tiles of the item `it`
    auto request_alpha = [&](const PrepItem& it) {
        mbar_arrive_expect_tx(bAlpha, 4 * kTileBytes);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            tma_load_3d(a0 + j * kSlab + kTileBytes, &maps.alpha, bAlpha, 64 * j, it.head, (int)it.row_t0);
    };
    auto request_kq = [&](const PrepItem& it) {
        mbar_arrive_expect_tx(bKQ, 4 * kTileBytes);
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
            tma_load_3d(a0 + kh * kSlab, &maps.k, bKQ, 64 * kh, it.head, (int)it.row_t0);
            tma_load_3d(a0 + (2 + kh) * kSlab, &maps.q, bKQ, 64 * kh, it.head, (int)it.row_t0);
        }
    };

    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_init(bAlpha, 1);
        mbar_init(bKQ, 1);
        mbar_init(bV, 1);
        *abort_flag = 0u;
        fence_barrier_init();
        const PrepItem first = prep_item(p, (int)blockIdx.x);
        request_alpha(first);
        request_kq(first);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;
    uint32_t in_phase = 0;

    PrepItem cur = prep_item(p, (int)blockIdx.x);
    // beta of the block (inactive tokens: 0); the later items' are fetched an item ahead
    if (tid < kL) s_beta[tid] = (tid >= cur.t_lo && tid < cur.t_hi) ? p.beta[(cur.row_t0 + tid) * H + cur.head] : 0.f;
    for (int item = (int)blockIdx.x;;) {
        const int head = cur.head, blk = cur.blk, t_lo = cur.t_lo, t_hi = cur.t_hi;
        const int64_t row_t0 = cur.row_t0;
        const size_t bh = (size_t)cur.gb * H + head;
        const int row_ws = (int)(bh * kL);                         // the item's first row in the workspace arrays

        // ---- cuts and decay products.  A sub-block starts at the first active token and after every token that
        //      completes a periodic snapshot position; with those cuts alone the decay products (from each sub-block's
        //      start, the start's own alpha excluded) are formed by two threads per channel, one per half of the block,
        //      the second half picking up the first half's last value.  Only if some product fell below 2^-40 are the
        //      extra cuts found, one at a time, by the slow path below.
        uint64_t mask = 1ull << t_lo;
        if (p.snap_interval > 0) {
            for (int t = t_lo; t + 1 < t_hi; ++t)
                if (((int64_t)blk * kL + t + 1) % p.snap_interval == 0) mask |= 1ull << (t + 1);
        }
        ok = __syncthreads_and(mbar_wait(bAlpha, in_phase, abort_flag));
        if (!ok) break;
        const int ch = tid & 127, half = tid >> 7;
        float gmin = 1.f;
        if (mask == 1ull && t_hi == kL) {
            // the usual block: all 64 tokens, no cut inside.  The second half forms its own products in registers while
            // the first half runs, then scales them by the first half's last value.
            if (half == 0) {
                float gacc = 1.f;
                *Gp(0, ch) = 1.f;
#pragma unroll
                for (int t = 1; t < 32; ++t) {
                    float* gp = Gp(t, ch);
                    gacc *= *gp;
                    *gp = gacc;
                    gmin = fminf(gmin, gacc);
                }
                named_bar(1, kPrepThreads);
            } else {
                float x[32];
                x[0] = *Gp(32, ch);
#pragma unroll
                for (int i = 1; i < 32; ++i) x[i] = x[i - 1] * *Gp(32 + i, ch);
                named_bar(1, kPrepThreads);
                const float carry = *Gp(31, ch);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    x[i] *= carry;
                    *Gp(32 + i, ch) = x[i];
                    gmin = fminf(gmin, x[i]);
                }
            }
        } else {
            {
                float gacc = 1.f;
                const int tb = half * 32;
#pragma unroll 8
                for (int t = tb; t < tb + 32; ++t) {
                    const bool active = t >= t_lo && t < t_hi;
                    float* gp = Gp(t, ch);
                    gacc = (!active || ((mask >> t) & 1ull)) ? 1.f : gacc * *gp;
                    *gp = gacc;
                }
            }
            __syncthreads();
            if (half == 1) {
                // tokens 32.. up to the first cut in this half continue the first half's product
                const uint64_t cuts = mask >> 32;
                const int n_carry = cuts ? (__ffsll((long long)cuts) - 1) : 32;
                const float carry = (31 >= t_lo && 31 < t_hi) ? *Gp(31, ch) : 1.f;
                for (int t = 32; t < 32 + n_carry; ++t)
                    if (t >= t_lo && t < t_hi) *Gp(t, ch) *= carry;
            }
            __syncthreads();
            {
                const int tb = half * 32;
#pragma unroll 8
                for (int t = tb; t < tb + 32; ++t) gmin = fminf(gmin, *Gp(t, ch));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) gmin = fminf(gmin, __shfl_xor_sync(0xffffffffu, gmin, o));
        if (lane == 0) s_red[warp] = gmin;
        __syncthreads();
        gmin = fminf(fminf(fminf(s_red[0], s_red[1]), fminf(s_red[2], s_red[3])),
                     fminf(fminf(s_red[4], s_red[5]), fminf(s_red[6], s_red[7])));
        if (!(gmin >= kMinGamma)) {
            // ---- slow path (rare): some channel decays below 2^-40 inside a sub-block.  The token that causes it starts
            //      a new sub-block; thread c < 128 follows channel c, the cuts are found one at a time.
            __syncthreads();
            for (int i = tid; i < kL * (kD / 4); i += kPrepThreads) {
                const int t = i >> 5, c4 = (i & 31) * 4;
                float4 a = make_float4(1.f, 1.f, 1.f, 1.f);
                if (t >= t_lo && t < t_hi) a = *reinterpret_cast<const float4*>(p.alpha + ((row_t0 + t) * H + head) * kD + c4);
                *reinterpret_cast<float4*>(Gp(t, c4)) = a;
            }
            __syncthreads();
            for (int round = 0; round < kL; ++round) {
                int first_bad = kL;
                if (tid < 128) {
                    float gacc = 1.f;
                    for (int t = t_lo + 1; t < t_hi; ++t) {
                        if ((mask >> t) & 1ull) { gacc = 1.f; continue; }
                        gacc *= *Gp(t, tid);
                        if (!(gacc >= kMinGamma)) { first_bad = t; break; }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) first_bad = min(first_bad, __shfl_xor_sync(0xffffffffu, first_bad, o));
                    if (lane == 0) s_redi[warp] = first_bad;
                }
                __syncthreads();
                first_bad = min(min(s_redi[0], s_redi[1]), min(s_redi[2], s_redi[3]));
                __syncthreads();
                if (first_bad >= kL) break;
                mask |= 1ull << first_bad;
            }
            if (tid < 128) {
                float gacc = 1.f;
                for (int t = 0; t < kL; ++t) {
                    if (t < t_lo || t >= t_hi) { *Gp(t, tid) = 1.f; continue; }
                    gacc = ((mask >> t) & 1ull) ? 1.f : gacc * *Gp(t, tid);
                    *Gp(t, tid) = gacc;
                }
            }
            __syncthreads();
        }
        // the last row of every sub-block goes to the workspace (the chain scales the state by it)
        if (tid < 128) {
            int a = t_lo;
            while (a < t_hi) {
                const int e = sub_end(mask, a, t_hi);
                p.ws_e[(bh * kL + e - 1) * kD + tid] = *Gp(e - 1, tid);
                a = e;
            }
        }
        if (tid == 0) p.ws_mask[bh] = mask;

        // ---- Kt = k G, Kh = k / G, Kb = Kh G_end, Qt = q G as hi/lo bf16.  Kt and Kh go to shared memory (MMA operands),
        //      Kb to the workspace; Qt waits in registers for the slots the decay products occupy.  A thread handles 8
        //      consecutive channels of a token at a time; the raw keys and queries sit where its Kt terms go.
        ok = __syncthreads_and(mbar_wait(bKQ, in_phase, abort_flag));
        if (!ok) break;
        uint4 qt_h[4], qt_l[4];
        float ee[8];                       // the decay products at the end of the sub-block, for this thread's channels
        int e_have = -1;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int idx = it * kPrepThreads + tid, t = idx >> 4, c8 = idx & 15, c0 = c8 * 8;
            const bool active = t >= t_lo && t < t_hi;
            const uint32_t sw = sw_off(t, c8 & 7);
            const int kh = c8 >> 3;
            uint4 kt_h = make_uint4(0, 0, 0, 0), kt_l = kt_h, kh_h = kt_h, kh_l = kt_h, kb_h = kt_h, kb_l = kt_h;
            qt_h[it] = kt_h; qt_l[it] = kt_h;
            if (active) {
                const int e_t = sub_end(mask, t, t_hi) - 1;
                const uint4 kraw = *reinterpret_cast<const uint4*>(sm + kh * kSlab + sw);
                const uint4 qraw = *reinterpret_cast<const uint4*>(sm + (2 + kh) * kSlab + sw);
                const uint32_t rw[4] = {kraw.x, kraw.y, kraw.z, kraw.w}, rq[4] = {qraw.x, qraw.y, qraw.z, qraw.w};
                const float4 g0 = *reinterpret_cast<const float4*>(Gp(t, c0)), g1 = *reinterpret_cast<const float4*>(Gp(t, c0 + 4));
                if (e_t != e_have) {
                    const float4 e0 = *reinterpret_cast<const float4*>(Gp(e_t, c0)), e1 = *reinterpret_cast<const float4*>(Gp(e_t, c0 + 4));
                    ee[0] = e0.x; ee[1] = e0.y; ee[2] = e0.z; ee[3] = e0.w; ee[4] = e1.x; ee[5] = e1.y; ee[6] = e1.z; ee[7] = e1.w;
                    e_have = e_t;
                }
                const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                uint32_t o[8][4];
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float k0 = __uint_as_float(rw[w] << 16), k1 = __uint_as_float(rw[w] & 0xffff0000u);
                    const float q0 = __uint_as_float(rq[w] << 16), q1 = __uint_as_float(rq[w] & 0xffff0000u);
                    const float i0 = rcp_approx(gg[2 * w]), i1 = rcp_approx(gg[2 * w + 1]);      // g >= 2^-40: finite
                    const float h0 = k0 * i0, h1 = k1 * i1;
                    split2(k0 * gg[2 * w], k1 * gg[2 * w + 1], o[0][w], o[1][w]);
                    split2(h0, h1, o[2][w], o[3][w]);
                    split2(h0 * ee[2 * w], h1 * ee[2 * w + 1], o[4][w], o[5][w]);
                    split2(q0 * gg[2 * w], q1 * gg[2 * w + 1], o[6][w], o[7][w]);
                }
                kt_h = make_uint4(o[0][0], o[0][1], o[0][2], o[0][3]); kt_l = make_uint4(o[1][0], o[1][1], o[1][2], o[1][3]);
                kh_h = make_uint4(o[2][0], o[2][1], o[2][2], o[2][3]); kh_l = make_uint4(o[3][0], o[3][1], o[3][2], o[3][3]);
                kb_h = make_uint4(o[4][0], o[4][1], o[4][2], o[4][3]); kb_l = make_uint4(o[5][0], o[5][1], o[5][2], o[5][3]);
                qt_h[it] = make_uint4(o[6][0], o[6][1], o[6][2], o[6][3]); qt_l[it] = make_uint4(o[7][0], o[7][1], o[7][2], o[7][3]);
            }
            *reinterpret_cast<uint4*>(sm + kh * kSlab + sw) = kt_h;
            *reinterpret_cast<uint4*>(sm + (2 + kh) * kSlab + sw) = kt_l;
            *reinterpret_cast<uint4*>(r2 + kh * kTileBytes + sw) = kh_h;
            *reinterpret_cast<uint4*>(r2 + (2 + kh) * kTileBytes + sw) = kh_l;
            const size_t go = bh * tile_elems + (size_t)t * kD + c0;
            *reinterpret_cast<uint4*>(p.ws_kb_h + go) = kb_h;
            *reinterpret_cast<uint4*>(p.ws_kb_l + go) = kb_l;
        }
        __syncthreads();                   // every read of the decay products is done: Qt takes their place
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int idx = it * kPrepThreads + tid, t = idx >> 4, c8 = idx & 15;
            const uint32_t off = (uint32_t)((c8 >> 3) * kSlab + kTileBytes) + sw_off(t, c8 & 7);
            *reinterpret_cast<uint4*>(sm + off) = qt_h[it];
            *reinterpret_cast<uint4*>(sm + 2 * kSlab + off) = qt_l[it];
        }
        fence_proxy_async_smem();
        __syncthreads();

        // ---- [Kt; Qt] Kh^T -> columns [0, 64): lanes 0..63 carry Kt Kh^T, lanes 64..127 Qt Kh^T;
        //      (hi + lo)(hi + lo)^T without the lo x lo term.  The Qt tiles leave for the workspace from where they are.
        if (tid == 0) {
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(64, 0, 0);
            const uint32_t a_hi = a0, a_lo = a0 + 2 * kSlab, b_hi = a2, b_lo = a2 + 2 * kTileBytes;
            const uint32_t aa[3] = {a_hi, a_hi, a_lo}, bb[3] = {b_hi, b_lo, b_hi};
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint64_t ad = smem_desc_sw128(aa[term], 16, 1024), bd = smem_desc_sw128(bb[term], 16, 1024);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t offa = (uint64_t)(((kk >> 2) * kSlab + (kk & 3) * 32) >> 4);
                    const uint64_t offb = (uint64_t)(((kk >> 2) * kTileBytes + (kk & 3) * 32) >> 4);
                    mma_ss(tmem, ad + offa, bd + offb, idesc, (term | kk) ? 1u : 0u);
                }
            }
            mma_commit(bar);
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                tma_store_2d(&maps.qt_h, a0 + kh * kSlab + kTileBytes, 64 * kh, row_ws);
                tma_store_2d(&maps.qt_l, a0 + (2 + kh) * kSlab + kTileBytes, 64 * kh, row_ws);
            }
            bulk_commit();
            bulk_wait_read_all();          // before the slots are written again
        }
        ok = __syncthreads_and(mbar_wait(bar, 0, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // the block's values into slots 2 and 3, on their way while the inverse is formed
        if (tid == 0) {
            mbar_arrive_expect_tx(bV, 2 * kTileBytes);
            tma_load_3d(a0 + 2 * kSlab + kTileBytes, &maps.v, bV, 0, head, (int)row_t0);
            tma_load_3d(a0 + 3 * kSlab + kTileBytes, &maps.v, bV, 64, head, (int)row_t0);
        }

        // ---- rows of the two products.  Warps w with (w & 3) < 2 own lanes of Kt Kh^T, whose strictly lower part within
        //      a sub-block, scaled by beta_t, is the triangular matrix (to slots 0 and 1); the others own lanes of
        //      M = tril(Qt Kh^T), which goes to the workspace through staging tiles in R2 (the Kh tiles are spent).
        //      Warps 0..3 take columns [0, 32), warps 4..7 columns [32, 64).
        {
            const int qd = warp & 3, cb = (warp >> 2) * 32;
            const int t = (qd & 1) * 32 + lane;
            const bool active = t >= t_lo && t < t_hi;
            const int s0 = active ? sub_start(mask, t) : kL;    // columns [s0, t) (and t itself for M) count
            float x[32];
            tmem_ld32(tmem + ((uint32_t)(qd * 32) << 16) + cb, reinterpret_cast<uint32_t*>(x));
            tmem_wait_ld();
            if (qd < 2) {
                const float bt = s_beta[t];
#pragma unroll
                for (int s4 = 0; s4 < 8; ++s4) {
                    float4 a;
                    a.x = (active && cb + 4 * s4 + 0 >= s0 && cb + 4 * s4 + 0 < t) ? bt * x[4 * s4 + 0] : 0.f;
                    a.y = (active && cb + 4 * s4 + 1 >= s0 && cb + 4 * s4 + 1 < t) ? bt * x[4 * s4 + 1] : 0.f;
                    a.z = (active && cb + 4 * s4 + 2 >= s0 && cb + 4 * s4 + 2 < t) ? bt * x[4 * s4 + 2] : 0.f;
                    a.w = (active && cb + 4 * s4 + 3 >= s0 && cb + 4 * s4 + 3 < t) ? bt * x[4 * s4 + 3] : 0.f;
                    *reinterpret_cast<float4*>(Ap(t, cb + 4 * s4)) = a;
                }
            } else {
#pragma unroll
                for (int i8 = 0; i8 < 4; ++i8) {
                    uint32_t oh[4], ol[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int s = i8 * 8 + 2 * i;
                        const float m0 = (active && cb + s >= s0 && cb + s <= t) ? x[s] : 0.f;
                        const float m1 = (active && cb + s + 1 >= s0 && cb + s + 1 <= t) ? x[s + 1] : 0.f;
                        split2(m0, m1, oh[i], ol[i]);
                    }
                    const uint32_t off = sw_off(t, (cb >> 3) + i8);
                    *reinterpret_cast<uint4*>(r2 + off) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
                    *reinterpret_cast<uint4*>(r2 + kTileBytes + off) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tma_store_2d(&maps.m_h, a2, 0, row_ws);
            tma_store_2d(&maps.m_l, a2 + kTileBytes, 0, row_ws);
            bulk_commit();
        }
        // ---- T = (I + A)^-1 diag(beta).  The unit lower triangular 64 x 64 matrix L = I + A is inverted by halving: the
        //      four 16 x 16 diagonal blocks by forward substitution (64 threads, one column each, while the others zero
        //      the blocks above the diagonal), then twice [[X11, 0], [-X22 L21 X11, X22]]: for the two 32 x 32 diagonal
        //      blocks (16 x 16 products) and for the whole matrix (32 x 32 products), each as two small products with
        //      every thread busy.  X lives in the upper half of R2, where (and over the staging tiles of M) the T
        //      tiles go afterwards.
        auto Xp = [&](int r, int c) -> float* {                           // [64][64] fp32
            return reinterpret_cast<float*>(r2 + 2 * kTileBytes) + r * kL + ((((c >> 2) ^ (r & 7)) << 2) | (c & 3));
        };
        {
            if (tid < kL) {
                const int bi = tid >> 4, c = tid & 15;
                float x[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    float acc = (r == c) ? 1.f : 0.f;
#pragma unroll
                    for (int q = 0; q < r; ++q) acc = fmaf(-*Ap(bi * 16 + r, bi * 16 + q), x[q], acc);
                    x[r] = acc;
                    *Xp(bi * 16 + r, bi * 16 + c) = acc;
                }
            } else {
                for (int i = tid - kL; i < 6 * 64; i += kPrepThreads - kL) {
                    const int b = i >> 6, r = (i & 63) >> 2, c4 = (i & 3) * 4;      // blocks (0,1) (0,2) (0,3) (1,2) (1,3) (2,3)
                    const int bi = b < 3 ? 0 : (b < 5 ? 1 : 2), bj = b < 3 ? b + 1 : (b < 5 ? b - 1 : 3);
                    *reinterpret_cast<float4*>(Xp(bi * 16 + r, bj * 16 + c4)) = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            __syncthreads();
            {
                // blocks (1, 0) and (3, 2): thread -> (which, row, 2 columns)
                const int pr = tid >> 7, er = (tid >> 3) & 15, ec = (tid & 7) * 2;
                const int i = 2 * pr + 1, j = 2 * pr;
                float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                for (int q4 = 0; q4 < 16; q4 += 4) {
                    const float4 l = *reinterpret_cast<const float4*>(Ap(i * 16 + er, j * 16 + q4));
                    const float lq[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float2 xv = *reinterpret_cast<const float2*>(Xp(j * 16 + q4 + q, j * 16 + ec));
                        acc.x = fmaf(lq[q], xv.x, acc.x); acc.y = fmaf(lq[q], xv.y, acc.y);
                    }
                }
                *reinterpret_cast<float2*>(Tmp + pr * 256 + er * 16 + ec) = acc;
                __syncthreads();
                acc = make_float2(0.f, 0.f);
#pragma unroll
                for (int q4 = 0; q4 < 16; q4 += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(Xp(i * 16 + er, i * 16 + q4));
                    const float xq[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float2 tv = *reinterpret_cast<const float2*>(Tmp + pr * 256 + (q4 + q) * 16 + ec);
                        acc.x = fmaf(xq[q], tv.x, acc.x); acc.y = fmaf(xq[q], tv.y, acc.y);
                    }
                }
                *reinterpret_cast<float2*>(Xp(i * 16 + er, j * 16 + ec)) = make_float2(-acc.x, -acc.y);
                __syncthreads();
            }
            {
                // rows 32..63, columns 0..31: thread -> (row, 4 columns).  Eight steps at a time: the swizzle of the rows
                // walked then folds into constants.
                const int er = tid >> 3, ec = (tid & 7) * 4;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
                for (int k8 = 0; k8 < 32; k8 += 8) {
                    const float4 l0 = *reinterpret_cast<const float4*>(Ap(32 + er, k8));
                    const float4 l1 = *reinterpret_cast<const float4*>(Ap(32 + er, k8 + 4));
                    const float lq[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
                    const float* xrow = reinterpret_cast<const float*>(r2 + 2 * kTileBytes) + k8 * kL + (ec & 3);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 xv = *reinterpret_cast<const float4*>(xrow + q * kL + (((ec >> 2) ^ q) << 2));
                        acc.x = fmaf(lq[q], xv.x, acc.x); acc.y = fmaf(lq[q], xv.y, acc.y);
                        acc.z = fmaf(lq[q], xv.z, acc.z); acc.w = fmaf(lq[q], xv.w, acc.w);
                    }
                }
                *reinterpret_cast<float4*>(Tmp + er * 32 + ec) = acc;
                __syncthreads();
                acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
                for (int k8 = 0; k8 < 32; k8 += 8) {
                    const float4 x0 = *reinterpret_cast<const float4*>(Xp(32 + er, 32 + k8));
                    const float4 x1 = *reinterpret_cast<const float4*>(Xp(32 + er, 32 + k8 + 4));
                    const float xq[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 tv = *reinterpret_cast<const float4*>(Tmp + (k8 + q) * 32 + ec);
                        acc.x = fmaf(xq[q], tv.x, acc.x); acc.y = fmaf(xq[q], tv.y, acc.y);
                        acc.z = fmaf(xq[q], tv.z, acc.z); acc.w = fmaf(xq[q], tv.w, acc.w);
                    }
                }
                *reinterpret_cast<float4*>(Xp(32 + er, ec)) = make_float4(-acc.x, -acc.y, -acc.z, -acc.w);
                __syncthreads();
            }
            // T[t][c] = X[t][c] beta_c as hi/lo operand tiles, each stored twice: thread -> (row, 16 columns)
            {
                const int t = tid >> 2, cb = (tid & 3) * 16;
                uint4 th[2], tl[2];
#pragma unroll
                for (int j8 = 0; j8 < 2; ++j8) {
                    uint32_t oh[4], ol[4];
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int c = cb + j8 * 8 + 4 * i;
                        const float4 x = *reinterpret_cast<const float4*>(Xp(t, c));
                        const float4 b = *reinterpret_cast<const float4*>(s_beta + c);
                        split2(x.x * b.x, x.y * b.y, oh[2 * i], ol[2 * i]);
                        split2(x.z * b.z, x.w * b.w, oh[2 * i + 1], ol[2 * i + 1]);
                    }
                    th[j8] = make_uint4(oh[0], oh[1], oh[2], oh[3]);
                    tl[j8] = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                }
                if (tid == 0) bulk_wait_read_all();     // the staging tiles of M have been read
                __syncthreads();                        // and so has the inverse: the tiles take their place
#pragma unroll
                for (int j8 = 0; j8 < 2; ++j8) {
                    const uint32_t off = sw_off(t, (cb >> 3) + j8);
                    *reinterpret_cast<uint4*>(r2 + off) = th[j8];
                    *reinterpret_cast<uint4*>(r2 + kTileBytes + off) = th[j8];
                    *reinterpret_cast<uint4*>(r2 + 2 * kTileBytes + off) = tl[j8];
                    *reinterpret_cast<uint4*>(r2 + 3 * kTileBytes + off) = tl[j8];
                }
            }
        }
        // rows of V that belong to no token of this request (a block at either end of a chunk) are whatever lies
        // next to the chunk in the array: they meet zero columns of T, but must be finite for that to give zero
        if (t_lo > 0 || t_hi < kL) {
            ok = __syncthreads_and(mbar_wait(bV, in_phase, abort_flag));
            if (!ok) break;
            for (int i = tid; i < kL * 16; i += kPrepThreads) {
                const int t = i >> 4, c8 = i & 15;
                if (t < t_lo || t >= t_hi)
                    *reinterpret_cast<uint4*>(sm + (2 + (c8 >> 3)) * kSlab + kTileBytes + sw_off(t, c8 & 7)) = make_uint4(0, 0, 0, 0);
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        // ---- W0 = T Kt -> columns [0, 128), U0 = T V -> columns [128, 256)   (V is bf16: it has no lo term); lanes
        //      64..127 repeat lanes 0..63
        if (tid == 0) {
            const bool okv = mbar_wait(bV, in_phase, abort_flag);
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(128, 0, 1);
            const uint32_t t_hi_a = a2, t_lo_a = a2 + 2 * kTileBytes;
            const uint32_t kt_hi = a0, kt_lo = a0 + 2 * kSlab, v_a = a0 + 2 * kSlab + kTileBytes;
            const uint32_t aa[5] = {t_hi_a, t_hi_a, t_lo_a, t_hi_a, t_lo_a}, bb[5] = {kt_hi, kt_lo, kt_hi, v_a, v_a};
            if (okv) {
#pragma unroll
                for (int term = 0; term < 5; ++term) {
                    const uint64_t ad = smem_desc_sw128(aa[term], 16, 1024), bd = smem_desc_sw128(bb[term], kSlab, 1024);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ss(tmem + (term >= 3 ? 128 : 0), ad + (uint64_t)(kk * 2), bd + (uint64_t)(kk * 128), idesc,
                               ((term == 0 || term == 3) && kk == 0) ? 0u : 1u);
                }
            }
            mma_commit(bar);
        }
        ok = __syncthreads_and(mbar_wait(bar, 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // the next item's alpha is requested as soon as the slots are free, and its beta fetched
        const int next = item + (int)gridDim.x;
        const bool more = next < n_items;
        PrepItem nxt = cur;
        float beta_next = 0.f;
        if (more) {
            nxt = prep_item(p, next);
            if (tid == 0) request_alpha(nxt);
            if (tid < kL && tid >= nxt.t_lo && tid < nxt.t_hi) beta_next = p.beta[(nxt.row_t0 + tid) * H + nxt.head];
        }
        // ---- rows of W0 (warps 0..3: hi/lo bf16, staged in R2) and of U0 (warps 4..7: fp32, staged in the Kt tiles); a
        //      warp's lanes are tokens 32 (w & 1) + lane, and it takes columns [64 ((w & 3) >> 1), +64)
        {
            const int qd = warp & 3, t = (qd & 1) * 32 + lane, cbase = (qd >> 1) * 64;
            const uint32_t lane_addr = tmem + ((uint32_t)(qd * 32) << 16) + (warp >= 4 ? 128 : 0) + cbase;
            if (warp < 4) {
                uint8_t* hi_tile = r2 + (cbase >> 6) * kTileBytes;            // khalf = cbase / 64
                uint8_t* lo_tile = r2 + (2 + (cbase >> 6)) * kTileBytes;
#pragma unroll 1
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    float x[32];
                    tmem_ld32(lane_addr + c0, reinterpret_cast<uint32_t*>(x));
                    tmem_wait_ld();
#pragma unroll
                    for (int i8 = 0; i8 < 4; ++i8) {
                        uint32_t oh[4], ol[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) split2(x[i8 * 8 + 2 * i], x[i8 * 8 + 2 * i + 1], oh[i], ol[i]);
                        const uint32_t off = sw_off(t, (c0 >> 3) + i8);
                        *reinterpret_cast<uint4*>(hi_tile + off) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
                        *reinterpret_cast<uint4*>(lo_tile + off) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                    }
                }
            } else {
#pragma unroll 1
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    float x[32];
                    tmem_ld32(lane_addr + c0, reinterpret_cast<uint32_t*>(x));
                    tmem_wait_ld();
                    uint8_t* tile = sm + ((cbase + c0) >> 5) * kSlab;         // 32 fp32 columns per tile
#pragma unroll
                    for (int i4 = 0; i4 < 8; ++i4)
                        *reinterpret_cast<float4*>(tile + sw_off(t, i4)) = make_float4(x[4 * i4], x[4 * i4 + 1], x[4 * i4 + 2], x[4 * i4 + 3]);
                }
            }
        }
        if (tid < kL) s_beta[tid] = beta_next;
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (tid == 0) {
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                tma_store_2d(&maps.w0_h, a2 + kh * kTileBytes, 64 * kh, row_ws);
                tma_store_2d(&maps.w0_l, a2 + (2 + kh) * kTileBytes, 64 * kh, row_ws);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) tma_store_2d(&maps.u0, a0 + j * kSlab, 64 * j, row_ws);
            bulk_commit();
            bulk_wait_read_all();          // the Kt tiles and R2 are free again
            if (more) request_kq(nxt);
        }
        if (!more) break;
        cur = nxt;
        item = next;
        in_phase ^= 1u;
    }
    if (tid == 0) {
        // a wait that gave up leaves copies in flight: give them time to land before the CTA's shared memory is released
        if (!ok)
            for (int i = 0; i < 200; ++i) __nanosleep(1000);
        bulk_wait_all();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, 256);
    }
    if (!ok && tid == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------------------------
// Chain: one CTA per (request, head).  Warps 0-3 and 4-7: two row warpgroups (thread r of either = tensor-memory lane r
// = column r of S); they share the per-step conversions half and half, and the second one also writes the outputs.
// Warp 8: operand loader (TMA); warp 9: one thread issues the MMAs; warp 10: publishes the step records.
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
    int store_slot;      // state slot to write after the step (periodic snapshot), or -1
    int pad[3];
    int64_t row_t0;      // row of the block's token 0 in the packed arrays
};
struct ChainSmem {
    // operand tiles of one block.  WQ: W0 and Qt stacked as one 128-row operand per 64-column tile (rows 0..63 W0,
    // rows 64..127 Qt), so that X = W0 S_0' and the first part of the outputs, Qt S_0', are ONE product of N = 128:
    // [W0 hi0 | Qt hi0][W0 hi1 | Qt hi1][W0 lo0 | Qt lo0][W0 lo1 | Qt lo1]
    static constexpr int kOffWQ = 0;
    static constexpr int kOffKb = kOffWQ + 8 * kTileBytes;    // hi0 hi1 lo0 lo1
    static constexpr int kOffM = kOffKb + 4 * kTileBytes;     // hi lo
    static constexpr int kOffU0 = kOffM + 2 * kTileBytes;     // fp32 [64][128], plain rows
    static constexpr int kOffOut = kOffU0 + kL * kD * 4;      // bf16 [64][128]: a step's outputs on their way to global memory
    static constexpr int kOffVec = kOffOut + kL * kD * 2;     // per ring slot: alpha of the step's first token, decay product at its end
    static constexpr int kOffRec = kOffVec + kStepRing * 2 * kD * 4;
    static constexpr int kOffBars = kOffRec + kStepRing * (int)sizeof(StepRec);
    static constexpr int kNumBars = 2 * kStepRing + 8 + 7;
    static constexpr int kOffMisc = kOffBars + 8 * kNumBars;
    static constexpr int kBytes = kOffMisc + 64 + 1024;
};
// tensor-memory columns: the state, its hi/lo operand form, and two result regions used by alternate steps.  A result
// region holds X = W0 S_0' in its first 64 columns - replaced in place by U as a hi/lo operand: tokens 0..31 hi in
// columns [0, 16), lo in [16, 32), tokens 32..63 hi in [32, 48), lo in [48, 64) - and the output accumulator in its
// last 64 columns.
constexpr uint32_t kColS = 0, kColShl = 128, kColD = 256;
__device__ __forceinline__ uint32_t col_d(int step) { return kColD + 128u * (uint32_t)(step & 1); }

__global__ void __launch_bounds__(352, 1)
kda_tc_chain_kernel(const __grid_constant__ CUtensorMap tm_w0_h, const __grid_constant__ CUtensorMap tm_w0_l,
                    const __grid_constant__ CUtensorMap tm_qt_h, const __grid_constant__ CUtensorMap tm_qt_l,
                    const __grid_constant__ CUtensorMap tm_kb_h, const __grid_constant__ CUtensorMap tm_kb_l,
                    const __grid_constant__ CUtensorMap tm_m_h, const __grid_constant__ CUtensorMap tm_m_l,
                    const KdaTcParams p) {
    using CS = ChainSmem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + CS::kOffBars;
    auto bStepFull = [&](int s) { return bars + 8 * s; };
    auto bStepEmpty = [&](int s) { return bars + 8 * (kStepRing + s); };
    const uint32_t b0 = bars + 16 * kStepRing;
    // operand buffers (one block in flight each), in the order a block's last step releases them: WQ, U0, Kb, M
    const uint32_t bWQFull = b0, bWQEmpty = b0 + 8, bU0Full = b0 + 16, bU0Empty = b0 + 24, bKbFull = b0 + 32,
                   bKbEmpty = b0 + 40, bMFull = b0 + 48, bMEmpty = b0 + 56;
    const uint32_t b1 = b0 + 64;
    const uint32_t bShlReady = b1, bXReady = b1 + 8, bUhlReady = b1 + 16, bSReady = b1 + 24, bOReady = b1 + 32;
    // o_free, one per result region: a waiter may lag a barrier by at most one phase, and the issuing thread asks for
    // the read-out of two steps back while the row threads may already have signalled the one after it
    auto bOFree = [&](int n) { return b1 + 40 + 8 * (uint32_t)(n & 1); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + CS::kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    const float* s_vec = reinterpret_cast<const float*>(sm + CS::kOffVec);
    const float* s_u0 = reinterpret_cast<const float*>(sm + CS::kOffU0);
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
        for (int s = 0; s < kStepRing; ++s) { mbar_init(bStepFull(s), 1); mbar_init(bStepEmpty(s), 256 + 1); }
        mbar_init(bWQFull, 1); mbar_init(bWQEmpty, 1); mbar_init(bKbFull, 1); mbar_init(bKbEmpty, 1);
        mbar_init(bMFull, 1); mbar_init(bMEmpty, 1);
        mbar_init(bU0Full, 1);
        mbar_init(bU0Empty, 256);          // the U0 tile is released by the 256 row threads
        mbar_init(bShlReady, 256); mbar_init(bXReady, 1); mbar_init(bUhlReady, 256); mbar_init(bSReady, 1);
        mbar_init(bOReady, 1); mbar_init(bOFree(0), 128); mbar_init(bOFree(1), 128);
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
        // ================================================================ operand loader
        // One buffer per operand; a block's operands are released, in this order, as its last step proceeds (WQ after
        // the first product, U0 by the row threads, Kb after the state product, M after the second output product),
        // and each is requested again for the next block the moment it is free.
        uint32_t ph_e = 0;
        for (int b = 0; b < g.n_blocks; ++b) {
            const size_t bh = (size_t)(gb0 + b) * H + head;
            const int row = (int)(bh * kL);
            bool okw = __all_sync(0xffffffffu, mbar_wait(bWQEmpty, ph_e ^ 1u, abort_flag));
            if (!okw) break;
            if (lane == 0) mbar_arrive_expect_tx(bWQFull, 8 * kTileBytes);
            __syncwarp();
            if (lane < 8) {
                // lane = 4 * (lo part) + 2 * (column half) + (0: W0, 1: Qt)
                const bool lo_part = lane & 4, qt = lane & 1;
                const int half = (lane >> 1) & 1;
                const CUtensorMap* tm = qt ? (lo_part ? &tm_qt_l : &tm_qt_h) : (lo_part ? &tm_w0_l : &tm_w0_h);
                tma_load_2d(base + CS::kOffWQ + ((lane >> 1) * 2 + (lane & 1)) * kTileBytes, tm, bWQFull, half * 64, row);
            }
            okw = __all_sync(0xffffffffu, mbar_wait(bU0Empty, ph_e ^ 1u, abort_flag));
            if (!okw) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(bU0Full, kL * kD * 4);
                bulk_load(base + CS::kOffU0, p.ws_u0 + bh * (size_t)kL * kD, kL * kD * 4, bU0Full);
            }
            okw = __all_sync(0xffffffffu, mbar_wait(bKbEmpty, ph_e ^ 1u, abort_flag));
            if (!okw) break;
            if (lane == 0) mbar_arrive_expect_tx(bKbFull, 4 * kTileBytes);
            __syncwarp();
            if (lane < 4)
                tma_load_2d(base + CS::kOffKb + lane * kTileBytes, (lane & 2) ? &tm_kb_l : &tm_kb_h, bKbFull, (lane & 1) * 64, row);
            okw = __all_sync(0xffffffffu, mbar_wait(bMEmpty, ph_e ^ 1u, abort_flag));
            if (!okw) break;
            if (lane == 0) mbar_arrive_expect_tx(bMFull, 2 * kTileBytes);
            __syncwarp();
            if (lane < 2) tma_load_2d(base + CS::kOffM + lane * kTileBytes, lane ? &tm_m_l : &tm_m_h, bMFull, 0, row);
            ph_e ^= 1u;
        }
    } else if (warp == 10) {
        // ================================================================ step records
        Ring step = {0, 0};
        bool dead = false;
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
        uint32_t ph_wq = 0, ph_kb = 0, ph_m = 0, ph_shl = 0, ph_uhl = 0, ph_ofree[2] = {0, 0};
        constexpr uint32_t idesc64 = idesc_bf16(64, 0, 0), idesc128 = idesc_bf16(128, 0, 0), idesc128mn = idesc_bf16(128, 0, 1);
        const uint32_t tS = tmem + kColS, tShl = tmem + kColShl;
        // descriptors of the operand buffers (they never move)
        const uint64_t wq_hi = smem_desc_sw128(base + CS::kOffWQ, 16, 1024), wq_lo = smem_desc_sw128(base + CS::kOffWQ + 4 * kTileBytes, 16, 1024);
        const uint64_t kb_hi = smem_desc_sw128(base + CS::kOffKb, kTileBytes, 1024), kb_lo = smem_desc_sw128(base + CS::kOffKb + 2 * kTileBytes, kTileBytes, 1024);
        const uint64_t m_hi = smem_desc_sw128(base + CS::kOffM, 16, 1024), m_lo = smem_desc_sw128(base + CS::kOffM + kTileBytes, 16, 1024);
        int n = 0;                     // step counter: selects the result region
        while (true) {
            if (!mbar_wait(bStepFull(step.stage), step.phase, abort_flag)) break;
            const int a = s_rec[step.stage].a;
            const bool first = s_rec[step.stage].first, last = s_rec[step.stage].last;
            mbar_arrive(bStepEmpty(step.stage));
            step.advance(kStepRing);
            if (a < 0) break;
            const uint32_t tD = tmem + col_d(n);
            // ---- [X^T | O^T] = S_0'^T [W0; Qt]^T   (the region's previous outputs, two steps back, must have been read)
            if (n >= 2) { if (!mbar_wait(bOFree(n), ph_ofree[n & 1], abort_flag)) break; ph_ofree[n & 1] ^= 1u; }
            if (!mbar_wait(bShlReady, ph_shl, abort_flag)) break;
            ph_shl ^= 1u;
            if (first) { if (!mbar_wait(bWQFull, ph_wq, abort_flag)) break; ph_wq ^= 1u; }
            tc_fence_after();
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint32_t a_tm = tShl + (term == 2 ? 64u : 0u);
                const uint64_t bd = (term == 1) ? wq_lo : wq_hi;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * 2 * kTileBytes + (kk & 3) * 32) >> 4);
                    if (term == 0 && kk == 0) mma_ts_overwrite(tD, a_tm, bd + off, idesc128);
                    else mma_ts_accumulate(tD, a_tm + kk * 8, bd + off, idesc128);
                }
            }
            mma_commit(bXReady);
            if (last) mma_commit(bWQEmpty);
            // ---- S_b^T += U^T Kb   (the accumulator was preset to the decayed S_0'),   O^T += U^T M^T
            if (!mbar_wait(bUhlReady, ph_uhl, abort_flag)) break;
            ph_uhl ^= 1u;
            if (first) { if (!mbar_wait(bKbFull, ph_kb, abort_flag)) break; ph_kb ^= 1u; }
            tc_fence_after();
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint64_t bd = (term == 1) ? kb_lo : kb_hi;          // MN-major: 64-column halves kTileBytes apart
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts_accumulate(tS, tD + (kk >> 1) * 32 + (kk & 1) * 8 + (term == 2 ? 16u : 0u), bd + (uint64_t)(kk * 128), idesc128mn);
            }
            mma_commit(bSReady);
            if (last) mma_commit(bKbEmpty);
            if (first) { if (!mbar_wait(bMFull, ph_m, abort_flag)) break; ph_m ^= 1u; }
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint64_t bd = (term == 1) ? m_lo : m_hi;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts_accumulate(tD + 64, tD + (kk >> 1) * 32 + (kk & 1) * 8 + (term == 2 ? 16u : 0u), bd + (uint64_t)(kk * 2), idesc64);
            }
            mma_commit(bOReady);
            if (last) mma_commit(bMEmpty);
            ++n;
        }
    } else if (warp < 8) {
        // ================================================================ the state's rows (thread r = column r of S)
        const int wg = warp >> 2;                      // 0: channels [0, 64), tokens [0, 32);  1: the other halves + outputs
        const int r = tid & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const int cbase = wg * 64;                     // this warpgroup's channels (columns of S^T)
        // initial state: S[c][r] for this warpgroup's c
        {
            const float* src = slot_in >= 0 ? p.state_pool + ((size_t)slot_in * H + head) * head_floats + r : nullptr;
#pragma unroll 1
            for (int c0 = cbase; c0 < cbase + 64; c0 += 32) {
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
            for (int c0 = cbase; c0 < cbase + 64; c0 += 32) {
                float x[32];
                tmem_ld32(lane_addr + kColS + c0, reinterpret_cast<uint32_t*>(x));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) dst[(size_t)(c0 + i) * kD] = x[i];
            }
        };
        // outputs of a finished step (second warpgroup): rows [a, b) of the block, from result region `n`.  A thread
        // holds one value column of all 64 tokens; the tile is turned round in shared memory so that global memory
        // sees 16-byte stores of whole rows.
        uint32_t ph_o = 0;
        __nv_bfloat16* s_out = reinterpret_cast<__nv_bfloat16*>(sm + CS::kOffOut);
        auto write_outputs = [&](int a, int b, int64_t row_t0, int n) -> bool {
            const bool oko = mbar_wait(bOReady, ph_o, abort_flag);
            if (!__all_sync(0xffffffffu, oko)) return false;
            ph_o ^= 1u;
            tc_fence_after();
            float o[64];
            tmem_ld32(lane_addr + col_d(n) + 64, reinterpret_cast<uint32_t*>(o));
            tmem_ld32(lane_addr + col_d(n) + 96, reinterpret_cast<uint32_t*>(o) + 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bOFree(n));
#pragma unroll
            for (int t = 0; t < kL; ++t) s_out[t * kD + r] = __float2bfloat16_rn(o[t]);
            named_bar(1, 128);
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const int item = it * 128 + r, t = item >> 4, c0 = (item & 15) * 8;
                if (t >= a && t < b)
                    *reinterpret_cast<uint4*>(p.out + ((row_t0 + t) * H + head) * kD + c0) =
                        *reinterpret_cast<const uint4*>(s_out + t * kD + c0);
            }
            named_bar(1, 128);                   // the tile may be overwritten by the next step's outputs
            return true;
        };
        Ring step = {0, 0};
        uint32_t ph_x = 0, ph_s = 0, ph_u0 = 0;
        bool s_pending = false;          // an S_b product is in flight: wait for it before touching S
        bool dead = false;
        int prev_a = -1, prev_b = -1;    // the step whose outputs are still to be written
        int64_t prev_row = 0;
        int n = 0;
        while (!dead) {
            const bool okw = mbar_wait(bStepFull(step.stage), step.phase, abort_flag);
            if (!__all_sync(0xffffffffu, okw)) { dead = true; break; }
            const int slot_ring = step.stage;
            const int a = s_rec[slot_ring].a, b = s_rec[slot_ring].b;
            const bool first = s_rec[slot_ring].first, last = s_rec[slot_ring].last;
            const int store_slot = s_rec[slot_ring].store_slot;
            const int64_t row_t0 = s_rec[slot_ring].row_t0;
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
            {
                float x[64];
                tmem_ld32(lane_addr + kColS + cbase, reinterpret_cast<uint32_t*>(x));
                tmem_ld32(lane_addr + kColS + cbase + 32, reinterpret_cast<uint32_t*>(x) + 32);
                tmem_wait_ld();
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int i4 = 0; i4 < 16; ++i4) {
                    const float4 al = *reinterpret_cast<const float4*>(v_alpha + cbase + 4 * i4);
                    const float4 en = *reinterpret_cast<const float4*>(v_end + cbase + 4 * i4);
                    const float2 ya = __fmul2_rn(make_float2(x[4 * i4], x[4 * i4 + 1]), make_float2(al.x, al.y));
                    const float2 yb = __fmul2_rn(make_float2(x[4 * i4 + 2], x[4 * i4 + 3]), make_float2(al.z, al.w));
                    split2(ya.x, ya.y, hi[2 * i4], lo[2 * i4]);
                    split2(yb.x, yb.y, hi[2 * i4 + 1], lo[2 * i4 + 1]);
                    const float2 za = __fmul2_rn(ya, make_float2(en.x, en.y)), zb = __fmul2_rn(yb, make_float2(en.z, en.w));
                    x[4 * i4] = za.x; x[4 * i4 + 1] = za.y; x[4 * i4 + 2] = zb.x; x[4 * i4 + 3] = zb.y;
                }
                tmem_st32(lane_addr + kColShl + cbase / 2, hi);
                tmem_st32(lane_addr + kColShl + 64 + cbase / 2, lo);
                tmem_st32(lane_addr + kColS + cbase, reinterpret_cast<const uint32_t*>(x));
                tmem_st32(lane_addr + kColS + cbase + 32, reinterpret_cast<const uint32_t*>(x) + 32);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bShlReady);
            mbar_arrive(bStepEmpty(slot_ring));      // the record and its vectors have been consumed
            // ---- U^T = (U0 - X)^T for the step's tokens, zero elsewhere, as the hi/lo operand, in place of X
            if (first) {
                const bool oku = mbar_wait(bU0Full, ph_u0, abort_flag);
                if (!__all_sync(0xffffffffu, oku)) { dead = true; break; }
                ph_u0 ^= 1u;
            }
            {
                const bool okx = mbar_wait(bXReady, ph_x, abort_flag);
                if (!__all_sync(0xffffffffu, okx)) { dead = true; break; }
                ph_x ^= 1u;
            }
            tc_fence_after();
            {
                const int tb = wg * 32;
                float x[32];
                uint32_t hi[16], lo[16];
                tmem_ld32(lane_addr + col_d(n) + tb, reinterpret_cast<uint32_t*>(x));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int t0 = tb + 2 * i;
                    const float u0 = (t0 >= a && t0 < b) ? s_u0[t0 * kD + r] - x[2 * i] : 0.f;
                    const float u1 = (t0 + 1 >= a && t0 + 1 < b) ? s_u0[(t0 + 1) * kD + r] - x[2 * i + 1] : 0.f;
                    split2(u0, u1, hi[i], lo[i]);
                }
                tmem_st8(lane_addr + col_d(n) + tb, hi);
                tmem_st8(lane_addr + col_d(n) + tb + 8, hi + 8);
                tmem_st8(lane_addr + col_d(n) + tb + 16, lo);
                tmem_st8(lane_addr + col_d(n) + tb + 24, lo + 8);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bUhlReady);
            if (last) mbar_arrive(bU0Empty);
            s_pending = true;
            // ---- the second warpgroup writes the previous step's outputs while the state product runs
            if (wg == 1 && prev_a >= 0) {
                if (!write_outputs(prev_a, prev_b, prev_row, n - 1)) { dead = true; break; }
            }
            prev_a = a; prev_b = b; prev_row = row_t0;
            step.advance(kStepRing);
            ++n;
            if (store_slot >= 0) {
                const bool oks = mbar_wait(bSReady, ph_s, abort_flag);
                if (!__all_sync(0xffffffffu, oks)) { dead = true; break; }
                ph_s ^= 1u;
                s_pending = false;
                tc_fence_after();
                store_state(store_slot);
            }
        }
        if (!dead && wg == 1 && prev_a >= 0) dead = !write_outputs(prev_a, prev_b, prev_row, n - 1);
        if (!dead && slot_out >= 0) {
            bool oks = true;
            if (s_pending) oks = mbar_wait(bSReady, ph_s, abort_flag);
            if (__all_sync(0xffffffffu, oks)) {
                tc_fence_after();
                store_state(slot_out);
            }
        }
    }

    // ---- teardown (the second warpgroup has seen the last output product land: nothing is in flight)
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

extern "C" int wpp_launch_kda_tc(const wpp::KdaTcParams* p, const CUtensorMap* maps, int max_blocks, int num_sms,
                                 void* stream) {
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
        PrepMaps pm;
        pm.w0_h = maps[0]; pm.w0_l = maps[1]; pm.qt_h = maps[2]; pm.qt_l = maps[3]; pm.m_h = maps[6]; pm.m_l = maps[7];
        pm.u0 = maps[8]; pm.q = maps[9]; pm.k = maps[10]; pm.v = maps[11]; pm.alpha = maps[12];
        const long long items = (long long)max_blocks * p->num_heads;
        const unsigned grid_a = (unsigned)(items < 2ll * num_sms ? items : 2ll * num_sms);
        kda_tc_prep_kernel<<<grid_a, kPrepThreads, PrepSmem::kBytes, st>>>(pm, *p);
    }
    dim3 grid_b((unsigned)p->num_heads, (unsigned)p->num_requests);
    kda_tc_chain_kernel<<<grid_b, 352, ChainSmem::kBytes, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], maps[6],
                                                               maps[7], *p);
    return (int)cudaGetLastError();
}
