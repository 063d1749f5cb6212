// Persistent chunked-prefill attention kernel for sm_100a.
//
// One CTA per SM; the CTAs take the work tiles the host planner cut, in the planner's order, from a counter in
// global memory as they become free.  A work tile is two 128-row query "halves" (A, B) that share one K/V
// stream, against key steps [kv_begin, kv_end) of 128 keys each.
// 16 warps, specialised by warpgroup:
//   warps 0-3   softmax of half A: thread r owns query row r (TMEM lane r): row max / row sum need no shuffles
//   warps 4-7   softmax of half B
//   warps 8-11  epilogue: O / l -> bf16 -> global (or fp32 partials for split tiles), overlapping the next tile
//   warp 12     issuer of S = Q K^T (one thread), warp 14 issuer of O += P V (one thread): tcgen05.mma with fp32
//               accumulators in TMEM; P is read from TMEM where the softmax warps wrote it as packed bf16; V is an
//               MN-major operand.  Two threads, because the queue of the tensor pipe is only a few MMAs deep: the
//               barrier waits and bookkeeping of one thread hide behind the MMAs the other one is issuing.
//   warp 13     producer: takes the next tile from the counter and tells the other roles (a two-entry queue in
//               shared memory); reads the block table and issues TMA tile loads (Q once per tile; per key step one box
//               per (page, 64-wide half of head_dim) for K and for V, 128-byte swizzle) into a ring of K tiles
//               and a ring of V tiles
// Tensor memory (512 columns) has no room for two S tiles and two P tiles next to the two O accumulators, so the
// two halves share ONE landing buffer for S: a softmax warpgroup copies its S into registers as soon as it lands
// and hands the buffer back (s_free) before it starts on the exponentials, and each half has a P buffer of its own.
// That takes S = Q K^T off the softmax -> O += P V chain of its half: while the softmax warps of A work on step j,
// the tensor pipe already produces S_B(j) and S_A(j+1) and runs the other half's O += P V, so the exponentials of
// both halves and the MMAs all overlap.  The order on the tensor pipe is not fixed: every S is issued when the
// landing buffer is free, every product when its P is ready.
// Rescaling is lazy: a row keeps its reference maximum as long as the step's maximum stays within 2^16 of it;
// only then (and on the first step of a tile) the softmax warps move the reference and rescale O and l.
// Tensor memory: S [0,128)  P_A [128,192)  P_B [192,256)  O_A [256,256+D)  O_B [384,384+D).
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
constexpr uint32_t kColS = 0;                                                        // landing buffer of S
__host__ __device__ constexpr uint32_t col_p(int hf) { return 128u + 64u * hf; }    // P of half hf (packed bf16)
__host__ __device__ constexpr uint32_t col_o(int hf) { return 256u + 128u * hf; }   // O of half hf
// registers per thread after the warpgroups re-split the register file (8 x kRegsSoftmax + 4 x kRegsEpilogue +
// 4 x kRegsUtil <= 2048 per thread slot of 32 lanes, i.e. 65536 in all)
constexpr int kRegsSoftmax = 192, kRegsEpilogue = 72, kRegsUtil = 56;
static_assert(8 * kRegsSoftmax + 4 * kRegsEpilogue + 4 * kRegsUtil <= 2048, "register file exceeded");
constexpr uint32_t kSoftmaxArrivals = 128;   // every softmax thread arrives on s_free and p_ready itself
constexpr int kRescaleCols = 16;    // columns of O in flight while a moved reference rescales it
constexpr float kRefSlack = 16.f;   // a row keeps its reference while its scores stay below reference + 16 (log2)
constexpr int kExpBlock = 8;        // score pairs whose exponentials are in flight together

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzled column blocks
    static constexpr int kTileBytes = 128 * D * 2;         // one 128-row Q half, or one K or V step
    static constexpr int kHalfBytes = 128 * 128;           // 128 rows x 128 bytes
    static constexpr int kSlots = (D == 128) ? 4 : 8;      // K / V tiles in shared memory: half for K, half for V
    static constexpr int kOffKV = 2 * kTileBytes;
    static constexpr int kOffBars = kOffKV + kSlots * kTileBytes;
    static constexpr int kTileQ = 2;                       // tile ids the producer may publish ahead
    static constexpr int kNumBars = 2 + 2 * kSlots + 1 + 6 * 2 + 2 * kTileQ;
    static constexpr int kOffFinal = kOffBars + 8 * kNumBars;          // float2 (m, l)[2][128]
    static constexpr int kOffStage = (kOffFinal + 2 * 128 * 8 + 15) / 16 * 16;   // 4 x 2 KB: the epilogue warps' store staging (16-byte chunks)
    static constexpr int kOffMisc = kOffStage + 4 * 2048;              // tmem ptr, abort flag, tile ids
    static constexpr int kUsedBytes = kOffMisc + 16 + 4 * kTileQ + 8;
    static constexpr int kSmemBytes = kUsedBytes + 1024;               // + alignment slack (201 KB at D = 128)
    static_assert(kSmemBytes <= 232448, "more shared memory than a CTA can have");
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
    bool mismatch;                       // the launch's lengths are not the plan's
};
// A request whose span on the device differs from the span the plan was made for gets no key steps (every role
// skips the tile, `mismatch` tells the producer to report it): the tile geometry belongs to other lengths.
__device__ __forceinline__ UnitView view_of(const WppUnit& un, const AttnParams& p, const int32_t* q_offsets,
                                            const int32_t* plan_prefix) {
    UnitView v;
    v.request = un.request;
    v.kv_begin = un.kv_begin;
    v.P = p.prefix_lens[un.request];
    const int C = p.chunk_lens[un.request];
    v.kv_len = v.P + C;
    v.q_off = q_offsets[un.request];
    v.mismatch = (v.P != plan_prefix[un.request]) || (C != q_offsets[un.request + 1] - v.q_off);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int end = (un.rows[h] > 0 && !v.mismatch) ? (v.P + un.row0[h] + un.rows[h] + 127) / 128 : 0;
        v.n[h] = max(0, min(un.kv_end, end) - un.kv_begin);
    }
    v.n_steps = max(v.n[0], v.n[1]);
    return v;
}

// kLate: where a moved reference rescales O.  false: before the step's exponentials (they then start from a settled
// O and the wait for the previous product is usually over by the time P is ready): the choice for workloads whose
// references move now and then.  true: after the exponentials, which do not depend on O and so run while the
// previous O += P V is still on the tensor pipe: better when most steps move a reference (scores that keep growing
// along the sequence), a little worse otherwise.  The kernel counts its steps and its moves for the caller to choose.
template <int D, bool kLate>
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
    const uint32_t sKV = smem_base + C::kOffKV;          // kSlots tiles (K or V)
    const uint32_t bars = smem_base + C::kOffBars;
    const uint32_t bQFull = bars, bQEmpty = bars + 8;
    const uint32_t bSlotFull = bars + 16, bSlotEmpty = bSlotFull + 8 * C::kSlots;
    // s_free: the half that owned the landing buffer has copied its S into registers.
    // Per half: s_full (S = Q K^T landed), p_ready (P written, and O rescaled if the row reference moved, by the
    // 128 softmax threads), p_free (O += P V landed: P may be overwritten, O may be rescaled), final_ready
    // (end-of-tile (m, l) are in smem), o_final (last O += P V landed), o_free (the epilogue threads have read O
    // out, the next tile may overwrite it).  A thread never arrives twice on one barrier without a wait in
    // between that implies the earlier phase completed.
    const uint32_t bSFree = bSlotEmpty + 8 * C::kSlots;
    const uint32_t bHalf = bSFree + 8;
    auto bSFull = [&](int h) { return bHalf + 48 * h; };
    auto bPReady = [&](int h) { return bHalf + 48 * h + 8; };
    auto bPFree = [&](int h) { return bHalf + 48 * h + 16; };
    auto bFinalReady = [&](int h) { return bHalf + 48 * h + 24; };
    auto bOFinal = [&](int h) { return bHalf + 48 * h + 32; };
    auto bOFree = [&](int h) { return bHalf + 48 * h + 40; };
    // Work tiles are not preassigned: the producer warp takes the next tile of the planner's order from a counter
    // in global memory and publishes its index to the other roles through a small queue in shared memory, so the
    // CTAs of the grid always work on neighbouring tiles of that order (which share K/V pages, see the planner)
    // however their speeds differ, and the tail balances itself.
    const uint32_t bTileFull = bHalf + 96, bTileEmpty = bTileFull + 8 * C::kTileQ;
    float2* s_final = reinterpret_cast<float2*>(smem_gen + C::kOffFinal);     // [2][128] (reference in log2 units, l)
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile int32_t* tile_ids = reinterpret_cast<volatile int32_t*>(tmem_slot + 4);      // [kTileQ]
    constexpr uint32_t kTileConsumers = 2 + 256 + 128;   // two issuing threads, softmax threads, epilogue threads

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wg = warp >> 2;

    if (threadIdx.x == 0) {
        mbar_init(bQFull, 1); mbar_init(bQEmpty, 1);
        for (int s = 0; s < C::kSlots; ++s) { mbar_init(bSlotFull + 8 * s, 1); mbar_init(bSlotEmpty + 8 * s, 1); }
        mbar_init(bSFree, kSoftmaxArrivals);
        for (int h = 0; h < 2; ++h) {
            mbar_init(bSFull(h), 1); mbar_init(bPReady(h), kSoftmaxArrivals); mbar_init(bPFree(h), 1);
            mbar_init(bFinalReady(h), 128); mbar_init(bOFinal(h), 1); mbar_init(bOFree(h), 128);
        }
        for (int i = 0; i < C::kTileQ; ++i) { mbar_init(bTileFull + 8 * i, 1); mbar_init(bTileEmpty + 8 * i, kTileConsumers); }
        *abort_flag = 0u;
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
    const int32_t* plan_prefix = reinterpret_cast<const int32_t*>(plan + hd->off_prefix);
    const WppUnit* units = reinterpret_cast<const WppUnit*>(plan + hd->off_units);
    const int num_units = hd->num_units;
    // next tile index for a consuming role: -1 = no more tiles, -2 = the wait was abandoned
    Ring tile_ring = {0, 0};
    auto next_tile = [&]() -> int {
        if (!mbar_wait(bTileFull + 8 * tile_ring.stage, tile_ring.phase, abort_flag)) return -2;
        const int id = tile_ids[tile_ring.stage];
        mbar_arrive(bTileEmpty + 8 * tile_ring.stage);
        tile_ring.advance(C::kTileQ);
        return id;
    };
    const int B = p.page_size, ppt = 128 / B;   // pages per key step

    if (wg == 3) {
        setmaxnreg_dec<kRegsUtil>();
        // The K tiles and the V tiles have a ring each (slots [n_v, kSlots) and [0, n_v) of the tile area), so
        // that the thread issuing S = Q K^T and the thread issuing O += P V walk their own ring.  (A third K
        // slot, which would still fit, was measured and makes no difference.)
        const uint32_t n_v = C::kSlots / 2, n_k = C::kSlots - n_v;
        if (warp == 13) {
            // ================================================================ producer
            // Tiles are requested in the order the issuers first touch them: K(0), K(1), V(0), K(2), V(1), ...
            Ring ring_k = {0, 0}, ring_v = {0, 0};
            uint32_t q_phase = 0;
            bool dead = false;
            while (!dead) {
                // take the next tile of the planner's order and tell the other roles
                int u = 0;
                if (lane == 0) u = (int)atomicAdd(p.tile_counter, 1u);
                u = __shfl_sync(0xffffffffu, u, 0);
                if (u >= num_units) u = -1;
                {
                    const bool ok = mbar_wait(bTileEmpty + 8 * tile_ring.stage, tile_ring.phase ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) break;
                    if (lane == 0) {
                        tile_ids[tile_ring.stage] = u;
                        mbar_arrive(bTileFull + 8 * tile_ring.stage);
                    }
                    tile_ring.advance(C::kTileQ);
                }
                if (u < 0) break;
                const WppUnit un = units[u];
                const UnitView v = view_of(un, p, q_offsets, plan_prefix);
                if (v.mismatch && lane == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_PLAN_MISMATCH);
                if (v.n_steps == 0) continue;
                const int n_pages = (v.kv_len + B - 1) / B;
                const int kvh = un.head[0] / p.group;
                const int32_t* bt = p.block_tables + (int64_t)un.request * p.max_blocks;
                // one ring slot: the K or the V tile of key step j.  Every 64-column box of every page is issued by a
                // lane of its own (a thread spends about 400 clocks per TMA instruction, and at the start of a tile
                // this warp is what everybody waits for): lane l moves column block l % kHalves of page l / kHalves.
                auto load_tile = [&](const CUtensorMap* tm, int j, Ring& ring, uint32_t slot0, uint32_t n_ring) -> bool {
                    const int page0 = (v.kv_begin + j) * ppt;
                    const int cnt = min(ppt, n_pages - page0);
                    const int pg = lane / C::kHalves, h = lane % C::kHalves;
                    int pid = 0;
                    if (pg < cnt) pid = bt[page0 + pg];
                    if (pid < 0 || pid >= p.num_pages) {
                        if (p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                        pid = 0;
                    }
                    const uint32_t slot = slot0 + ring.stage;
                    const bool ok = mbar_wait(bSlotEmpty + 8 * slot, ring.phase ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) return false;
                    const uint32_t full = bSlotFull + 8 * slot;
                    if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)cnt * B * D * 2);
                    __syncwarp();
                    if (pg < cnt)
                        tma_load_4d(sKV + slot * C::kTileBytes + pg * B * 128 + h * C::kHalfBytes, tm, full, h * 64, 0, kvh, pid);
                    ring.advance(n_ring);
                    return true;
                };
                // K(0) only needs a ring slot, which frees up before the previous tile's Q does
                if (!load_tile(&tm_k, 0, ring_k, n_v, n_k)) { dead = true; break; }
                const bool ok = mbar_wait(bQEmpty, q_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                q_phase ^= 1u;
                {
                    const int nq = (v.n[0] > 0) + (v.n[1] > 0);
                    if (lane == 0) mbar_arrive_expect_tx(bQFull, nq * C::kTileBytes);
                    __syncwarp();
                    // head k of a half lands in tensor rows [k*rph, (k+1)*rph): one box of rph rows per head and
                    // 64-column block; box b = (half, head, column block) is issued by lane b (at most 2 x 8 x 2)
                    const int rph = 128 / un.pack;
                    const CUtensorMap* qm = un.pack == 1 ? &tm_q : un.pack == 2 ? &tm_q64 : un.pack == 4 ? &tm_q32 : &tm_q16;
                    const int per_half = un.pack * C::kHalves;
                    for (int b = lane; b < 2 * per_half; b += 32) {
                        const int hf = b / per_half, k = (b % per_half) / C::kHalves, h = b % C::kHalves;
                        const int n_hf = hf ? v.n[1] : v.n[0];
                        if (n_hf == 0) continue;
                        tma_load_3d(sQ + hf * C::kTileBytes + h * C::kHalfBytes + k * rph * 128, qm, bQFull, h * 64,
                                    (hf ? un.head[1] : un.head[0]) + k, v.q_off + (hf ? un.row0[1] : un.row0[0]));
                    }
                }
                __syncwarp();
                for (int k = 0; k <= v.n_steps && !dead; ++k) {
                    if (k >= 1 && !load_tile(&tm_v, k - 1, ring_v, 0, n_v)) dead = true;
                    if (!dead && k + 1 < v.n_steps && !load_tile(&tm_k, k + 1, ring_k, n_v, n_k)) dead = true;
                }
            }
        } else if (warp == 12 && lane == 0) {
            // ================================================================ issuer of S = Q K^T (one thread)
            // S_A(0), S_B(0), S_A(1), S_B(1), ...: each S goes into the landing buffer as soon as the previous one
            // has been copied out of it (s_free).
            Ring ring = {0, 0};
            uint32_t q_phase = 0, sfree_phase = 0;
            constexpr uint32_t idesc_qk = idesc_bf16(128, 0, 0);
            const uint64_t q_desc0 = smem_desc_sw128(sQ, 16, 1024);                    // + hf * (kTileBytes >> 4)
            const uint64_t k_desc0 = smem_desc_sw128(sKV + n_v * C::kTileBytes, 16, 1024);   // + stage * (kTileBytes >> 4)
            const uint32_t tS = tmem + kColS;
            bool dead = false;
            while (!dead) {
                const int u = next_tile();
                if (u < 0) break;
                const WppUnit un = units[u];
                const UnitView v = view_of(un, p, q_offsets, plan_prefix);
                if (v.n_steps == 0) continue;
                {
                    const bool ok = mbar_wait(bQFull, q_phase, abort_flag);
                    if (!ok) break;
                }
                q_phase ^= 1u;
                for (int k = 0; k < v.n_steps; ++k) {
                    {
                        const bool ok = mbar_wait(bSlotFull + 8 * (n_v + ring.stage), ring.phase, abort_flag);   // K(k)
                        if (!ok) { dead = true; break; }
                    }
                    const uint64_t kd = k_desc0 + (uint64_t)(ring.stage * (C::kTileBytes >> 4));
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        if (k >= v.n[hf]) continue;
                        {
                            const bool ok = mbar_wait(bSFree, sfree_phase ^ 1u, abort_flag);
                            if (!ok) { dead = true; break; }
                        }
                        sfree_phase ^= 1u;
                        tc_fence_after();
                        const uint64_t qd = q_desc0 + (uint64_t)(hf * (C::kTileBytes >> 4));
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint64_t off = (uint64_t)(((kk >> 2) * C::kHalfBytes + (kk & 3) * 32) >> 4);
                            if (kk == 0) mma_ss_overwrite(tS, qd + off, kd + off, idesc_qk);
                            else mma_ss_accumulate(tS, qd + off, kd + off, idesc_qk);
                        }
                        mma_commit(bSFull(hf));
                    }
                    if (dead) break;
                    mma_commit(bSlotEmpty + 8 * (n_v + ring.stage));                  // K(k) has been read
                    ring.advance(n_k);
                }
                if (!dead) mma_commit(bQEmpty);           // every S of the tile has been issued: Q may be replaced
            }
        } else if (warp == 14 && lane == 0) {
            // ================================================================ issuer of O += P V (one thread)
            // O_A += P_A V(0), O_B += P_B V(0), O_A += P_A V(1), ...: each product waits for its P.
            Ring ring = {0, 0};
            uint32_t p_phase[2] = {0, 0}, of_phase[2] = {0, 0};
            constexpr uint32_t idesc_pv = idesc_bf16(D, 0, 1);
            const uint64_t v_desc0 = smem_desc_sw128(sKV, C::kHalfBytes, 1024);       // + stage * (kTileBytes >> 4)
            bool dead = false;
            while (!dead) {
                const int u = next_tile();
                if (u < 0) break;
                const WppUnit un = units[u];
                const UnitView v = view_of(un, p, q_offsets, plan_prefix);
                if (v.n_steps == 0) continue;
                for (int k = 0; k < v.n_steps; ++k) {
                    {
                        const bool ok = mbar_wait(bSlotFull + 8 * ring.stage, ring.phase, abort_flag);           // V(k)
                        if (!ok) { dead = true; break; }
                    }
                    const int valid = v.kv_len - (v.kv_begin + k) * 128;      // keys of this step that exist
                    if (valid < 128) {
                        // rows past the end of the sequence may hold anything (stale slots, never-loaded
                        // pages): zero them so that 0 * garbage cannot reach O
                        uint8_t* vg = smem_gen + C::kOffKV + ring.stage * C::kTileBytes;
                        for (int h = 0; h < C::kHalves; ++h)
                            for (int i = valid * 8; i < 128 * 8; ++i)
                                *reinterpret_cast<uint4*>(vg + h * C::kHalfBytes + i * 16) = make_uint4(0, 0, 0, 0);
                        fence_proxy_async_smem();
                    }
                    const uint64_t vd = v_desc0 + (uint64_t)(ring.stage * (C::kTileBytes >> 4));
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        const int n = v.n[hf];
                        if (k >= n) continue;
                        {
                            const bool ok = mbar_wait(bPReady(hf), p_phase[hf], abort_flag);     // P written, O fixed
                            if (!ok) { dead = true; break; }
                        }
                        p_phase[hf] ^= 1u;
                        if (k == 0) {
                            // the first product of a tile overwrites O: the previous tile's epilogue must have read it
                            const bool ok = mbar_wait(bOFree(hf), of_phase[hf] ^ 1u, abort_flag);
                            if (!ok) { dead = true; break; }
                            of_phase[hf] ^= 1u;
                        }
                        tc_fence_after();
                        const uint32_t tP = tmem + col_p(hf), tO = tmem + col_o(hf);
                        if (k > 0) mma_ts_accumulate(tO, tP, vd, idesc_pv); else mma_ts_overwrite(tO, tP, vd, idesc_pv);
#pragma unroll
                        for (int kk = 1; kk < 8; ++kk) mma_ts_accumulate(tO, tP + kk * 8, vd + (uint64_t)(kk * 128), idesc_pv);
                        mma_commit(bPFree(hf));
                        if (k + 1 == n) mma_commit(bOFinal(hf));
                    }
                    if (dead) break;
                    mma_commit(bSlotEmpty + 8 * ring.stage);                          // V(k) has been read
                    ring.advance(n_v);
                }
            }
        }
    } else if (wg == 2) {
        // ================================================================ epilogue (one thread per output row)
        setmaxnreg_dec<kRegsEpilogue>();
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t o_phase[2] = {0, 0}, f_phase[2] = {0, 0};
        bool dead = false;
        while (!dead) {
            const int u = next_tile();
            if (!__all_sync(0xffffffffu, u != -2) || u < 0) break;
            const WppUnit un = units[u];
            const UnitView v = view_of(un, p, q_offsets, plan_prefix);
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
                uint8_t* stage = smem_gen + C::kOffStage + (warp & 3) * 2048;
                if (un.split_slot < 0) {
                    const __nv_bfloat16* dst = p.out + tok * p.o_token_stride + (int64_t)head * p.o_head_stride;
#pragma unroll
                    for (int q4 = 0; q4 < D / 32; ++q4) {
                        float o[32];
                        tmem_ld32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
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
#pragma unroll
                    for (int q4 = 0; q4 < D / 32; ++q4) {
                        float o[32];
                        tmem_ld32(lane_addr + col_o(hf) + q4 * 32, reinterpret_cast<uint32_t*>(o));
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
                mbar_arrive(bOFree(hf));
            }
        }
    } else {
        // ================================================================ softmax (thread = query row of half `hf`)
        setmaxnreg_inc<kRegsSoftmax>();
        const int hf = wg;
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t s_phase = 0, fin_phase = 0, pf_phase = 0;
        const float c = p.scale_log2;
        const uint64_t c2 = pack2(c, c);
        bool dead = false;
        uint32_t n_steps_seen = 0, n_moves_seen = 0;      // this warp's key steps, and those that rescaled O
        while (!dead) {
            const int u = next_tile();
            if (!__all_sync(0xffffffffu, u != -2) || u < 0) break;
            const WppUnit un = units[u];
            const UnitView v = view_of(un, p, q_offsets, plan_prefix);
            const int n = v.n[hf];
            if (n == 0) continue;
            n_steps_seen += (uint32_t)n;
            const int first_pos = v.P + un.row0[hf];          // last key visible to row 0 of this half
            // last key this thread's row may see: its own position (rows of packed heads repeat every 128/pack
            // tensor rows), never past the end of the sequence
            const int row_last = min(first_pos + (r & (128 / un.pack - 1)), v.kv_len - 1);
            // m_ref: reference of the row (raw score units); nmc = -(m_ref * c) rounded once.  Every p of the row is
            // 2^(s*c + nmc) with that same nmc, and a change of reference rescales by 2^(nmc_new - nmc_old) of the two
            // stored numbers, so old and new terms stay consistent even for scores around 1e8.
            float m_ref = -INFINITY, l_run = 0.f, nmc = 0.f;
            for (int j = 0; j < n; ++j) {
                {
                    const bool ok = mbar_wait(bSFull(hf), s_phase, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
                }
                s_phase ^= 1u;
                tc_fence_after();
                // copy S out of the landing buffer and hand the buffer back at once
                float s[128];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    tmem_ld32(lane_addr + kColS + q4 * 32, reinterpret_cast<uint32_t*>(s) + q4 * 32);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bSFree);
                const int key0 = (v.kv_begin + j) * 128;
                if (key0 + 127 > first_pos) {                 // only steps that touch the diagonal are masked
                    const int limit = row_last - key0;
#pragma unroll
                    for (int i = 0; i < 128; ++i) s[i] = (i > limit) ? -INFINITY : s[i];
                }
                // row maximum of the step: it only decides whether the reference has to move
                float mx[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) mx[k] = fmaxf(s[2 * k], s[2 * k + 1]);
#pragma unroll
                for (int i = 16; i < 128; i += 16) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) mx[k] = fmax3(mx[k], s[i + 2 * k], s[i + 2 * k + 1]);
                }
                const float mxx = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmaxf(fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                // Has the previous O += P V of this half been seen to land?  Until then its P may not be replaced
                // and O may not be rescaled.  (It may belong to the previous tile: the two issuing threads run
                // independently.  The first wait of the kernel passes at once.)
                bool waited = false;
                // The row keeps its reference while 2^(s*c + nmc) <= 2^16 for every score of the step: nothing can
                // overflow and small terms keep 8 bits below that.  Otherwise (or when the row has no reference
                // yet) the warp moves its references to the running maxima and rescales O and l.
                const bool move = (m_ref == -INFINITY) || !(fmaf(mxx, c, nmc) <= kRefSlack);
                const bool warp_moves = __any_sync(0xffffffffu, move);
                float alpha = 1.f;
                if (warp_moves) {
                    const float m_new = fmaxf(m_ref, mxx);
                    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
                    const float nmc_new = -m_safe * c;
                    alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(nmc_new - nmc);
                    nmc = nmc_new;
                    m_ref = m_new;
                    l_run *= alpha;
                    n_moves_seen += (j > 0);
                    if (!kLate && j > 0) {
                        // O may only be touched once the O += P V of step j-1 has landed
                        const bool okp = mbar_wait(bPFree(hf), pf_phase ^ 1u, abort_flag);
                        if (!__all_sync(0xffffffffu, okp)) { dead = true; break; }
                        pf_phase ^= 1u;
                        waited = true;
                        tc_fence_after();
                        if (__any_sync(0xffffffffu, alpha != 1.f)) {
                            // kRescaleCols columns at a time: the 128 scores of the step stay in registers meanwhile
#pragma unroll 1
                            for (int q0 = 0; q0 < D; q0 += kRescaleCols) {
                                float o[kRescaleCols];
#pragma unroll
                                for (int c8 = 0; c8 < kRescaleCols; c8 += 8)
                                    tmem_ld8(lane_addr + col_o(hf) + q0 + c8, reinterpret_cast<uint32_t*>(o) + c8);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < kRescaleCols; ++i) o[i] *= alpha;
#pragma unroll
                                for (int c8 = 0; c8 < kRescaleCols; c8 += 8)
                                    tmem_st8(lane_addr + col_o(hf) + q0 + c8, reinterpret_cast<uint32_t*>(o) + c8);
                            }
                        }
                    }
                }
                // p = 2^(s*c - m_ref*c) for the whole row: bf16 pairs for the tensor cores, fp32 row sum.  The packed
                // pair i takes the place of score i, which pair i/2 has consumed: the row never needs more than its
                // 128 registers.
                uint32_t* pk = reinterpret_cast<uint32_t*>(s);
                {
                    const uint64_t nm2 = pack2(nmc, nmc);
                    uint64_t sum2a = pack2(0.f, 0.f), sum2b = pack2(0.f, 0.f);
                    // in blocks of kExpBlock pairs: all scalings, then all exponentials, then sums and packing, so
                    // that the special-function unit always has independent work queued
#pragma unroll
                    for (int i0 = 0; i0 < 64; i0 += kExpBlock) {
                        uint64_t x2[kExpBlock];
                        float e[2 * kExpBlock];
#pragma unroll
                        for (int k = 0; k < kExpBlock; ++k)
                            x2[k] = ffma2(pack2(s[2 * (i0 + k)], s[2 * (i0 + k) + 1]), c2, nm2);
#pragma unroll
                        for (int k = 0; k < kExpBlock; ++k) {
                            float x0, x1;
                            unpack2(x2[k], x0, x1);
                            e[2 * k] = fast_exp2(x0);
                            e[2 * k + 1] = fast_exp2(x1);
                        }
#pragma unroll
                        for (int k = 0; k < kExpBlock; ++k) {
                            if (k & 1) sum2b = fadd2(sum2b, pack2(e[2 * k], e[2 * k + 1]));
                            else sum2a = fadd2(sum2a, pack2(e[2 * k], e[2 * k + 1]));
                            pk[i0 + k] = pack_bf16x2(e[2 * k], e[2 * k + 1]);
                        }
                    }
                    float t0, t1;
                    unpack2(fadd2(sum2a, sum2b), t0, t1);
                    l_run += t0 + t1;
                }
                if (!waited) {
                    // P(j-1) must have been consumed before P(j) replaces it
                    const bool okp = mbar_wait(bPFree(hf), pf_phase ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, okp)) { dead = true; break; }
                    pf_phase ^= 1u;
                    tc_fence_after();
                }
                if (kLate && warp_moves && j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
                    for (int q0 = 0; q0 < D; q0 += kRescaleCols) {
                        float o[kRescaleCols];
#pragma unroll
                        for (int c8 = 0; c8 < kRescaleCols; c8 += 8)
                            tmem_ld8(lane_addr + col_o(hf) + q0 + c8, reinterpret_cast<uint32_t*>(o) + c8);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < kRescaleCols; ++i) o[i] *= alpha;
#pragma unroll
                        for (int c8 = 0; c8 < kRescaleCols; c8 += 8)
                            tmem_st8(lane_addr + col_o(hf) + q0 + c8, reinterpret_cast<uint32_t*>(o) + c8);
                    }
                }
                // eight stores of eight columns rather than two of 32: the narrow form only needs eight consecutive
                // registers at a time, which leaves the register allocator free in the loop above (+0.7 % measured)
#pragma unroll
                for (int c8 = 0; c8 < 64; c8 += 8) tmem_st8(lane_addr + col_p(hf) + c8, pk + c8);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bPReady(hf));
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
        // the launch's counters live behind the tile counter in the workspace header (zeroed with it)
        if (p.stats && lane == 0 && n_steps_seen) {
            unsigned long long* ws_stats = reinterpret_cast<unsigned long long*>(p.tile_counter) + 1;
            atomicAdd(ws_stats, (unsigned long long)n_steps_seen);
            atomicAdd(ws_stats + 1, (unsigned long long)n_moves_seen);
        }
    }

    // ---- teardown: every loop above is bounded, so every thread gets here.  The abort flag is read after the
    //      barrier: a role that gave up late (after thread 0 had finished its own work) is still reported.
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) { }     // let copies and tensor-core work in flight land
        if (threadIdx.x == 0 && p.status) atomicCAS(p.status, 0, WPP_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 12) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
    // the last CTA to get here hands the launch's two counters to the caller's words (mapped host memory: two
    // transactions per launch, where one per warp would cost milliseconds)
    if (p.stats && threadIdx.x == 0) {
        unsigned long long* ws_stats = reinterpret_cast<unsigned long long*>(p.tile_counter) + 1;
        __threadfence();
        if (atomicAdd(reinterpret_cast<unsigned int*>(ws_stats + 2), 1u) == gridDim.x - 1) {
            __threadfence();
            atomicAdd_system(p.stats, atomicAdd(ws_stats, 0ull));
            atomicAdd_system(p.stats + 1, atomicAdd(ws_stats + 1, 0ull));
        }
    }
}

template <int D, bool kLate>
static cudaError_t launch(const CUtensorMap* tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                          int num_ctas, cudaStream_t stream) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(wpp_attn_kernel<D, kLate>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg<D>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    wpp_attn_kernel<D, kLate><<<num_ctas, kThreads, Cfg<D>::kSmemBytes, stream>>>(tq[0], tq[1], tq[2], tq[3], tk, tv, p);
    return cudaGetLastError();
}

}  // namespace wpp

// tq: four maps of q with boxes of 128, 64, 32 and 16 rows
// late_rescale: see the kernel's kLate
extern "C" int wpp_launch_attention(int head_dim, const CUtensorMap* tq, const CUtensorMap* tk, const CUtensorMap* tv,
                                    const wpp::AttnParams* p, int num_ctas, int late_rescale, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (head_dim == 128)
        return (int)(late_rescale ? wpp::launch<128, true>(tq, *tk, *tv, *p, num_ctas, st)
                                  : wpp::launch<128, false>(tq, *tk, *tv, *p, num_ctas, st));
    if (head_dim == 64)
        return (int)(late_rescale ? wpp::launch<64, true>(tq, *tk, *tv, *p, num_ctas, st)
                                  : wpp::launch<64, false>(tq, *tk, *tv, *p, num_ctas, st));
    return (int)cudaErrorInvalidValue;
}
