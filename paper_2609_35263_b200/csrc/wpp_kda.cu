// Recurrent-state (KDA) layer of a chunk (Section 3.1): per request and head, token by token,
//     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,     o_t = S_t^T q_t,
// resumed from a snapshot and snapshotted at the chunk end and at periodic boundaries (Section 3.2).
//
// The columns of S evolve independently: with s = S[:, j],
//     s' = alpha * s,    c = beta (v_j - k . s'),    s <- s' + c k,    o_j = q . s' + c (q . k).
// One CTA owns one (request, head).  256 compute threads hold the 128 x 128 fp32 state in registers: a thread has
// four adjacent columns and an eighth of the rows (64 values, packed in pairs for the two-wide fp32 FMA).  The
// shared vectors alpha, k, q reach the registers of every thread that needs them through shared memory, whose
// 128 bytes per clock bound this layout: four columns per thread need 12 sixteen-byte loads per token and thread
// (two columns needed 24 and ran at the shared-memory limit), paid for with an eight-lane reduction per column,
// done as exchange-and-halve steps (4 shuffles for four columns, 3 more to hand the results round).  A ninth warp
// stages the next 32 tokens while the others work: it widens q, k, v to fp32, forms q . k once per token (shared by all 128 columns) and leaves
// them with alpha and beta in shared memory, where the eight row groups read 128 consecutive bytes (no bank
// conflicts) and the four column groups of a warp read the same words (broadcast).  A thread's operands for the
// next token are requested while it still works on this one: the shared-memory latency is off the token chain,
// which is what bounds a recurrence (two warps per scheduler cannot hide it otherwise).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/wpp.h"
#include "wpp_device.h"

namespace wpp {
namespace {

constexpr int kDK = 128, kDV = 128;
constexpr int kComputeWarps = 8;

constexpr int kStageTokens = 32;
constexpr int kThreads = (kComputeWarps + 1) * 32;

struct KdaStage {
    float al[kStageTokens][kDK];    // alpha
    float kk[kStageTokens][kDK];    // k
    float qq[kStageTokens][kDK];    // q
    float v[kStageTokens][kDV];
    float beta[kStageTokens];
    float qk[kStageTokens];         // q . k
};

// Pairs of fp32 values for the two-wide FMA of sm_100 (scalar FMAs were 25 % slower here).
__device__ __forceinline__ float2 pk(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ void upk(float2 v, float& lo, float& hi) {
    lo = v.x;
    hi = v.y;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    return __ffma2_rn(a, b, c);
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
    return __fmul2_rn(a, b);
}
__device__ __forceinline__ void widen4(uint2 raw, float (&f)[4]) {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    f[0] = __low2float(a);
    f[1] = __high2float(a);
    f[2] = __low2float(b);
    f[3] = __high2float(b);
}

// Staging by one warp: n <= 4 tokens starting at absolute row `row` go to slots slot0 .. of the stage; their loads
// are in flight together.  The warp widens q, k, v and forms q . k (shared by all 128 columns).
__device__ __forceinline__ void kda_fill4(const KdaParams& p, KdaStage* st, int64_t row, int slot0, int n, int head, int lane) {
    const int H = p.num_heads;
    uint2 rq[4], rk[4], rv[4];
    float4 ra[4];
    float rb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        if (u < n) {
            const int64_t rh = (row + u) * H + head;
            rq[u] = *reinterpret_cast<const uint2*>(p.q + rh * kDK + lane * 4);
            rk[u] = *reinterpret_cast<const uint2*>(p.k + rh * kDK + lane * 4);
            rv[u] = *reinterpret_cast<const uint2*>(p.v + rh * kDV + lane * 4);
            ra[u] = *reinterpret_cast<const float4*>(p.alpha + rh * kDK + lane * 4);
            rb[u] = p.beta[rh];
        }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        if (u < n) {
            const int t = slot0 + u;
            float q[4], k[4], v[4], part = 0.f;
            widen4(rq[u], q);
            widen4(rk[u], k);
            widen4(rv[u], v);
#pragma unroll
            for (int e = 0; e < 4; ++e) part = fmaf(q[e], k[e], part);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
            *reinterpret_cast<float4*>(&st->al[t][lane * 4]) = ra[u];
            *reinterpret_cast<float4*>(&st->kk[t][lane * 4]) = make_float4(k[0], k[1], k[2], k[3]);
            *reinterpret_cast<float4*>(&st->qq[t][lane * 4]) = make_float4(q[0], q[1], q[2], q[3]);
            *reinterpret_cast<float4*>(&st->v[t][lane * 4]) = make_float4(v[0], v[1], v[2], v[3]);
            if (lane == 0) {
                st->beta[t] = rb[u];
                st->qk[t] = part;
            }
        }
    }
}

// Stage `s` of the request (tokens s * kStageTokens ...), filled by the staging warp four tokens at a time.
__device__ __forceinline__ void kda_fill_stage(const KdaParams& p, KdaStage* st, int64_t row0, int C, int s, int head,
                                               int lane) {
    const int first = s * kStageTokens, n = min(kStageTokens, C - first);
    for (int base = 0; base < n; base += 4) kda_fill4(p, st, row0 + first + base, base, min(4, n - base), head, lane);
}

// kSplit = lanes that share a column's rows.  8: a CTA owns all 128 columns of a (request, head), a thread holds
// 4 columns x 16 rows - the throughput build.  32: a CTA owns 32 columns (four CTAs per head), a thread holds
// 4 columns x 4 rows, so a token costs a quarter of the FMAs per thread and two more shuffle steps - the build for
// waves with too few (request, head) pairs to fill the SMs, where the length of the token chain is all that counts.
template <int kSplit>
__global__ void __launch_bounds__(kThreads, 1) wpp_kda_chunk_kernel(const KdaParams p) {
    constexpr int kM = 32 / kSplit;                      // 16-byte row groups per thread
    constexpr int kQuadsPerWarp = 32 / kSplit;           // column quads per warp
    constexpr int kSlices = kDV / (kComputeWarps * kQuadsPerWarp * 4);
    using Stage = KdaStage;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Stage* stages = reinterpret_cast<Stage*>(smem_raw);

    const int head = blockIdx.x / kSlices, slice = blockIdx.x % kSlices, req = blockIdx.y, H = p.num_heads;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row0 = p.row_offsets[req];
    const int C = (int)(p.row_offsets[req + 1] - row0);
    const int n_stages = (C + kStageTokens - 1) / kStageTokens;

    // slot ids: anything outside [-1, num_slots) is reported and treated as -1
    int slot_in = p.state_in[req], slot_out = p.state_out[req];
    if (slot_in < -1 || slot_in >= p.num_slots || slot_out < -1 || slot_out >= p.num_slots) {
        if (p.status && threadIdx.x == 0) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
        if (slot_in < -1 || slot_in >= p.num_slots) slot_in = -1;
        if (slot_out < -1 || slot_out >= p.num_slots) slot_out = -1;
    }

    if (warp == kComputeWarps) {
        if (n_stages > 0) kda_fill_stage(p, &stages[0], row0, C, 0, head, lane);
        __syncthreads();
        for (int s = 0; s < n_stages; ++s) {
            if (s + 1 < n_stages) kda_fill_stage(p, &stages[(s + 1) & 1], row0, C, s + 1, head, lane);
            __syncthreads();
        }
        return;
    }

    // ---- compute threads: rows 4 kSplit m + 4r + e (m < kM, e < 4; r = lane mod kSplit) of columns 4cq .. 4cq + 3
    const int r = lane & (kSplit - 1), cq = (slice * kComputeWarps + warp) * kQuadsPerWarp + lane / kSplit;
    const bool b0 = lane & 1, b1 = lane & 2;
    const int my_col = (b0 ? 2 : 0) + (b1 ? 1 : 0);                    // the column whose dot products end on this lane
    const size_t head_floats = (size_t)kDK * kDV;
    float2 S[4][kM][2];                                                // [column][m][row pair]
    if (slot_in >= 0) {
        const float* src = p.state_pool + ((size_t)slot_in * H + head) * head_floats + 4 * cq;
#pragma unroll
        for (int m = 0; m < kM; ++m) {
            float4 x[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) x[e] = *reinterpret_cast<const float4*>(src + (size_t)(4 * kSplit * m + 4 * r + e) * kDV);
            S[0][m][0] = pk(x[0].x, x[1].x), S[0][m][1] = pk(x[2].x, x[3].x);
            S[1][m][0] = pk(x[0].y, x[1].y), S[1][m][1] = pk(x[2].y, x[3].y);
            S[2][m][0] = pk(x[0].z, x[1].z), S[2][m][1] = pk(x[2].z, x[3].z);
            S[3][m][0] = pk(x[0].w, x[1].w), S[3][m][1] = pk(x[2].w, x[3].w);
        }
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int m = 0; m < kM; ++m) S[c][m][0] = S[c][m][1] = make_float2(0.f, 0.f);
    }

    auto store_state = [&](int slot) {
        float* dst = p.state_pool + ((size_t)slot * H + head) * head_floats + 4 * cq;
#pragma unroll
        for (int m = 0; m < kM; ++m) {
            float x[4][4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                upk(S[c][m][0], x[c][0], x[c][1]);
                upk(S[c][m][1], x[c][2], x[c][3]);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e)
                *reinterpret_cast<float4*>(dst + (size_t)(4 * kSplit * m + 4 * r + e) * kDV) =
                    make_float4(x[0][e], x[1][e], x[2][e], x[3][e]);
        }
    };

    // Sum over the eight row groups of four per-column partial sums: after two exchange-and-halve steps and one
    // plain step, every lane holds the complete sum of column `my_col` (4 shuffles instead of 12).
    auto reduce_scatter = [&](const float2 (&acc)[4]) -> float {
        float x[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float lo, hi;
            upk(acc[c], lo, hi);
            x[c] = lo + hi;
        }
        const float y0 = (b0 ? x[2] : x[0]) + __shfl_xor_sync(0xffffffffu, b0 ? x[0] : x[2], 1);
        const float y1 = (b0 ? x[3] : x[1]) + __shfl_xor_sync(0xffffffffu, b0 ? x[1] : x[3], 1);
        float z = (b1 ? y1 : y0) + __shfl_xor_sync(0xffffffffu, b1 ? y0 : y1, 2);
        z += __shfl_xor_sync(0xffffffffu, z, 4);
        if (kSplit == 32) {
            z += __shfl_xor_sync(0xffffffffu, z, 8);
            z += __shfl_xor_sync(0xffffffffu, z, 16);
        }
        return z;
    };

    // periodic snapshots: the next sequence position at which one is due
    const int interval = p.snap_interval;
    int64_t pos = 0, next_snap = -1;
    int n_snap = 0;
    if (interval > 0) {
        pos = p.prefix_lens ? p.prefix_lens[req] : 0;
        next_snap = (pos / interval + 1) * (int64_t)interval;
    }

    __nv_bfloat16* out = p.out + (row0 * H + head) * kDV + 4 * cq + my_col;
    __syncthreads();                                                    // stage 0 is filled
    for (int s = 0; s < n_stages; ++s) {
        const Stage* st = &stages[s & 1];
        const int n = min(kStageTokens, C - s * kStageTokens);
        // operands of the stage's first token; after that, each token's are requested one token ahead
        float4 A[kM], K[kM], Q[kM];
#pragma unroll
        for (int m = 0; m < kM; ++m) {
            A[m] = reinterpret_cast<const float4*>(st->al[0])[m * kSplit + r];
            K[m] = reinterpret_cast<const float4*>(st->kk[0])[m * kSplit + r];
            Q[m] = reinterpret_cast<const float4*>(st->qq[0])[m * kSplit + r];
        }
        for (int t = 0; t < n; ++t) {
            const int tn = min(t + 1, n - 1);                          // the last token re-reads itself (unused)
            const float4* al4 = reinterpret_cast<const float4*>(st->al[tn]) + r;
            const float4* kk4 = reinterpret_cast<const float4*>(st->kk[tn]) + r;
            const float4* qq4 = reinterpret_cast<const float4*>(st->qq[tn]) + r;
            const float v_col = st->v[t][4 * cq + my_col];
            const float beta = st->beta[t], qk = st->qk[t];
            float2 d[4], e[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) d[c] = e[c] = make_float2(0.f, 0.f);
#pragma unroll
            for (int m = 0; m < kM; ++m) {
                const float2 a01 = pk(A[m].x, A[m].y), a23 = pk(A[m].z, A[m].w);
                const float2 k01 = pk(K[m].x, K[m].y), k23 = pk(K[m].z, K[m].w);
                const float2 q01 = pk(Q[m].x, Q[m].y), q23 = pk(Q[m].z, Q[m].w);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    S[c][m][0] = mul2(a01, S[c][m][0]);                 // s' = alpha * s
                    S[c][m][1] = mul2(a23, S[c][m][1]);
                    d[c] = fma2(k01, S[c][m][0], d[c]);                 // k . s'
                    d[c] = fma2(k23, S[c][m][1], d[c]);
                    e[c] = fma2(q01, S[c][m][0], e[c]);                 // q . s'
                    e[c] = fma2(q23, S[c][m][1], e[c]);
                }
                A[m] = al4[m * kSplit];
                Q[m] = qq4[m * kSplit];
            }
            // c = beta (v - k . s') for this lane's column, then all four columns' values to every lane
            const float c_mine = beta * (v_col - reduce_scatter(d));
            const float c_pair = __shfl_xor_sync(0xffffffffu, c_mine, 2);
            const float lo = b1 ? c_pair : c_mine, hi = b1 ? c_mine : c_pair;        // columns 2 b0 and 2 b0 + 1
            const float lo_x = __shfl_xor_sync(0xffffffffu, lo, 1), hi_x = __shfl_xor_sync(0xffffffffu, hi, 1);
            const float cc[4] = {b0 ? lo_x : lo, b0 ? hi_x : hi, b0 ? lo : lo_x, b0 ? hi : hi_x};
#pragma unroll
            for (int m = 0; m < kM; ++m) {
                const float2 k01 = pk(K[m].x, K[m].y), k23 = pk(K[m].z, K[m].w);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float2 c2 = pk(cc[c], cc[c]);
                    S[c][m][0] = fma2(c2, k01, S[c][m][0]);             // s = s' + c k
                    S[c][m][1] = fma2(c2, k23, S[c][m][1]);
                }
                K[m] = kk4[m * kSplit];
            }
            const float o_col = fmaf(c_mine, qk, reduce_scatter(e));
            if (!(lane & (kSplit - 1) & ~3)) out[(size_t)(s * kStageTokens + t) * H * kDV] = __float2bfloat16_rn(o_col);
            if (interval > 0) {
                ++pos;
                if (pos == next_snap) {
                    if (p.snap_slots && n_snap < p.max_snaps) {
                        const int slot = p.snap_slots[(size_t)req * p.max_snaps + n_snap];
                        if (slot >= 0 && slot < p.num_slots) {
                            store_state(slot);
                        } else if (slot != -1 && p.status && threadIdx.x == 0) {
                            atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
                        }
                    }
                    ++n_snap;
                    next_snap += interval;
                }
            }
        }
        __syncthreads();
    }
    if (slot_out >= 0) store_state(slot_out);
}

}  // namespace
}  // namespace wpp

template <int kSplit>
static int launch_kda(const wpp::KdaParams* p, void* stream) {
    static bool attr_set[64] = {};
    const int smem = 2 * (int)sizeof(wpp::KdaStage);
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(wpp::wpp_kda_chunk_kernel<kSplit>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             smem);
        if (e != cudaSuccess) return (int)e;
        attr_set[dev] = true;
    }
    dim3 grid((unsigned)p->num_heads * (kSplit == 32 ? 4 : 1), (unsigned)p->num_requests);
    wpp::wpp_kda_chunk_kernel<kSplit><<<grid, wpp::kThreads, smem, (cudaStream_t)stream>>>(*p);
    return (int)cudaGetLastError();
}

// layout: 0 = choose (the column-sliced build when its four CTAs per (request, head) pair still fit the SMs in one
// round: measured, 1 x 16,384 tokens x 32 heads 5.3 ms against 7.3 ms, but 2 x 8,192 5.3 ms against 3.7 ms),
// 1 = one CTA per (request, head), 2 = four CTAs per (request, head).
extern "C" int wpp_launch_kda(const wpp::KdaParams* p, int num_sms, int layout, void* stream) {
    const long long pairs = (long long)p->num_heads * p->num_requests;
    const bool sliced = layout == 2 || (layout == 0 && 4 * pairs <= num_sms);
    return sliced ? launch_kda<32>(p, stream) : launch_kda<8>(p, stream);
}
