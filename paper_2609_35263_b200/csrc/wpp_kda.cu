// Recurrent-state (KDA) layer of a chunk (Section 3.1): per request and head, token by token,
//     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,     o_t = S_t^T q_t,
// resumed from a snapshot and snapshotted at the chunk end and at periodic boundaries (Section 3.2).
//
// The columns of S evolve independently: with s = S[:, j], d = (k*alpha) . s and c = v_j - d,
//     s <- alpha * s + c * (beta k),        o_j = (q*alpha) . s_old + c * (q . beta k).
// One CTA owns one (request, head).  256 compute threads hold the 128 x 128 fp32 state in registers: a thread has
// two adjacent columns and a quarter of the rows (64 values, packed in pairs for the two-wide fp32 FMA), so a dot
// product over d_k is 16 packed FMAs per column and two shuffles.  A ninth warp stages the next 16 tokens while
// the others work: it widens q, k, v, forms k*alpha, q*alpha, beta*k and q . (beta k) once per token (shared by
// all 128 columns) and leaves them in shared memory, where the four row quarters read 64 consecutive bytes
// (no bank conflicts) and the eight column pairs of a warp read the same words (broadcast).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/wpp.h"
#include "wpp_device.h"

namespace wpp {
namespace {

constexpr int kDK = 128, kDV = 128;
constexpr int kStageTokens = 16;
constexpr int kComputeWarps = 8;
constexpr int kThreads = (kComputeWarps + 1) * 32;

struct KdaStage {
    float ka[kStageTokens][kDK];    // k * alpha
    float qa[kStageTokens][kDK];    // q * alpha
    float kb[kStageTokens][kDK];    // beta * k
    float al[kStageTokens][kDK];    // alpha
    float v[kStageTokens][kDV];
    float qkb[kStageTokens];        // q . (beta k)
    float pad[kStageTokens];
};

__device__ __forceinline__ uint64_t pk(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float quad_sum(uint64_t a, uint64_t b) {      // lanes of a row-quarter group: xor 1, 2
    float lo, hi;
    upk(add2(a, b), lo, hi);
    float x = lo + hi;
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    return x;
}
__device__ __forceinline__ void widen4(uint2 raw, float (&f)[4]) {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    f[0] = __low2float(a);
    f[1] = __high2float(a);
    f[2] = __low2float(b);
    f[3] = __high2float(b);
}

// The staging warp: tokens [first, first + n) of the request (rows row0 + first ...), four at a time so that
// their loads are in flight together.
__device__ __forceinline__ void kda_fill(const KdaParams& p, KdaStage* st, int64_t row0, int first, int n, int head,
                                         int lane) {
    const int H = p.num_heads;
    for (int base = 0; base < n; base += 4) {
        uint2 rq[4], rk[4], rv[4];
        float4 ra[4];
        float rb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int t = base + u;
            if (t < n) {
                const int64_t rh = (row0 + first + t) * H + head;
                rq[u] = *reinterpret_cast<const uint2*>(p.q + rh * kDK + lane * 4);
                rk[u] = *reinterpret_cast<const uint2*>(p.k + rh * kDK + lane * 4);
                rv[u] = *reinterpret_cast<const uint2*>(p.v + rh * kDV + lane * 4);
                ra[u] = *reinterpret_cast<const float4*>(p.alpha + rh * kDK + lane * 4);
                rb[u] = p.beta[rh];
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int t = base + u;
            if (t < n) {
                float q[4], k[4], v[4];
                widen4(rq[u], q);
                widen4(rk[u], k);
                widen4(rv[u], v);
                const float a[4] = {ra[u].x, ra[u].y, ra[u].z, ra[u].w};
                float ka[4], qa[4], kb[4], part = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    ka[e] = k[e] * a[e];
                    qa[e] = q[e] * a[e];
                    kb[e] = rb[u] * k[e];
                    part = fmaf(q[e], kb[e], part);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                *reinterpret_cast<float4*>(&st->ka[t][lane * 4]) = make_float4(ka[0], ka[1], ka[2], ka[3]);
                *reinterpret_cast<float4*>(&st->qa[t][lane * 4]) = make_float4(qa[0], qa[1], qa[2], qa[3]);
                *reinterpret_cast<float4*>(&st->kb[t][lane * 4]) = make_float4(kb[0], kb[1], kb[2], kb[3]);
                *reinterpret_cast<float4*>(&st->al[t][lane * 4]) = ra[u];
                *reinterpret_cast<float4*>(&st->v[t][lane * 4]) = make_float4(v[0], v[1], v[2], v[3]);
                if (lane == 0) st->qkb[t] = part;
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1) wpp_kda_chunk_kernel(const KdaParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    KdaStage* stages = reinterpret_cast<KdaStage*>(smem_raw);

    const int head = blockIdx.x, req = blockIdx.y, H = p.num_heads;
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
        if (n_stages > 0) kda_fill(p, &stages[0], row0, 0, min(kStageTokens, C), head, lane);
        __syncthreads();
        for (int s = 0; s < n_stages; ++s) {
            if (s + 1 < n_stages)
                kda_fill(p, &stages[(s + 1) & 1], row0, (s + 1) * kStageTokens, min(kStageTokens, C - (s + 1) * kStageTokens),
                         head, lane);
            __syncthreads();
        }
        return;
    }

    // ---- compute threads: rows 16m + 4r + e (m < 8, e < 4) of columns 2cp and 2cp + 1
    const int r = lane & 3, cp = warp * 8 + (lane >> 2);
    const size_t head_floats = (size_t)kDK * kDV;
    uint64_t sA[8][2], sB[8][2];
    if (slot_in >= 0) {
        const float* src = p.state_pool + ((size_t)slot_in * H + head) * head_floats + 2 * cp;
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            float2 x[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) x[e] = *reinterpret_cast<const float2*>(src + (size_t)(16 * m + 4 * r + e) * kDV);
            sA[m][0] = pk(x[0].x, x[1].x);
            sA[m][1] = pk(x[2].x, x[3].x);
            sB[m][0] = pk(x[0].y, x[1].y);
            sB[m][1] = pk(x[2].y, x[3].y);
        }
    } else {
#pragma unroll
        for (int m = 0; m < 8; ++m) sA[m][0] = sA[m][1] = sB[m][0] = sB[m][1] = 0ull;
    }

    auto store_state = [&](int slot) {
        float* dst = p.state_pool + ((size_t)slot * H + head) * head_floats + 2 * cp;
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            float a[4], b[4];
            upk(sA[m][0], a[0], a[1]);
            upk(sA[m][1], a[2], a[3]);
            upk(sB[m][0], b[0], b[1]);
            upk(sB[m][1], b[2], b[3]);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                *reinterpret_cast<float2*>(dst + (size_t)(16 * m + 4 * r + e) * kDV) = make_float2(a[e], b[e]);
        }
    };

    // periodic snapshots: the next sequence position at which one is due
    const int interval = p.snap_interval;
    int64_t pos = 0, next_snap = -1;
    int n_snap = 0;
    if (interval > 0) {
        pos = p.prefix_lens ? p.prefix_lens[req] : 0;
        next_snap = (pos / interval + 1) * (int64_t)interval;
    }

    __nv_bfloat16* out = p.out + (row0 * H + head) * kDV + 2 * cp;
    __syncthreads();                                                    // stage 0 is filled
    for (int s = 0; s < n_stages; ++s) {
        const KdaStage* st = &stages[s & 1];
        const int n = min(kStageTokens, C - s * kStageTokens);
        for (int t = 0; t < n; ++t) {
            const float4* ka4 = reinterpret_cast<const float4*>(st->ka[t]) + r;
            const float4* qa4 = reinterpret_cast<const float4*>(st->qa[t]) + r;
            uint64_t dA0 = 0, dA1 = 0, dB0 = 0, dB1 = 0, eA0 = 0, eA1 = 0, eB0 = 0, eB1 = 0;
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const float4 a = ka4[m * 4], b = qa4[m * 4];
                const uint64_t a01 = pk(a.x, a.y), a23 = pk(a.z, a.w), b01 = pk(b.x, b.y), b23 = pk(b.z, b.w);
                dA0 = fma2(a01, sA[m][0], dA0);
                dA1 = fma2(a23, sA[m][1], dA1);
                dB0 = fma2(a01, sB[m][0], dB0);
                dB1 = fma2(a23, sB[m][1], dB1);
                eA0 = fma2(b01, sA[m][0], eA0);
                eA1 = fma2(b23, sA[m][1], eA1);
                eB0 = fma2(b01, sB[m][0], eB0);
                eB1 = fma2(b23, sB[m][1], eB1);
            }
            const float2 vv = *reinterpret_cast<const float2*>(&st->v[t][2 * cp]);
            const float cA = vv.x - quad_sum(dA0, dA1), cB = vv.y - quad_sum(dB0, dB1);
            const uint64_t cA2 = pk(cA, cA), cB2 = pk(cB, cB);
            const float4* kb4 = reinterpret_cast<const float4*>(st->kb[t]) + r;
            const float4* al4 = reinterpret_cast<const float4*>(st->al[t]) + r;
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const float4 kb = kb4[m * 4], al = al4[m * 4];
                const uint64_t k01 = pk(kb.x, kb.y), k23 = pk(kb.z, kb.w), l01 = pk(al.x, al.y), l23 = pk(al.z, al.w);
                sA[m][0] = fma2(l01, sA[m][0], mul2(k01, cA2));
                sA[m][1] = fma2(l23, sA[m][1], mul2(k23, cA2));
                sB[m][0] = fma2(l01, sB[m][0], mul2(k01, cB2));
                sB[m][1] = fma2(l23, sB[m][1], mul2(k23, cB2));
            }
            const float qkb = st->qkb[t];
            const float oA = fmaf(cA, qkb, quad_sum(eA0, eA1)), oB = fmaf(cB, qkb, quad_sum(eB0, eB1));
            if (r == 0)
                *reinterpret_cast<__nv_bfloat162*>(out + (size_t)(s * kStageTokens + t) * H * kDV) =
                    __floats2bfloat162_rn(oA, oB);
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

extern "C" int wpp_launch_kda(const wpp::KdaParams* p, void* stream) {
    static bool attr_set[64] = {};
    const int smem = 2 * (int)sizeof(wpp::KdaStage);
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(wpp::wpp_kda_chunk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return (int)e;
        attr_set[dev] = true;
    }
    dim3 grid((unsigned)p->num_heads, (unsigned)p->num_requests);
    wpp::wpp_kda_chunk_kernel<<<grid, wpp::kThreads, smem, (cudaStream_t)stream>>>(*p);
    return (int)cudaGetLastError();
}
