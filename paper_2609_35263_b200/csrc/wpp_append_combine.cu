// KV append (bit-exact 16-byte vector copies into the reserved pages) and the split-KV combine pass.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "wpp_device.h"
#include "wpp_plan_format.h"
#include "wpp_ptx.cuh"

namespace wpp {

// One thread moves one 16-byte vector of K and the matching vector of V.  A vector index decomposes as
// (token, kv head, vector within the head row); the request is found by bisection in the row offsets.
// A request whose span on the device (prefix_lens, chunk_lens) is not the span the plan was made for is refused:
// nothing of it is written and the status word becomes WPP_ERR_PLAN_MISMATCH (Section 4.6: a position mismatch
// fails execution instead of writing against the wrong cache state).
__global__ void __launch_bounds__(256) wpp_append_kernel(const AppendParams p) {
    const char* plan = static_cast<const char*>(p.plan);
    const WppPlanHeader* hd = reinterpret_cast<const WppPlanHeader*>(plan);
    const int32_t* q_offsets = reinterpret_cast<const int32_t*>(plan + hd->off_q_offsets);
    const int32_t* plan_prefix = reinterpret_cast<const int32_t*>(plan + hd->off_prefix);
    const int64_t per_token = (int64_t)p.num_kv_heads * p.vec_per_row;
    const int64_t total = p.total_new_tokens * per_token;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += stride) {
        const int64_t tok = v / per_token;
        const int rem = (int)(v - tok * per_token);
        const int h = rem / p.vec_per_row, c = rem - h * p.vec_per_row;
        int lo = 0, hi = p.num_requests;          // largest i with q_offsets[i] <= tok
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (q_offsets[mid] <= tok) lo = mid; else hi = mid;
        }
        const int P = p.prefix_lens[lo];
        if (P != plan_prefix[lo] || p.chunk_lens[lo] != q_offsets[lo + 1] - q_offsets[lo]) {
            if (p.status) atomicCAS(p.status, 0, WPP_ERR_PLAN_MISMATCH);
            continue;
        }
        const int pos = P + (int)(tok - q_offsets[lo]);
        const int blk = pos / p.page_size, slot = pos - blk * p.page_size;
        const int page = (blk < p.max_blocks) ? p.block_tables[(int64_t)lo * p.max_blocks + blk] : -1;
        if (page < 0 || page >= p.num_pages) {
            if (p.status) atomicCAS(p.status, 0, WPP_ERR_BOUNDS);
            continue;
        }
        const int64_t src = tok * p.kvnew_token_stride + h * p.kvnew_head_stride + c;
        const int64_t dst = page * p.kv_page_stride + h * p.kv_head_stride + slot * p.kv_token_stride + c;
        const uint4 kv = p.k_new[src];
        const uint4 vv = p.v_new[src];
        p.k_cache[dst] = kv;
        p.v_cache[dst] = vv;
    }
}

// One block per split half tile; one warp per row, lanes across head_dim.  Partials are merged in increasing split
// order with weights exp2(lse_s - max lse), so the result does not depend on scheduling.
__global__ void __launch_bounds__(256) wpp_combine_kernel(const CombineParams p) {
    const char* plan = static_cast<const char*>(p.plan);
    const WppPlanHeader* hd = reinterpret_cast<const WppPlanHeader*>(plan);
    const int32_t* q_offsets = reinterpret_cast<const int32_t*>(plan + hd->off_q_offsets);
    const WppCombine cu = reinterpret_cast<const WppCombine*>(plan + hd->off_combine)[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = p.head_dim;
    for (int r = warp; r < cu.rows; r += 8) {
        float m = -INFINITY;
        for (int s = 0; s < cu.num_splits; ++s)
            m = fmaxf(m, p.ws_lse[((int64_t)(cu.slot0 + s) * 2 + cu.half) * 128 + cu.lane0 + r]);
        const int64_t tok = (int64_t)q_offsets[cu.request] + cu.row0 + r;
        __nv_bfloat16* dst = p.out + tok * p.o_token_stride + (int64_t)cu.head * p.o_head_stride;
        float wsum = 0.f;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        if (m > -INFINITY) {
            for (int s = 0; s < cu.num_splits; ++s) {
                const int64_t row = ((int64_t)(cu.slot0 + s) * 2 + cu.half) * 128 + cu.lane0 + r;
                const float l = p.ws_lse[row];
                if (l == -INFINITY) continue;       // that part saw no key of this row; its O row is not defined
                const float w = exp2f(l - m);
                wsum += w;
                for (int e = lane, k = 0; e < D; e += 32, ++k) acc[k] += w * p.ws_o[row * D + e];
            }
        }
        const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
        for (int e = lane, k = 0; e < D; e += 32, ++k) dst[e] = __float2bfloat16_rn(acc[k] * inv);
        if (p.lse && lane == 0)
            p.lse[tok * p.num_q_heads + cu.head] =
                wsum > 0.f ? (m + log2f(wsum)) * 0.6931471805599453f : -INFINITY;
    }
}

// Self-test of the bounded wait every kernel of the library relies on: one warp waits, with a short limit, on
// a barrier that nothing ever arrives on.  The wait must give up, raise the abort flag and let the kernel end
// normally with WPP_ERR_TIMEOUT in the status word - it never hangs and never traps.
__global__ void wpp_selftest_wait_kernel(long long limit_cycles, int32_t* status, long long* waited_cycles) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0u;
        fence_barrier_init();
    }
    __syncthreads();
    const long long t0 = clock64();
    const bool ok = mbar_wait_limit(b, 0, &abort_flag, limit_cycles);
    const long long t1 = clock64();
    if (!__all_sync(0xffffffffu, ok) && threadIdx.x == 0) {
        if (status) atomicCAS(status, 0, WPP_ERR_TIMEOUT);
        if (waited_cycles) *waited_cycles = t1 - t0;
    }
}

}  // namespace wpp

extern "C" int wpp_launch_selftest_wait(long long limit_cycles, int32_t* status, long long* waited_cycles,
                                        void* stream) {
    wpp::wpp_selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_cycles, status, waited_cycles);
    return (int)cudaGetLastError();
}

extern "C" int wpp_launch_append(const wpp::AppendParams* p, int num_sms, void* stream) {
    const int64_t total = p->total_new_tokens * p->num_kv_heads * p->vec_per_row;
    if (total == 0) return 0;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)num_sms * 16;
    if (blocks > cap) blocks = cap;
    wpp::wpp_append_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(*p);
    return (int)cudaGetLastError();
}

extern "C" int wpp_launch_combine(const wpp::CombineParams* p, int num_combine, void* stream) {
    if (num_combine == 0) return 0;
    wpp::wpp_combine_kernel<<<(unsigned)num_combine, 256, 0, (cudaStream_t)stream>>>(*p);
    return (int)cudaGetLastError();
}
