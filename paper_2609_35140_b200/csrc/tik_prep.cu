// Pre-attention step in one pass over the new tokens: per-head RMSNorm of Q and K, NeoX rotary
// embedding of Q and K, and the indexed write of K and V into the paged cache.  The paper's
// operator table lists these as separate unified operators next to attention; fusing them and
// the order norm -> rotation -> write (the Qwen3 layer order) are this library's choices.
//
// The step is bound by HBM traffic (every byte is touched once), so the kernel is plain
// coalesced loads and stores: one CTA per token, one warp per (token, head) vector, the lane
// holding element i also holds its rotation partner i + d/2.  Each (token, head) is computed by
// one warp from that vector alone, with a fixed reduction order, so its bits do not depend on
// how many tokens or sequences the call covers: the full-sequence call of the policy update and
// the token-wise calls of the rollout produce identical Q, K and cache contents.
#include <cuda_bf16.h>

#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

constexpr int PREP_WARPS = 8;
constexpr int PREP_BATCH = 4;      // vectors a warp keeps in flight

template <int D>
struct PrepVec {                   // the elements of one vector held by one lane
    static constexpr int EP = D / 64;      // per half: 2 for d = 128 (a bf16 pair), 1 for d = 64
    float lo[EP], hi[EP];
};

template <int D>
__device__ __forceinline__ void prep_load(const __nv_bfloat16* src, int lane, uint32_t& lo, uint32_t& hi) {
    if (D == 128) {
        lo = reinterpret_cast<const uint32_t*>(src)[lane];
        hi = reinterpret_cast<const uint32_t*>(src)[32 + lane];
    } else {
        lo = reinterpret_cast<const uint16_t*>(src)[lane];
        hi = reinterpret_cast<const uint16_t*>(src)[32 + lane];
    }
}
template <int D>
__device__ __forceinline__ void prep_store(__nv_bfloat16* dst, int lane, uint32_t lo, uint32_t hi) {
    if (D == 128) {
        reinterpret_cast<uint32_t*>(dst)[lane] = lo;
        reinterpret_cast<uint32_t*>(dst)[32 + lane] = hi;
    } else {
        reinterpret_cast<uint16_t*>(dst)[lane] = static_cast<uint16_t>(lo);
        reinterpret_cast<uint16_t*>(dst)[32 + lane] = static_cast<uint16_t>(hi);
    }
}
template <int D>
__device__ __forceinline__ void prep_unpack(uint32_t raw, float* x) {
    x[0] = __uint_as_float(raw << 16);                      // bf16 -> fp32 is exact
    if (D == 128) x[1] = __uint_as_float(raw & 0xffff0000u);
}
template <int D>
__device__ __forceinline__ uint32_t prep_pack(const float* x) {
    if (D == 128) return pack_bf16x2(x[0], x[1]);
    return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(x[0])));
}

template <int D>
__global__ void __launch_bounds__(PREP_WARPS * 32) prep_kernel(const PrepParams p) {
    constexpr int EP = D / 64;
    const int token = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int lo_s = 0, hi_s = p.S;      // sequence s with cu_new[s] <= token < cu_new[s+1]
    while (hi_s - lo_s > 1) {
        const int mid = (lo_s + hi_s) >> 1;
        if (p.cu_new[mid] <= token) lo_s = mid; else hi_s = mid;
    }
    const int s = lo_s;
    const int first = p.cu_new[s];
    if (token >= p.cu_new[s + 1]) return;
    const int n_s = p.cu_new[s + 1] - first;
    const int pos = (p.ctx_lens ? p.ctx_lens[s] - n_s : 0) + (token - first);
    if (pos < 0 || pos >= p.max_pos) {          // no table row: the token is left untouched
        if (threadIdx.x == 0) atomicOr(p.dev_status, TIK_DEV_BAD_POSITION);
        return;
    }
    bool to_cache = p.k_cache != nullptr;
    long long cache_row = 0;                    // (page, kv head 0, slot) in units of rows of D
    if (to_cache) {
        const int lp = pos / p.page_size;
        const int phys = (lp < p.max_blocks) ? p.block_table[static_cast<long long>(s) * p.max_blocks + lp] : -1;
        if (phys < 0 || phys >= p.num_pages) {
            if (threadIdx.x == 0) atomicOr(p.dev_status, TIK_DEV_BAD_BLOCK);
            to_cache = false;
        } else {
            cache_row = static_cast<long long>(phys) * p.Hkv * p.page_size + pos % p.page_size;
        }
    }
    // this lane's rotation coefficients and norm weights
    float cs[EP], sn[EP], wq_lo[EP], wq_hi[EP], wk_lo[EP], wk_hi[EP];
    {
        const float* row = p.cos_sin + static_cast<long long>(pos) * D;
#pragma unroll
        for (int e = 0; e < EP; ++e) {
            cs[e] = row[EP * lane + e];
            sn[e] = row[D / 2 + EP * lane + e];
        }
        uint32_t a = 0, b = 0;
        if (p.q_weight) {
            prep_load<D>(p.q_weight, lane, a, b);
            prep_unpack<D>(a, wq_lo);
            prep_unpack<D>(b, wq_hi);
        }
        if (p.k_weight) {
            prep_load<D>(p.k_weight, lane, a, b);
            prep_unpack<D>(a, wk_lo);
            prep_unpack<D>(b, wk_hi);
        }
    }
    const int nh = p.Hq + p.Hkv;
    for (int h0 = warp; h0 < nh; h0 += PREP_WARPS * PREP_BATCH) {
        uint32_t raw_lo[PREP_BATCH], raw_hi[PREP_BATCH];
#pragma unroll
        for (int b = 0; b < PREP_BATCH; ++b) {              // all loads first: memory-level parallelism
            const int h = h0 + b * PREP_WARPS;
            if (h < nh) {
                const __nv_bfloat16* src = (h < p.Hq)
                    ? p.q + (static_cast<long long>(token) * p.Hq + h) * D
                    : p.k + (static_cast<long long>(token) * p.Hkv + (h - p.Hq)) * D;
                prep_load<D>(src, lane, raw_lo[b], raw_hi[b]);
            }
        }
#pragma unroll
        for (int b = 0; b < PREP_BATCH; ++b) {
            const int h = h0 + b * PREP_WARPS;
            if (h >= nh) break;
            const bool is_q = h < p.Hq;
            float lo[EP], hi[EP];
            prep_unpack<D>(raw_lo[b], lo);
            prep_unpack<D>(raw_hi[b], hi);
            const __nv_bfloat16* w = is_q ? p.q_weight : p.k_weight;
            if (w) {
                const float ss = prep_sum_squares<EP>(lo, hi);
                const float inv = prep_inv_rms(ss, 1.0f / D, p.eps);
#pragma unroll
                for (int e = 0; e < EP; ++e) {
                    lo[e] = prep_norm(lo[e], inv, is_q ? wq_lo[e] : wk_lo[e]);
                    hi[e] = prep_norm(hi[e], inv, is_q ? wq_hi[e] : wk_hi[e]);
                }
            }
#pragma unroll
            for (int e = 0; e < EP; ++e) prep_rotate(lo[e], hi[e], cs[e], sn[e]);
            const uint32_t out_lo = prep_pack<D>(lo), out_hi = prep_pack<D>(hi);
            if (is_q) {
                prep_store<D>(p.q + (static_cast<long long>(token) * p.Hq + h) * D, lane, out_lo, out_hi);
            } else {
                const int hh = h - p.Hq;
                prep_store<D>(p.k + (static_cast<long long>(token) * p.Hkv + hh) * D, lane, out_lo, out_hi);
                if (to_cache)
                    prep_store<D>(p.k_cache + (cache_row + static_cast<long long>(hh) * p.page_size) * D, lane,
                                  out_lo, out_hi);
            }
        }
    }
    if (to_cache && p.v) {       // V rows go to the cache unchanged, 16 bytes per thread
        constexpr int VPH = D * 2 / 16;
        const uint4* src = reinterpret_cast<const uint4*>(p.v + static_cast<long long>(token) * p.Hkv * D);
        for (int i = threadIdx.x; i < p.Hkv * VPH; i += blockDim.x) {
            const int hh = i / VPH, e = i % VPH;
            reinterpret_cast<uint4*>(p.v_cache + (cache_row + static_cast<long long>(hh) * p.page_size) * D)[e] = src[i];
        }
    }
}

cudaError_t launch_prep(int d, const PrepParams& p, int64_t total_new, cudaStream_t stream) {
    if (total_new <= 0) return cudaSuccess;
    if (d == 128) prep_kernel<128><<<static_cast<unsigned>(total_new), PREP_WARPS * 32, 0, stream>>>(p);
    else prep_kernel<64><<<static_cast<unsigned>(total_new), PREP_WARPS * 32, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace tik
