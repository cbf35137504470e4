// Pre-attention step in one pass over the new tokens: per-head RMSNorm of Q and K, NeoX rotary
// embedding of Q and K, and the indexed write of K and V into the paged cache.  The paper's
// operator table lists these as separate unified operators next to attention; fusing them and
// the order norm -> rotation -> write (the Qwen3 layer order) are this library's choices.
//
// The step is bound by HBM traffic (every byte is touched once), so the kernel is plain
// coalesced vector loads and stores: one warp per token, sixteen lanes per (token, head) vector,
// the lane holding element i also holds its rotation partner i + d/2.  Each (token, head) is
// computed by its sixteen lanes from that vector alone, with a fixed reduction order, so its bits do not depend on
// how many tokens or sequences the call covers: the full-sequence call of the policy update and
// the token-wise calls of the rollout produce identical Q, K and cache contents.
#include <cuda_bf16.h>

#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

constexpr int PREP_WARPS = 4;
constexpr int PREP_BATCH = 4;      // vector pairs (8 heads) a warp requests at a time
constexpr int PREP_MIN_CTAS = 7;   // 28 warps per SM: the step is bound by bytes in flight, not by arithmetic

// Sixteen lanes hold one vector: lane l has EP = d/32 consecutive elements of the first half
// (EP*l ..) and their rotation partners (d/2 + EP*l ..); a warp works on two vectors at once.
template <int D>
__device__ __forceinline__ void prep_load(const __nv_bfloat16* src, int l16, uint32_t* lo, uint32_t* hi) {
    if (D == 128) {
        const uint2 a = reinterpret_cast<const uint2*>(src)[l16];
        const uint2 b = reinterpret_cast<const uint2*>(src)[16 + l16];
        lo[0] = a.x, lo[1] = a.y, hi[0] = b.x, hi[1] = b.y;
    } else {
        lo[0] = reinterpret_cast<const uint32_t*>(src)[l16];
        hi[0] = reinterpret_cast<const uint32_t*>(src)[16 + l16];
    }
}
template <int D>
__device__ __forceinline__ void prep_store(__nv_bfloat16* dst, int l16, const uint32_t* lo, const uint32_t* hi) {
    if (D == 128) {
        reinterpret_cast<uint2*>(dst)[l16] = make_uint2(lo[0], lo[1]);
        reinterpret_cast<uint2*>(dst)[16 + l16] = make_uint2(hi[0], hi[1]);
    } else {
        reinterpret_cast<uint32_t*>(dst)[l16] = lo[0];
        reinterpret_cast<uint32_t*>(dst)[16 + l16] = hi[0];
    }
}
template <int EP>
__device__ __forceinline__ void prep_unpack(const uint32_t* raw, float* x) {
#pragma unroll
    for (int e = 0; e < EP / 2; ++e) {
        x[2 * e] = __uint_as_float(raw[e] << 16);            // bf16 -> fp32 is exact
        x[2 * e + 1] = __uint_as_float(raw[e] & 0xffff0000u);
    }
}

template <int D>
__global__ void __launch_bounds__(PREP_WARPS * 32, PREP_MIN_CTAS) prep_kernel(const PrepParams p) {
    constexpr int EP = D / 32;
    constexpr int VPH = D * 2 / 16;             // 16-byte pieces of one V row
    pdl_launch_dependents();       // an attention kernel launched next may be scheduled behind this grid
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 4, l16 = lane & 15;
    const long long token = static_cast<long long>(blockIdx.x) * PREP_WARPS + warp;   // one warp per token
    if (token >= p.total_new) return;
    const int nh = p.Hq + p.Hkv;
    __nv_bfloat16* const q_tok = p.q + token * p.Hq * D;
    __nv_bfloat16* const k_tok = p.k + token * p.Hkv * D;

    // The vectors of a token are requested before anything else is known about it: the loads
    // depend on the token index only, and the look-ups below (sequence, position, page, table
    // row) then run while they are in flight.
    uint32_t raw_lo[PREP_BATCH][EP / 2], raw_hi[PREP_BATCH][EP / 2];
    auto load_batch = [&](int pi0) {
#pragma unroll
        for (int b = 0; b < PREP_BATCH; ++b) {
            const int h = 2 * (pi0 + b) + sub;
#pragma unroll
            for (int e = 0; e < EP / 2; ++e) raw_lo[b][e] = raw_hi[b][e] = 0;
            if (h < nh) prep_load<D>(h < p.Hq ? q_tok + h * D : k_tok + (h - p.Hq) * D, l16, raw_lo[b], raw_hi[b]);
        }
    };
    load_batch(0);

    int lo_s = 0, hi_s = p.S;      // sequence s with cu_new[s] <= token < cu_new[s+1]
    while (hi_s - lo_s > 1) {
        const int mid = (lo_s + hi_s) >> 1;
        if (p.cu_new[mid] <= token) lo_s = mid; else hi_s = mid;
    }
    const int s = lo_s;
    const int first = p.cu_new[s];
    if (token >= p.cu_new[s + 1]) return;
    const int n_s = p.cu_new[s + 1] - first;
    const int pos = (p.ctx_lens ? p.ctx_lens[s] - n_s : 0) + static_cast<int>(token - first);
    if (pos < 0 || pos >= p.max_pos) {          // no table row: the token is left untouched
        if (lane == 0) atomicOr(p.dev_status, TIK_DEV_BAD_POSITION);
        return;
    }
    bool to_cache = p.k_cache != nullptr;
    long long cache_row = 0;                    // (page, kv head 0, slot) in units of rows of D
    if (to_cache) {
        const int lp = pos / p.page_size;
        const int phys = (lp < p.max_blocks) ? p.block_table[static_cast<long long>(s) * p.max_blocks + lp] : -1;
        if (phys < 0 || phys >= p.num_pages) {
            if (lane == 0) atomicOr(p.dev_status, TIK_DEV_BAD_BLOCK);
            to_cache = false;
        } else {
            cache_row = static_cast<long long>(phys) * p.Hkv * p.page_size + pos % p.page_size;
        }
    }
    // this lane's rotation coefficients and norm weights
    // (the weights stay packed as loaded and are widened where used: registers buy occupancy here)
    float cs[EP], sn[EP];
    uint32_t wq_lo[EP / 2] = {}, wq_hi[EP / 2] = {}, wk_lo[EP / 2] = {}, wk_hi[EP / 2] = {};
    {
        const float* row = p.cos_sin + static_cast<long long>(pos) * D;
#pragma unroll
        for (int e = 0; e < EP; ++e) {
            cs[e] = row[EP * l16 + e];
            sn[e] = row[D / 2 + EP * l16 + e];
        }
        if (p.q_weight) prep_load<D>(p.q_weight, l16, wq_lo, wq_hi);
        if (p.k_weight) prep_load<D>(p.k_weight, l16, wk_lo, wk_hi);
    }
    if (to_cache) {       // V rows go to the cache unchanged, 16 bytes per lane and step
        const uint4* src = reinterpret_cast<const uint4*>(p.v + token * p.Hkv * D);
        const int nv = p.Hkv * VPH;
        for (int i0 = 0; i0 < nv; i0 += 4 * 32) {
            uint4 val[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (i0 + 32 * j + lane < nv) val[j] = src[i0 + 32 * j + lane];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = i0 + 32 * j + lane;
                if (i < nv)
                    reinterpret_cast<uint4*>(p.v_cache + (cache_row + static_cast<long long>(i / VPH) * p.page_size) * D)[i % VPH] = val[j];
            }
        }
    }
    for (int pi0 = 0; 2 * pi0 < nh; pi0 += PREP_BATCH) {
        if (pi0 > 0) load_batch(pi0);
#pragma unroll
        for (int b = 0; b < PREP_BATCH; ++b) {
            if (2 * (pi0 + b) >= nh) break;                  // warp-uniform
            const int h = 2 * (pi0 + b) + sub;
            const bool is_q = h < p.Hq;
            float lo[EP], hi[EP];
            prep_unpack<EP>(raw_lo[b], lo);
            prep_unpack<EP>(raw_hi[b], hi);
            const __nv_bfloat16* w = is_q ? p.q_weight : p.k_weight;
            // both halves of the warp take part in the exchange; a half without a norm ignores it
            const float ss = prep_sum_squares<EP>(lo, hi);
            if (w) {
                const float inv = prep_inv_rms(ss, 1.0f / D, p.eps);
                float w_lo[EP], w_hi[EP];
                prep_unpack<EP>(is_q ? wq_lo : wk_lo, w_lo);
                prep_unpack<EP>(is_q ? wq_hi : wk_hi, w_hi);
#pragma unroll
                for (int e = 0; e < EP; ++e) {
                    lo[e] = prep_norm(lo[e], inv, w_lo[e]);
                    hi[e] = prep_norm(hi[e], inv, w_hi[e]);
                }
            }
#pragma unroll
            for (int e = 0; e < EP; ++e) prep_rotate(lo[e], hi[e], cs[e], sn[e]);
            uint32_t out_lo[EP / 2], out_hi[EP / 2];
#pragma unroll
            for (int e = 0; e < EP / 2; ++e) {
                out_lo[e] = pack_bf16x2(lo[2 * e], lo[2 * e + 1]);
                out_hi[e] = pack_bf16x2(hi[2 * e], hi[2 * e + 1]);
            }
            if (h >= nh) continue;
            if (is_q) {
                prep_store<D>(q_tok + h * D, l16, out_lo, out_hi);
            } else {
                const int hh = h - p.Hq;
                prep_store<D>(k_tok + hh * D, l16, out_lo, out_hi);
                if (to_cache)
                    prep_store<D>(p.k_cache + (cache_row + static_cast<long long>(hh) * p.page_size) * D, l16,
                                  out_lo, out_hi);
            }
        }
    }
}

cudaError_t launch_prep(int d, const PrepParams& p, int64_t total_new, cudaStream_t stream) {
    if (total_new <= 0) return cudaSuccess;
    const unsigned grid = static_cast<unsigned>((total_new + PREP_WARPS - 1) / PREP_WARPS);
    count_launch();  // exactly one of the launches below runs
    if (d == 128) prep_kernel<128><<<grid, PREP_WARPS * 32, 0, stream>>>(p);
    else prep_kernel<64><<<grid, PREP_WARPS * 32, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace tik
