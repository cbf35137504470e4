// Hidden RMSNorm, fused residual + RMSNorm and SwiGLU: the element-wise operators around the
// attention and FFN blocks that the paper's operator table lists as unified operators.  All
// three touch every byte once and are bound by HBM traffic: 16-byte coalesced accesses, the
// whole row of a norm requested before anything is computed, and small CTAs so that enough of
// them are resident to keep the memory system busy.  A row's result depends on that row, the
// weight and eps only (fixed 128-thread reduction shape), never on the number of rows.
#include <cuda_bf16.h>

#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

constexpr int HN_THREADS = 128;

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    const uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(r[i] << 16);              // bf16 -> fp32 is exact
        f[2 * i + 1] = __uint_as_float(r[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
    return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                      pack_bf16x2(f[6], f[7]));
}

// One CTA per row; NV = 16-byte vectors per thread (H <= 1024 * NV).
template <int NV, bool RESIDUAL>
__global__ void __launch_bounds__(HN_THREADS) rmsnorm_kernel(const NormParams p) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long row = blockIdx.x;
    const int nvec = p.H / 8;
    const uint4* x = reinterpret_cast<const uint4*>(p.x) + row * nvec;
    uint4* res = RESIDUAL ? reinterpret_cast<uint4*>(p.residual) + row * nvec : nullptr;
    const uint4* w = reinterpret_cast<const uint4*>(p.weight);
    uint4* y = reinterpret_cast<uint4*>(p.y) + row * nvec;
    __shared__ float warp_tot[4];

    uint4 xv[NV], rv[RESIDUAL ? NV : 1];
#pragma unroll
    for (int j = 0; j < NV; ++j) {                           // the whole row is requested first
        const int v = tid + HN_THREADS * j;
        if (v < nvec) {
            xv[j] = x[v];
            if (RESIDUAL) rv[j] = res[v];
        }
    }
    float s[NV][8];
    float part = 0.0f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const int v = tid + HN_THREADS * j;
        if (v < nvec) {
            unpack8(xv[j], s[j]);
            if (RESIDUAL) {
                float r[8];
                unpack8(rv[j], r);
#pragma unroll
                for (int e = 0; e < 8; ++e) s[j][e] = hn_residual_sum(s[j][e], r[e]);
                res[v] = pack8(s[j]);                        // exact: the sums are bf16 values
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) part = __fmaf_rn(s[j][e], s[j][e], part);
        }
    }
    part = hn_warp_total(part);
    if (lane == 0) warp_tot[warp] = part;
    __syncthreads();
    const float inv = prep_inv_rms(hn_block_total(warp_tot), 1.0f / static_cast<float>(p.H), p.eps);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const int v = tid + HN_THREADS * j;
        if (v < nvec) {
            float wf[8], o[8];
            unpack8(w[v], wf);
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = prep_norm(s[j][e], inv, wf[e]);
            y[v] = pack8(o);
        }
    }
}

// out[t][i] = silu(gu[t][i]) * gu[t][I + i]; 16-byte vectors of 8 outputs, SW_VPT per thread (a block
// covers 256 * SW_VPT consecutive vectors).  Large calls take four: all eight loads of a thread are
// issued before the arithmetic, 128 bytes per thread in flight (6.3 -> 6.9 TB/s on 32 768 x 27 648);
// small calls (decode) take one, which spreads them over more blocks.
template <int SW_VPT>
__global__ void __launch_bounds__(256) swiglu_kernel(const __nv_bfloat16* __restrict__ gu,
                                                    __nv_bfloat16* __restrict__ out, long long T, int I) {
    const int vpr = I / 8;                                   // output vectors per row
    const long long nvec = T * vpr;
    const long long base = static_cast<long long>(blockIdx.x) * (256 * SW_VPT) + threadIdx.x;
    uint4 gv[SW_VPT], uv[SW_VPT];
#pragma unroll
    for (int j = 0; j < SW_VPT; ++j) {
        const long long idx = base + 256 * j;
        if (idx < nvec) {
            const long long t = idx / vpr;
            const int c = static_cast<int>(idx - t * vpr);
            const uint4* row = reinterpret_cast<const uint4*>(gu) + t * 2 * vpr;
            gv[j] = row[c];
            uv[j] = row[vpr + c];
        }
    }
#pragma unroll
    for (int j = 0; j < SW_VPT; ++j) {
        const long long idx = base + 256 * j;
        if (idx < nvec) {
            float g[8], u[8], o[8];
            unpack8(gv[j], g);
            unpack8(uv[j], u);
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = swiglu_value(g[e], u[e]);
            reinterpret_cast<uint4*>(out)[idx] = pack8(o);
        }
    }
}

template <bool RESIDUAL>
static cudaError_t launch_rmsnorm_t(const NormParams& p, cudaStream_t stream) {
    const unsigned grid = static_cast<unsigned>(p.T);
    const int nv = (p.H / 8 + HN_THREADS - 1) / HN_THREADS;
    count_launch();  // exactly one of the launches below runs
    if (nv <= 1) rmsnorm_kernel<1, RESIDUAL><<<grid, HN_THREADS, 0, stream>>>(p);
    else if (nv <= 2) rmsnorm_kernel<2, RESIDUAL><<<grid, HN_THREADS, 0, stream>>>(p);
    else if (nv <= 4) rmsnorm_kernel<4, RESIDUAL><<<grid, HN_THREADS, 0, stream>>>(p);
    else rmsnorm_kernel<8, RESIDUAL><<<grid, HN_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_rmsnorm(const NormParams& p, cudaStream_t stream) {
    if (p.T <= 0) return cudaSuccess;
    return p.residual ? launch_rmsnorm_t<true>(p, stream) : launch_rmsnorm_t<false>(p, stream);
}

cudaError_t launch_swiglu(const void* gu, void* out, long long T, int I, cudaStream_t stream) {
    if (T <= 0) return cudaSuccess;
    const long long n = T * (I / 8);
    count_launch();  // exactly one of the launches below runs
    if (n >= (1ll << 20))
        swiglu_kernel<4><<<static_cast<unsigned>((n + 1023) / 1024), 256, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(gu), static_cast<__nv_bfloat16*>(out), T, I);
    else
        swiglu_kernel<1><<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(gu), static_cast<__nv_bfloat16*>(out), T, I);
    return cudaGetLastError();
}

}  // namespace tik
