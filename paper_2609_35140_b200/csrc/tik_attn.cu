// Unified causal GQA attention for sm_100a: one kernel body for the packed train-forward,
// the paged prefill and the paged decode regime, plus the split-KV combine and the
// KV-cache write.
//
// One CTA owns one MMA tile of 128 query rows and walks 128-key KV tiles in ascending
// order.  S = Q K^T and O += P V run on tcgen05 (M128 x N128 x K16 and M128 x Nd x K16,
// fp32 accumulators in TMEM); Q, K, V arrive by TMA into 128B-swizzled shared memory
// (K/V of the paged regimes are gathered page by page through the block table); the
// online softmax is one thread per row, straight out of TMEM, with the arithmetic of
// tik_core.cuh.  What differs between regimes is only where rows come from and where they
// go:
//   train   : rows = 128 consecutive tokens of one (sequence, query head); K/V packed
//   prefill : same rows, aligned to absolute positions; K/V from pages
//   decode  : rows 0..G-1 = the G query heads of one KV head for one sequence (other rows
//             zero); K/V from pages; one CTA per 2048-key chunk, partial (m, l, O) to scratch
// Query tiles are aligned to absolute positions (multiples of 128) in every regime, so a
// row never meets a tile or chunk in which all of its keys are masked.
#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

enum { MODE_TRAIN = 0, MODE_PREFILL = 1, MODE_DECODE = 2 };

template <int D>
struct AttnSmem {
    static constexpr uint32_t ATOM = 128 * 128;          // 128 rows x 64 bf16
    static constexpr uint32_t TILE = (D / 64) * ATOM;    // one Q, K or V tile
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = TILE;              // two stages
    static constexpr uint32_t OFF_V = 3 * TILE;          // two stages
    static constexpr uint32_t OFF_P = 5 * TILE;          // 128 rows x 128 keys bf16
    static constexpr uint32_t OFF_BAR = OFF_P + 2 * ATOM;
    static constexpr uint32_t BYTES = OFF_BAR + 128;
    static constexpr uint32_t ALLOC = BYTES + 1024;      // slack for 1 KiB alignment
};

template <int D, int MODE>
__global__ void __launch_bounds__(128, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    using L = AttnSmem<D>;
    constexpr int NATOM = D / 64;
    constexpr uint32_t TMEM_COLS = (D == 128) ? 512u : 256u;
    constexpr uint32_t COL_S = 0, COL_OA = 128, COL_OB = 128 + D;
    constexpr uint32_t IDESC_QK = mma_idesc_bf16(128, 128, false);
    constexpr uint32_t IDESC_PV = mma_idesc_bf16(128, D, true);

    const int tid = threadIdx.x, warp = tid >> 5;

    // ---------------------------------------------------------------- work item
    int seq, head, kvh, T = 0, chunk = 0, ctx = 0, pos0 = 0;
    long long qrow0 = 0;       // token row of tile row 0 (train/prefill), may be negative
    long long tok0 = 0;        // first token of the sequence in the packed K/V (train)
    int row_lo = 0, row_hi = 0;   // valid tile rows [row_lo, row_hi)
    int tile_first, tile_last;
    if (MODE == MODE_TRAIN) {
        seq = blockIdx.z;
        head = blockIdx.y;
        kvh = head / p.G;
        T = gridDim.x - 1 - blockIdx.x;
        tok0 = p.cu_seqlens[seq];
        const int len = p.cu_seqlens[seq + 1] - static_cast<int>(tok0);
        if (128 * T >= len) return;
        ctx = len;
        qrow0 = tok0 + 128ll * T;
        row_lo = 0;
        row_hi = min(128, len - 128 * T);
        tile_first = 0;
        tile_last = T;
    } else if (MODE == MODE_PREFILL) {
        seq = blockIdx.z;
        head = blockIdx.y;
        kvh = head / p.G;
        const int qb = p.cu_seqlens[seq];
        const int qlen = p.cu_seqlens[seq + 1] - qb;
        ctx = p.ctx_lens[seq];
        pos0 = ctx - qlen;
        if (qlen <= 0 || pos0 < 0) return;
        T = pos0 / 128 + (gridDim.x - 1 - blockIdx.x);
        if (128 * T >= ctx) return;
        qrow0 = static_cast<long long>(qb) + 128ll * T - pos0;
        row_lo = max(0, pos0 - 128 * T);
        row_hi = min(128, ctx - 128 * T);
        tile_first = 0;
        tile_last = T;
    } else {
        seq = blockIdx.z;
        kvh = blockIdx.y;
        head = kvh * p.G;
        chunk = blockIdx.x;
        ctx = p.ctx_lens[seq];
        if (ctx <= 0 || chunk * CHUNK >= ctx) return;
        tile_first = chunk * TILES_PER_CHUNK;
        tile_last = min(tile_first + TILES_PER_CHUNK - 1, (ctx - 1) / 128);
        row_lo = 0;
        row_hi = p.G;
    }
    const int n_tiles = tile_last - tile_first + 1;

    // ---------------------------------------------------------------- shared memory
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw_addr + pad;
    const uint32_t sQ = sbase + L::OFF_Q, sK = sbase + L::OFF_K, sV = sbase + L::OFF_V,
                   sP = sbase + L::OFF_P;
    const uint32_t bar_q = sbase + L::OFF_BAR, bar_kv0 = bar_q + 8, bar_s = bar_q + 24,
                   bar_o = bar_q + 32;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_BAR + 40);
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 44);

    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv0, 1);
        mbar_init(bar_kv0 + 8, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    }
    if (MODE == MODE_DECODE) {
        // rows >= G of the Q tile are never loaded: make them zero; P rows of idle warps too
        uint4 z = make_uint4(0, 0, 0, 0);
        for (uint32_t i = tid; i < L::TILE / 16; i += 128)
            reinterpret_cast<uint4*>(smem + L::OFF_Q)[i] = z;
        for (uint32_t i = tid; i < 2 * L::ATOM / 16; i += 128)
            reinterpret_cast<uint4*>(smem + L::OFF_P)[i] = z;
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tlane = tmem + (static_cast<uint32_t>(warp * 32) << 16);

    // ---------------------------------------------------------------- loaders (thread 0)
    auto load_q = [&]() {
        if (MODE == MODE_DECODE) {
            mbar_expect_tx(bar_q, static_cast<uint32_t>(p.G) * 128u * NATOM);
            for (int a = 0; a < NATOM; ++a)
                tma_load_3d(sQ + a * L::ATOM, &tmQ, bar_q, a * 64, head, seq);
        } else {
            mbar_expect_tx(bar_q, L::TILE);
            for (int a = 0; a < NATOM; ++a)
                tma_load_3d(sQ + a * L::ATOM, &tmQ, bar_q, a * 64, head, static_cast<int>(qrow0));
        }
    };
    auto load_kv = [&](int j, int st) {
        const uint32_t bar = bar_kv0 + 8 * st;
        const uint32_t dK = sK + st * L::TILE, dV = sV + st * L::TILE;
        mbar_expect_tx(bar, 2 * L::TILE);
        if (MODE == MODE_TRAIN) {
            const int row = static_cast<int>(tok0) + 128 * j;
            for (int a = 0; a < NATOM; ++a) {
                tma_load_3d(dK + a * L::ATOM, &tmK, bar, a * 64, kvh, row);
                tma_load_3d(dV + a * L::ATOM, &tmV, bar, a * 64, kvh, row);
            }
        } else {
            const int lp0 = (128 * j) / p.page_size;
            for (int i = 0; i < p.pages_per_tile; ++i) {
                const int lp = lp0 + i;
                int phys = p.num_pages;   // out of range: the box is filled with zeros
                if (lp * p.page_size < ctx) {
                    if (lp < p.max_blocks) phys = p.block_table[static_cast<long long>(seq) * p.max_blocks + lp];
                    else phys = -1;
                    if (phys < 0 || phys >= p.num_pages) {
                        atomicOr(p.dev_status, TIK_DEV_BAD_BLOCK);
                        phys = p.num_pages;
                    }
                }
                const uint32_t off = static_cast<uint32_t>(i * p.page_size) * 128u;
                for (int a = 0; a < NATOM; ++a) {
                    tma_load_4d(dK + a * L::ATOM + off, &tmK, bar, a * 64, 0, kvh, phys);
                    tma_load_4d(dV + a * L::ATOM + off, &tmV, bar, a * 64, 0, kvh, phys);
                }
            }
        }
    };

    if (tid == 0) {
        load_q();
        load_kv(tile_first, 0);
    }

    // ---------------------------------------------------------------- per-row state
    const int r = tid;                                      // tile row == TMEM lane
    const int qpos = (MODE == MODE_DECODE) ? (ctx - 1) : (128 * T + r);
    const bool softmax_active = (MODE != MODE_DECODE) || (warp == 0);
    const float c = p.c;
    float m_run = -CUDART_INF_F, l_run = 0.0f;              // state of the current chunk
    float M_g = -CUDART_INF_F, L_g = 0.0f;                  // folded state of earlier chunks
    uint32_t par_s = 0, par_o = 0, par_kv[2] = {0, 0};
    uint32_t col_o = COL_OA;                                // chunk 0 accumulates in place

    for (int it = 0; it < n_tiles; ++it) {
        const int j = tile_first + it;
        const int st = it & 1;
        const bool chunk_start = (j % TILES_PER_CHUNK) == 0;
        const bool chunk_end = ((j % TILES_PER_CHUNK) == TILES_PER_CHUNK - 1) || (it == n_tiles - 1);
        const int chunk_idx = j / TILES_PER_CHUNK;
        if (MODE != MODE_DECODE && chunk_start) col_o = (chunk_idx == 0) ? COL_OA : COL_OB;

        if (tid == 0) {
            if (it + 1 < n_tiles) load_kv(j + 1, st ^ 1);
            if (it == 0) mbar_wait(bar_q, 0, abort_word, p.dev_status);
            mbar_wait(bar_kv0 + 8 * st, par_kv[st], abort_word, p.dev_status);
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint32_t koff = (ks >> 2) * L::ATOM + (ks & 3) * 32;
                mma_ss(tmem + COL_S, smem_desc_sw128(sQ + koff, 0, 1024),
                       smem_desc_sw128(sK + st * L::TILE + koff, 0, 1024), IDESC_QK, ks > 0);
            }
            mma_commit(bar_s);
        }
        par_kv[st] ^= 1;
        mbar_wait(bar_s, par_s, abort_word, p.dev_status);
        par_s ^= 1;
        tc_fence_after();

        if (softmax_active) {
            const int kmax = qpos - 128 * j;      // columns > kmax are masked
            // pass 1: tile maximum
            float mt = -CUDART_INF_F;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t v[32];
                tmem_ld32(tlane + COL_S + 32 * cc, v);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float s = __uint_as_float(v[i]);
                    if (32 * cc + i > kmax) s = -CUDART_INF_F;
                    mt = fmaxf(mt, s);
                }
            }
            const float m_new = fmaxf(m_run, mt);
            const float neg_mc = -__fmul_rn(m_new, c);
            const float alpha = softmax_alpha(m_run, m_new, c);
            // pass 2: p, row sum, bf16 P into swizzled shared memory
            RowSum8 rs;
            rs.reset();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t v[32];
                tmem_ld32(tlane + COL_S + 32 * cc, v);
                tmem_wait_ld();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float p0 = softmax_p(__uint_as_float(v[i]), c, neg_mc);
                    float p1 = softmax_p(__uint_as_float(v[i + 1]), c, neg_mc);
                    if (32 * cc + i > kmax) p0 = 0.0f;
                    if (32 * cc + i + 1 > kmax) p1 = 0.0f;
                    rowsum_add(rs, 32 * cc + i, p0);
                    rowsum_add(rs, 32 * cc + i + 1, p1);
                    pk[i >> 1] = pack_bf16x2(p0, p1);
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int chunk16 = 4 * (cc & 1) + q4;      // 16-byte chunk within the 128 B row
                    const uint32_t off = L::OFF_P + (cc >> 1) * L::ATOM + r * 128 +
                                         ((chunk16 ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(smem + off) =
                        make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
                }
            }
            l_run = __fmaf_rn(l_run, alpha, rs.total());
            m_run = m_new;
            // rescale the chunk accumulator (not on the first tile of a chunk, which overwrites)
            if (!chunk_start && !__all_sync(0xffffffffu, alpha == 1.0f)) {
#pragma unroll
                for (int cc = 0; cc < D / 32; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(tlane + col_o + 32 * cc, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        v[i] = __float_as_uint(rescale_o(__uint_as_float(v[i]), alpha));
                    tmem_st32(tlane + col_o + 32 * cc, v);
                }
                tmem_wait_st();
            }
            fence_proxy_async_smem();
        }
        tc_fence_before();
        __syncthreads();

        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t poff = (ks >> 2) * L::ATOM + (ks & 3) * 32;
                mma_ss(tmem + col_o, smem_desc_sw128(sP + poff, 0, 1024),
                       smem_desc_sw128(sV + st * L::TILE + ks * 2048, L::ATOM, 1024), IDESC_PV,
                       (chunk_start && ks == 0) ? 0u : 1u);
            }
            mma_commit(bar_o);
        }
        mbar_wait(bar_o, par_o, abort_word, p.dev_status);
        par_o ^= 1;
        tc_fence_after();

        if (chunk_end) {
            if (MODE == MODE_DECODE) {
                if (warp == 0 && r < p.G) {
                    const long long slot =
                        (static_cast<long long>(seq) * p.Hq + head + r) * p.nchunk_max + chunk;
                    p.part_ml[2 * slot] = m_run;
                    p.part_ml[2 * slot + 1] = l_run;
                }
                if (warp == 0) {
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t v[32];
                        tmem_ld32(tlane + col_o + 32 * cc, v);
                        tmem_wait_ld();
                        if (r < p.G) {
                            const long long slot =
                                (static_cast<long long>(seq) * p.Hq + head + r) * p.nchunk_max + chunk;
                            float4* dst = reinterpret_cast<float4*>(p.part_o + slot * D + 32 * cc);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                                     __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                        }
                    }
                }
            } else {
                if (chunk_idx == 0) {
                    M_g = m_run;
                    L_g = l_run;
                } else {
                    const FoldCoef f = fold_coef(M_g, m_run, c);
                    L_g = fold_value(L_g, l_run, f);
                    M_g = f.M_new;
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t a[32], b[32];
                        tmem_ld32(tlane + COL_OA + 32 * cc, a);
                        tmem_ld32(tlane + COL_OB + 32 * cc, b);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            a[i] = __float_as_uint(fold_value(__uint_as_float(a[i]), __uint_as_float(b[i]), f));
                        tmem_st32(tlane + COL_OA + 32 * cc, a);
                    }
                    tmem_wait_st();
                }
                m_run = -CUDART_INF_F;
                l_run = 0.0f;
            }
        }
    }

    // ---------------------------------------------------------------- finalise (train / prefill)
    if (MODE != MODE_DECODE) {
        const float inv = finalize_inv(L_g);
        const bool valid = (r >= row_lo) && (r < row_hi);
        const long long orow = (qrow0 + r) * p.Hq + head;
        __nv_bfloat16* optr = reinterpret_cast<__nv_bfloat16*>(p.o) + orow * D;
#pragma unroll
        for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t v[32];
            tmem_ld32(tlane + COL_OA + 32 * cc, v);
            tmem_wait_ld();
            if (valid) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    pk[i] = pack_bf16x2(finalize_o(__uint_as_float(v[2 * i]), inv),
                                        finalize_o(__uint_as_float(v[2 * i + 1]), inv));
                uint4* dst = reinterpret_cast<uint4*>(optr + 32 * cc);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
            }
        }
        if (valid && p.lse) p.lse[orow] = finalize_lse(M_g, L_g, c);
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_word) {   // let copies in flight land before the CTA's shared memory is released
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// ------------------------------------------------------------------ split-KV combine
// One block per (sequence, query head), one thread per head_dim column; folds the chunk
// partials in ascending chunk order and normalises.
template <int D>
__global__ void __launch_bounds__(D) combine_kernel(const AttnParams p) {
    const int b = blockIdx.x / p.Hq;
    const int ctx = p.ctx_lens[b];
    if (ctx <= 0) return;
    const int nc = (ctx + CHUNK - 1) / CHUNK;
    const long long slot0 = static_cast<long long>(blockIdx.x) * p.nchunk_max;
    const int col = threadIdx.x;
    float M = p.part_ml[2 * slot0], Lsum = p.part_ml[2 * slot0 + 1];
    float O = p.part_o[slot0 * D + col];
    for (int ch = 1; ch < nc; ++ch) {
        const float m_c = p.part_ml[2 * (slot0 + ch)], l_c = p.part_ml[2 * (slot0 + ch) + 1];
        const float o_c = p.part_o[(slot0 + ch) * D + col];
        const FoldCoef f = fold_coef(M, m_c, p.c);
        Lsum = fold_value(Lsum, l_c, f);
        O = fold_value(O, o_c, f);
        M = f.M_new;
    }
    const float inv = finalize_inv(Lsum);
    reinterpret_cast<__nv_bfloat16*>(p.o)[static_cast<long long>(blockIdx.x) * D + col] =
        __float2bfloat16_rn(finalize_o(O, inv));
    if (p.lse && col == 0) p.lse[blockIdx.x] = finalize_lse(M, Lsum, p.c);
}

// ------------------------------------------------------------------ KV-cache write
__global__ void __launch_bounds__(128)
kv_write_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                const int32_t* __restrict__ cu_new, const int32_t* __restrict__ ctx_lens,
                uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                const int32_t* __restrict__ block_table, int max_blocks, int S, int Hkv,
                int vec_per_head /* d*2/16 */, int page_size, int num_pages, int* dev_status) {
    const int token = blockIdx.x;
    int lo = 0, hi = S;            // find s with cu_new[s] <= token < cu_new[s+1]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu_new[mid] <= token) lo = mid; else hi = mid;
    }
    const int s = lo;
    const int n_s = cu_new[s + 1] - cu_new[s];
    if (token >= cu_new[s + 1]) return;
    const int pos = ctx_lens[s] - n_s + (token - cu_new[s]);
    if (pos < 0) return;
    const int lp = pos / page_size, row = pos % page_size;
    int phys = (lp < max_blocks) ? block_table[static_cast<long long>(s) * max_blocks + lp] : -1;
    if (phys < 0 || phys >= num_pages) {
        if (threadIdx.x == 0) atomicOr(dev_status, TIK_DEV_BAD_BLOCK);
        return;
    }
    const int nvec = Hkv * vec_per_head;
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
        const int hh = i / vec_per_head, e = i % vec_per_head;
        const long long dst = ((static_cast<long long>(phys) * Hkv + hh) * page_size + row) * vec_per_head + e;
        const long long src = static_cast<long long>(token) * nvec + i;
        k_cache[dst] = k_new[src];
        v_cache[dst] = v_new[src];
    }
}

// ------------------------------------------------------------------ launchers
template <int D, int MODE>
static cudaError_t launch_attn_t(dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                                 const CUtensorMap& tmV, const AttnParams& p, cudaStream_t stream) {
    auto kern = attn_kernel<D, MODE>;
    static bool configured = false;   // per instantiation; attribute is per device function
    cudaError_t e = cudaSuccess;
    if (!configured) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(AttnSmem<D>::ALLOC));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<grid, 128, AttnSmem<D>::ALLOC, stream>>>(tmQ, tmK, tmV, p);
    return cudaGetLastError();
}

cudaError_t launch_attn(int d, int mode, dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                        const CUtensorMap& tmV, const AttnParams& p, cudaStream_t stream) {
    if (d == 128) {
        if (mode == MODE_TRAIN) return launch_attn_t<128, MODE_TRAIN>(grid, tmQ, tmK, tmV, p, stream);
        if (mode == MODE_PREFILL) return launch_attn_t<128, MODE_PREFILL>(grid, tmQ, tmK, tmV, p, stream);
        return launch_attn_t<128, MODE_DECODE>(grid, tmQ, tmK, tmV, p, stream);
    }
    if (mode == MODE_TRAIN) return launch_attn_t<64, MODE_TRAIN>(grid, tmQ, tmK, tmV, p, stream);
    if (mode == MODE_PREFILL) return launch_attn_t<64, MODE_PREFILL>(grid, tmQ, tmK, tmV, p, stream);
    return launch_attn_t<64, MODE_DECODE>(grid, tmQ, tmK, tmV, p, stream);
}

cudaError_t launch_combine(int d, const AttnParams& p, int B, cudaStream_t stream) {
    if (d == 128) combine_kernel<128><<<B * p.Hq, 128, 0, stream>>>(p);
    else combine_kernel<64><<<B * p.Hq, 64, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_kv_write(const void* k_new, const void* v_new, const int32_t* cu_new,
                            const int32_t* ctx_lens, void* k_cache, void* v_cache,
                            const int32_t* block_table, int max_blocks, int S, int64_t total_new,
                            int Hkv, int d, int page_size, int num_pages, int* dev_status,
                            cudaStream_t stream) {
    if (total_new <= 0) return cudaSuccess;
    kv_write_kernel<<<static_cast<unsigned>(total_new), 128, 0, stream>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), cu_new, ctx_lens,
        static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), block_table, max_blocks, S, Hkv,
        d * 2 / 16, page_size, num_pages, dev_status);
    return cudaGetLastError();
}

}  // namespace tik
