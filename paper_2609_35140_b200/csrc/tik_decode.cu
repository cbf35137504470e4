// Decode attention for query groups of up to eight heads: a small CTA, two per SM.
//
// Decode streams every key and value once and is bound by HBM, and its work divides badly: one
// CTA per (sequence, KV head, 2048-key chunk) gives e.g. 256 equal items for 148 SMs -- with one
// resident CTA per SM that is two waves, the second one 27 % empty.  This kernel takes 113 KiB of
// shared memory, 256 tensor-memory columns and 192 threads, so two CTAs share an SM: 296 slots,
// every item resident at once, each SM's HBM stream split between two CTAs whose serial chains
// (K tile -> QK^T -> softmax -> PV) fill each other's gaps.
//
// The arithmetic is attn_kernel<D, decode>'s: the same 128-key tiles at absolute positions, the
// same M128 x N128 x K16 score MMAs and M128 x Nd x K16 value MMAs, the same column split of a
// row over four warps with one warp summing and packing in the contract's order, the same
// per-chunk partials for combine_kernel.  What changes is layout and schedule:
//   * Q is 8 rows x d in shared memory (1 KiB per 64 columns).  The MMA's A descriptor has a
//     stride of ZERO between its 8-row groups, so all sixteen groups of the 128-row operand read
//     the same rows: row i of the group sits on TMEM lanes i, i + 8, ..., in every lane quarter.
//     (attn_kernel spends a 32 KiB tile on the same effect.)
//   * the weights P overwrite the scores S in tensor memory (columns 0..63 of the score buffer):
//     S 128 + O d = 256 columns.  Per CTA the chain QK^T -> softmax -> PV is therefore serial;
//     the co-resident CTA supplies the overlap.
//   * one ring of three 128-key tiles takes K_0, V_0, K_1, V_1, ... in the order of use.
#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

constexpr int DC_THREADS = 192;     // warp 0 TMA (K, V), warp 1 MMA issuer, warps 2..5 softmax
constexpr int DC_SLOTS = 3;

template <int D>
struct DCSmem {
    static constexpr uint32_t ATOM = 128 * 128;          // 128 keys x 64 bf16
    static constexpr uint32_t TILE = (D / 64) * ATOM;    // one K or V tile
    static constexpr uint32_t OFF_RING = 0;
    static constexpr uint32_t OFF_Q = DC_SLOTS * TILE;                       // D / 64 atoms of 8 rows x 128 bytes
    static constexpr uint32_t OFF_XCH = OFF_Q + (D / 64) * 1024;             // 3 x 8 x 32 float4 weights + 4 x 32 maxima
    static constexpr uint32_t XCH_BYTES = 3 * 8 * 32 * 16 + 4 * 32 * 4;
    static constexpr uint32_t OFF_BAR = OFF_XCH + XCH_BYTES;
    static constexpr uint32_t BYTES = OFF_BAR + 128;
};

// QK^T chain for the compact query tile: A atoms are 1 KiB (64 descriptor units) apart, B atoms 16 KiB.
__device__ __forceinline__ void mma_ss_chain8_fresh_qcompact(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p0, pt;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p0;\n\t"
        TIK_MMA_SS_STEP(2, 2) TIK_MMA_SS_STEP(4, 4) TIK_MMA_SS_STEP(6, 6)
        TIK_MMA_SS_STEP(64, 1024) TIK_MMA_SS_STEP(66, 1026) TIK_MMA_SS_STEP(68, 1028)
        TIK_MMA_SS_STEP(70, 1030)
        "}" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
}

template <int D>
__global__ void __launch_bounds__(DC_THREADS, 2)
decode2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnParams p) {
    using L = DCSmem<D>;
    constexpr int NATOM = D / 64;
    constexpr uint32_t TMEM_COLS = 256;
    constexpr uint32_t COL_S = 0;              // scores (128 columns); the packed weights overwrite columns 0..63
    constexpr uint32_t COL_O = 128;            // the chunk's accumulator (D columns)
    constexpr uint32_t IDESC_QK = mma_idesc_bf16(128, 128, false);
    constexpr uint32_t IDESC_PV = mma_idesc_bf16(128, D, true);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_wait();
    pdl_launch_dependents();       // the combine kernel may be scheduled behind this grid's last wave

    const int seq = blockIdx.z, kvh = blockIdx.y;
    const int head = kvh * p.G;
    int ctx = p.ctx_lens[seq];
    if (ctx > p.max_ctx) {
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) atomicOr(p.dev_status, TIK_DEV_BAD_CONTEXT);
        ctx = p.max_ctx;
    }
    const int chunk0 = blockIdx.x * p.cpc;                      // a CTA streams cpc consecutive chunks
    if (ctx <= 0 || chunk0 * CHUNK >= ctx) return;
    const int tile_first = chunk0 * TILES_PER_CHUNK;
    const int tile_last = min(tile_first + p.cpc * TILES_PER_CHUNK - 1, (ctx - 1) / 128);
    const int n_tiles = tile_last - tile_first + 1;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    const uint32_t sbase = smem_u32(smem_raw);
    if (sbase & 1023u) {
        if (tid == 0) atomicOr(p.dev_status, TIK_DEV_WAIT_EXPIRED);
        return;
    }
    const uint32_t sRing = sbase + L::OFF_RING, sQ = sbase + L::OFF_Q;
    const uint32_t bar0 = sbase + L::OFF_BAR;
    const uint32_t bar_full = bar0;              // [3] tile landed in slot
    const uint32_t bar_empty = bar0 + 24;        // [3] the MMA that read the slot is done
    const uint32_t bar_q = bar0 + 48;            // query rows landed
    const uint32_t bar_sfull = bar0 + 56;        // scores of a tile ready
    const uint32_t bar_pfull = bar0 + 64;        // weights written over the scores, accumulator rescaled
    const uint32_t bar_pvdone = bar0 + 72;       // PV of a tile done
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_BAR + 80);
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 84);

    // ---------------------------------------------------------------- set-up
    // The producer warp prepares what it needs by itself (its ring barriers, the zeroed query
    // atoms) and puts the query rows and the first tiles in flight before the CTA-wide
    // synchronisation, so the first data arrive while tensor memory is being allocated.
    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            for (int i = 0; i < 7; ++i) mbar_init(bar0 + 8 * i, 1);       // full[3], empty[3], q
            fence_barrier_init();
        }
        // rows >= G of the query atoms are never loaded: zero them (finite scores for the unused rows)
        for (uint32_t i = lane; i < NATOM * 1024 / 16; i += 32)
            reinterpret_cast<uint4*>(smem + L::OFF_Q)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            for (int i = 7; i < 10; ++i) mbar_init(bar0 + 8 * i, 1);      // sfull, pfull, pvdone
            fence_barrier_init();
            *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
        }
        __syncwarp();
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    }
    int my_phys = p.num_pages;                              // producer: one block-table entry per lane
    auto produce = [&](int n) {                             // load n: K (even) or V (odd) of tile n / 2; whole warp 0
        const int tpb_mask = (32 >> p.ppt_shift) - 1;       // tiles per block-table batch - 1
        const int it = n >> 1, kv = n & 1;
        const int j = tile_first + it;
        if (kv == 0 && (it & tpb_mask) == 0) {
            const int lp = ((128 * j) >> p.page_shift) + lane;
            int ph = p.num_pages;       // out of range: the box is filled with zeros
            if ((lp << p.page_shift) < ctx) {
                ph = (lp < p.max_blocks) ? p.block_table[static_cast<long long>(seq) * p.max_blocks + lp] : -1;
                if (ph < 0 || ph >= p.num_pages) {
                    atomicOr(p.dev_status, TIK_DEV_BAD_BLOCK);
                    ph = p.num_pages;
                }
            }
            my_phys = ph;
        }
        const int in_batch = it & tpb_mask;
        const int my_page = __shfl_sync(0xffffffffu, my_phys, (in_batch << p.ppt_shift) + (lane & (p.pages_per_tile - 1)));
        const int slot = n % DC_SLOTS;
        const uint32_t use = n / DC_SLOTS;
        if (use > 0) mbar_wait(bar_empty + 8 * slot, (use - 1) & 1, abort_word, p.dev_status);
        const uint32_t full = bar_full + 8 * slot, dst = sRing + slot * L::TILE;
        if (lane == 0) mbar_expect_tx(full, L::TILE);
        __syncwarp();                                       // the expected byte count is registered first
        if (lane < p.pages_per_tile) {
            const uint32_t off = static_cast<uint32_t>(lane << p.page_shift) * 128u;
            for (int a = 0; a < NATOM; ++a)
                tma_load_4d(dst + a * L::ATOM + off, kv ? &tmV : &tmK, full, a * 64, 0, kvh, my_page);
        }
    };
    const int n_early = min(2 * n_tiles, DC_SLOTS);         // loads that need no slot release
    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(bar_q, static_cast<uint32_t>(p.G) * 128u * NATOM);
            for (int a = 0; a < NATOM; ++a) tma_load_3d(sQ + a * 1024, &tmQ, bar_q, a * 64, head, seq);
        }
        for (int n = 0; n < n_early; ++n) produce(n);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (whole warp)
        for (int n = n_early; n < 2 * n_tiles; ++n) {
            if (__any_sync(0xffffffffu, *abort_word != 0)) break;
            produce(n);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            mbar_wait(bar_q, 0, abort_word, p.dev_status);
            const uint64_t dq = smem_desc_sw128(sQ, 0, 0);      // stride 0 between 8-row groups: every group reads rows 0..7
            for (int it = 0; it < n_tiles; ++it) {
                if (*abort_word) break;
                const int nk = 2 * it, nv = 2 * it + 1;
                const int sk = nk % DC_SLOTS, sv = nv % DC_SLOTS;
                // scores: the previous tile's PV (issued by this thread, executed in order) has read
                // the weights that these scores overwrite
                mbar_wait(bar_full + 8 * sk, (nk / DC_SLOTS) & 1, abort_word, p.dev_status);
                tc_fence_after();
                const uint64_t dk = smem_desc_sw128(sRing + sk * L::TILE, 0, 1024);
                if (D == 128) mma_ss_chain8_fresh_qcompact(tmem + COL_S, dq, dk, IDESC_QK);
                else mma_ss_chain4_fresh(tmem + COL_S, dq, dk, IDESC_QK);
                mma_commit(bar_sfull);
                mma_commit(bar_empty + 8 * sk);
                // values
                mbar_wait(bar_full + 8 * sv, (nv / DC_SLOTS) & 1, abort_word, p.dev_status);
                mbar_wait(bar_pfull, it & 1, abort_word, p.dev_status);
                tc_fence_after();
                const bool fresh = ((tile_first + it) % TILES_PER_CHUNK) == 0;
                mma_ts_chain8(tmem + COL_O, tmem + COL_S, smem_desc_sw128(sRing + sv * L::TILE, L::ATOM, 1024),
                              IDESC_PV, fresh ? 0u : 1u);
                mma_commit(bar_pvdone);
                mma_commit(bar_empty + 8 * sv);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ softmax (warps 2..5)
        // Lane i < G of every lane quarter holds query head i.  Warp `quarter` takes columns
        // [32 quarter, 32 quarter + 32) of every row: tile maximum by an exchange through shared memory,
        // exponentials on all four warps, then the warp of quarter 0 alone adds the 128 weights of a
        // row in the contract's order, packs them and writes them over the scores.
        const int quarter = warp & 3;
        const uint32_t tlane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const float c = p.c;
        float4* xs = reinterpret_cast<float4*>(smem + L::OFF_XCH);                          // [3][8][32]
        float* xm = reinterpret_cast<float*>(smem + L::OFF_XCH + 3 * 8 * 32 * 16);          // [4][32]
        float m_run = -CUDART_INF_F, l_lo = 0.0f, l_hi = 0.0f;    // l_*: only the warp of quarter 0 keeps them

        auto wait_pv = [&](int x) {          // PV of this CTA's tile x
            mbar_wait(bar_pvdone, x & 1, abort_word, p.dev_status);
            tc_fence_after();
        };
        // partial of a finished chunk: (m, l_lo, l_hi) and the accumulator rows of the G heads
        auto write_partial = [&](int chunk_idx) {
            if (p.direct_out) {
                // one chunk per sequence: the partial is the result (see the decode mode of attn_kernel)
                const float Ltot = finalize_l(l_lo, l_hi);
                const float inv = finalize_inv(Ltot);
                const long long orow = static_cast<long long>(seq) * p.Hq + head + lane;
                __nv_bfloat16* const og = reinterpret_cast<__nv_bfloat16*>(p.o) + orow * D;
#pragma unroll 1
                for (int cc = 0; cc < D / 32; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(tlane + COL_O + 32 * cc, v);
                    tmem_wait_ld();
                    if (lane < p.G) {
                        uint4* dst = reinterpret_cast<uint4*>(og + 32 * cc);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            dst[i] = make_uint4(
                                pack_bf16x2(finalize_o(__uint_as_float(v[8 * i]), inv), finalize_o(__uint_as_float(v[8 * i + 1]), inv)),
                                pack_bf16x2(finalize_o(__uint_as_float(v[8 * i + 2]), inv), finalize_o(__uint_as_float(v[8 * i + 3]), inv)),
                                pack_bf16x2(finalize_o(__uint_as_float(v[8 * i + 4]), inv), finalize_o(__uint_as_float(v[8 * i + 5]), inv)),
                                pack_bf16x2(finalize_o(__uint_as_float(v[8 * i + 6]), inv), finalize_o(__uint_as_float(v[8 * i + 7]), inv)));
                    }
                }
                if (lane < p.G && p.lse) p.lse[orow] = finalize_lse(m_run, Ltot, c);
                return;
            }
            if (lane < p.G) {
                const long long slot = (static_cast<long long>(seq) * p.Hq + head + lane) * p.nchunk_max + chunk_idx;
                p.part_ml[4 * slot] = m_run;
                p.part_ml[4 * slot + 1] = l_lo;
                p.part_ml[4 * slot + 2] = l_hi;
            }
#pragma unroll 1
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t v[32];
                tmem_ld32(tlane + COL_O + 32 * cc, v);
                tmem_wait_ld();
                if (lane < p.G) {
                    const long long slot = (static_cast<long long>(seq) * p.Hq + head + lane) * p.nchunk_max + chunk_idx;
                    float4* dst = reinterpret_cast<float4*>(p.part_o + slot * D + 32 * cc);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                             __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                }
            }
        };

        for (int it = 0; it < n_tiles; ++it) {
            if (__any_sync(0xffffffffu, *abort_word != 0)) break;
            const int j = tile_first + it;
            const bool chunk_start = (j % TILES_PER_CHUNK) == 0;
            if (chunk_start && it > 0 && quarter == 0) {
                // a finished chunk precedes this tile: its partial leaves before this chunk's first PV
                // (which waits for this tile's weights) overwrites the accumulator
                wait_pv(it - 1);
                write_partial(j / TILES_PER_CHUNK - 1);
                tc_fence_before();
            }
            mbar_wait(bar_sfull, it & 1, abort_word, p.dev_status);
            tc_fence_after();
            uint32_t sc[32];
            tmem_ld32(tlane + COL_S + 32 * quarter, sc);
            tmem_wait_ld();
            const int kmax = (ctx - 1) - 128 * j - 32 * quarter;    // own columns > kmax are masked
            if (kmax < 31) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i > kmax) sc[i] = 0xff800000u;              // -inf
            }
            float mx[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) mx[q] = fmaxf(__uint_as_float(sc[2 * q]), __uint_as_float(sc[2 * q + 1]));
#pragma unroll
            for (int i = 8; i < 32; i += 8) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    mx[q] = fmax3(mx[q], __uint_as_float(sc[i + 2 * q]), __uint_as_float(sc[i + 2 * q + 1]));
            }
            xm[quarter * 32 + lane] = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            tc_fence_before();
            named_bar_sync(1, 128);              // maxima exchanged; every warp holds its scores in registers
            const float mt = fmaxf(fmaxf(xm[lane], xm[32 + lane]), fmaxf(xm[64 + lane], xm[96 + lane]));
            const float m_old = chunk_start ? -CUDART_INF_F : m_run;
            const float m_new = softmax_next_max(m_old, mt, c);
            m_run = m_new;
            const float neg_mc = -__fmul_rn(m_new, c);
            float x[32];
#pragma unroll
            for (int i = 0; i < 32; i += 8) softmax_x8(&sc[i], c, neg_mc, &x[i]);
            if (quarter != 0) {
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4)
                    xs[((quarter - 1) * 8 + c4) * 32 + lane] = make_float4(x[4 * c4], x[4 * c4 + 1], x[4 * c4 + 2], x[4 * c4 + 3]);
            }
            named_bar_sync(1, 128);              // weights of columns 32..127 are in shared memory
            if (quarter == 0) {
                tc_fence_after();
                RowSum4 rs_lo, rs_hi;
                rs_lo.reset();
                rs_hi.reset();
                uint32_t pk[32];
                // columns 0..63: own 32, then 32 of warp 1
#pragma unroll
                for (int i = 0; i < 32; i += 8) softmax_sum_pack8(&x[i], rs_lo, &pk[i >> 1]);
#pragma unroll
                for (int k4 = 0; k4 < 8; k4 += 2) {
                    const float4 a = xs[k4 * 32 + lane], b = xs[(k4 + 1) * 32 + lane];
                    const float y[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                    softmax_sum_pack8(y, rs_lo, &pk[16 + 2 * k4]);
                }
                tmem_st32(tlane + COL_S, pk);
                // columns 64..127
#pragma unroll
                for (int k4 = 8; k4 < 24; k4 += 2) {
                    const float4 a = xs[k4 * 32 + lane], b = xs[(k4 + 1) * 32 + lane];
                    const float y[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                    softmax_sum_pack8(y, rs_hi, &pk[2 * (k4 - 8)]);
                }
                tmem_st32(tlane + COL_S + 32, pk);
                const float alpha = softmax_alpha(m_old, m_new, c);
                l_lo = __fmaf_rn(chunk_start ? 0.0f : l_lo, alpha, rs_lo.total());
                l_hi = __fmaf_rn(chunk_start ? 0.0f : l_hi, alpha, rs_hi.total());
                if (!chunk_start && !__all_sync(0xffffffffu, alpha == 1.0f)) {
                    wait_pv(it - 1);             // the accumulator holds every earlier tile of the chunk
#pragma unroll 1
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t v[32];
                        tmem_ld32(tlane + COL_O + 32 * cc, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(rescale_o(__uint_as_float(v[i]), alpha));
                        tmem_st32(tlane + COL_O + 32 * cc, v);
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pfull);
            }
        }
        // ---- the last chunk's partial
        if (quarter == 0 && !__any_sync(0xffffffffu, *abort_word != 0)) {
            wait_pv(n_tiles - 1);
            write_partial(tile_last / TILES_PER_CHUNK);
        }
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_word) {   // let copies and MMAs in flight finish before shared memory and TMEM are released
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 1000000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

template <int D>
static cudaError_t launch_decode2_t(dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                    const AttnParams& p, cudaStream_t stream) {
    auto kern = decode2_kernel<D>;
    static DeviceOnce configured;     // the shared-memory opt-in belongs to the (function, device) pair
    cudaError_t e = configured.run([&]() {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(DCSmem<D>::BYTES));
    });
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(DC_THREADS);
    cfg.dynamicSmemBytes = DCSmem<D>::BYTES;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, p);
}

// Decode for G <= 8 (the caller checks); grid as for attn_kernel's decode mode.
cudaError_t launch_decode2(int d, dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                           const AttnParams& p, cudaStream_t stream) {
    if (d == 128) return launch_decode2_t<128>(grid, tmQ, tmK, tmV, p, stream);
    return launch_decode2_t<64>(grid, tmQ, tmK, tmV, p, stream);
}

}  // namespace tik
