// Token log-probability for sm_100a: lm_head GEMM on tcgen05 fused with a chunked
// log-sum-exp over the vocabulary and the target-logit gather.  The fp32 logits live only
// in TMEM; nothing of size T x V is ever written.
//
// One CTA = (128-token tile, 1024-column super-chunk).  For each of the (up to) four
// 256-column steps of the super-chunk, a TMA warp streams 64-wide K slices of hidden and
// lm_head through a shared-memory ring, an MMA warp accumulates the whole K range in
// ascending order into one of two 256-column TMEM accumulators (M128 x N256 x K16 MMAs, no
// split-K), and four epilogue warps (one thread per token row) reduce each of its two
// 128-column tiles to (max, sum of exp) with the fixed row-sum shape, fold them in ascending
// order into the super-chunk's running pair, and pick the target logit if a tile owns its
// column.  A finish kernel folds the super-chunk pairs of every token in
// ascending order and writes logprob = z_target - logsumexp.
#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

namespace lp {
constexpr int NB = 256;                      // vocabulary columns per MMA (two log-sum-exp tiles)
constexpr uint32_t A_BYTES = 128 * 128;      // 128 token rows x 64 bf16
constexpr int BAND = 32;                     // token tiles per L2 band (even: CTA pairs stay inside a band)
constexpr int THREADS = 192;                 // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
// PAIR: two CTAs on neighbouring SMs (a cluster of two) share every MMA: M = 256 token rows, each
// CTA stages its own 128 token rows and half (128 rows) of the 256 lm_head rows, so a stage is
// 32 KiB instead of 48 and the B operand crosses shared memory once per 256 token rows.
template <bool PAIR>
struct Cfg {
    static constexpr int STAGES = PAIR ? 6 : 4;
    static constexpr uint32_t B_BYTES = (PAIR ? NB / 2 : NB) * 128;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr uint32_t OFF_BAR = STAGES * STAGE_BYTES;
    static constexpr uint32_t BYTES = OFF_BAR + 256;
    static constexpr uint32_t ALLOC = BYTES + 1024;
};
}  // namespace lp

template <bool PAIR>
__global__ void __launch_bounds__(lp::THREADS, 1)
logprob_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const LogprobParams p) {
    using namespace lp;
    using C = Cfg<PAIR>;
    constexpr int STAGES = C::STAGES;
    constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES, OFF_BAR = C::OFF_BAR;
    constexpr uint32_t TMEM_COLS = 512;      // two 256-column accumulators
    constexpr uint32_t IDESC = mma_idesc_bf16(PAIR ? 256 : 128, NB, false);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;     // 0 = the CTA that issues the pair's MMAs
    pdl_launch_dependents();           // the finish kernel may be scheduled behind this grid's last wave

    // raster: bands of BAND token tiles; within a band the token tile varies fastest so the
    // CTAs in flight share one lm_head super-chunk and the band's hidden rows stay in L2
    const int ntile = static_cast<int>((p.T + 127) / 128);
    const int ngroup = (p.nsuper + p.spc - 1) / p.spc;      // a CTA walks spc consecutive super-chunks
    const long long per_band = static_cast<long long>(BAND) * ngroup;
    const int band = static_cast<int>(blockIdx.x / per_band);
    const int band_tiles = min(BAND, ntile - band * BAND);
    const long long rem = blockIdx.x - band * per_band;
    // (blockIdx.x enumerates BAND * nsuper slots per band; slots beyond a short last band exit)
    const int sup0 = static_cast<int>(rem / BAND) * p.spc;
    const int n_sp = min(p.spc, p.nsuper - sup0);
    const int tile_in_band = static_cast<int>(rem % BAND);
    // (a pair leaves only together: a lone tile at the end of T keeps its partner, whose rows lie
    // past T, arrive as zeros and are never stored)
    // Unit mode (calls of one or two token tiles, i.e. decode-sized batches): such a call streams all
    // of lm_head once and is bound by HBM, and V / 1024 super-chunks do not divide over the SMs (149
    // on 148: a second wave for one CTA).  There a CTA (pair) is persistent and takes the 256-column
    // accumulator steps u, u + n, u + 2n, ... of the vocabulary; every 128-column tile leaves its own
    // (max, sum) pair and the finish kernel folds them in the fixed order (tiles ascending inside a
    // super-chunk, then super-chunks ascending): the same operations on the same numbers.
    // With more than two token tiles (up to LP_UNIT_MODE_ROWS rows) a unit is (256-column step,
    // pair of token tiles), the pair index running fastest: the CTA pairs at work at one time share a
    // few steps of lm_head in L2, and the hidden rows stay there throughout.
    const bool unit_mode = p.unit_mode != 0;
    const int u_first = static_cast<int>(blockIdx.x) / (PAIR ? 2 : 1);
    const int u_stride = static_cast<int>(gridDim.x) / (PAIR ? 2 : 1);
    const int n_my_units = unit_mode ? (u_first < p.nunit ? (p.nunit - 1 - u_first) / u_stride + 1 : 0) : 0;
    if (!unit_mode && (PAIR ? (tile_in_band & ~1) : tile_in_band) >= band_tiles) return;
    const int ntp = unit_mode ? p.ntp : 1;
    const int tok_fixed = (band * BAND + tile_in_band) * 128;
    auto unit_col = [&](int sp) { return ((u_first + sp * u_stride) / ntp) * NB; };
    auto unit_tok = [&](int sp) {
        const int pi = (u_first + sp * u_stride) % ntp;
        return (PAIR ? 2 * pi + static_cast<int>(rank) : pi) * 128;
    };
    // 256-column accumulator steps of super-chunk sup0 + sp
    auto n_nt_of = [&](int sp) { return min(LP_SUPER / NB, (p.V - (sup0 + sp) * LP_SUPER + NB - 1) / NB); };
    const int n_kb = p.H / 64;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw_addr + pad;
    const uint32_t bar_full = sbase + OFF_BAR;               // STAGES barriers
    const uint32_t bar_empty = bar_full + 8 * STAGES;        // STAGES barriers
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES;    // 2
    const uint32_t bar_acc_empty = bar_acc_full + 16;        // 2
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 8 * (2 * STAGES + 4));
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8 * (2 * STAGES + 4) + 4);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, PAIR ? 256 : 128);   // the epilogue threads of every CTA of the pair
        }
        *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        if (PAIR) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();            // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // the leader's copies of the barriers that both CTAs signal (shared::cluster addresses)
    const uint32_t lead_full = PAIR ? mapa_cluster(bar_full, 0) : bar_full;
    const uint32_t lead_acc_empty = PAIR ? mapa_cluster(bar_acc_empty, 0) : bar_acc_empty;
    const uint32_t peer_empty = PAIR ? mapa_cluster(bar_empty, 1) : bar_empty;
    const uint32_t peer_acc_full = PAIR ? mapa_cluster(bar_acc_full, 1) : bar_acc_full;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            // accumulator steps of this CTA: unit mode a strided list, else spc super-chunks x up to 4
            const int n_sp_loop = unit_mode ? n_my_units : n_sp;
            for (int sp = 0; sp < n_sp_loop; ++sp)
            for (int nt = 0; nt < (unit_mode ? 1 : n_nt_of(sp)); ++nt) {
                const int col0 = unit_mode ? unit_col(sp) : (sup0 + sp) * LP_SUPER + nt * NB;
                const int tok0 = unit_mode ? unit_tok(sp) : tok_fixed;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    if (*abort_word) break;      // a wait expired somewhere: stop issuing copies
                    const int s = it % STAGES;
                    const uint32_t use = it / STAGES;
                    if (use > 0) mbar_wait(bar_empty + 8 * s, (use - 1) & 1, abort_word, p.dev_status);
                    if (PAIR) {
                        // both CTAs' bytes are counted on the leader's barrier, which the leader arms;
                        // a peer copy that lands first only makes the count negative for a moment
                        if (rank == 0) mbar_expect_tx(bar_full + 8 * s, 2 * STAGE_BYTES);
                        tma_load_2d_pair(sbase + s * STAGE_BYTES, &tmA, lead_full + 8 * s, kb * 64, tok0);
                        tma_load_2d_pair(sbase + s * STAGE_BYTES + A_BYTES, &tmB, lead_full + 8 * s, kb * 64,
                                         col0 + 128 * static_cast<int>(rank));
                    } else {
                        mbar_expect_tx(bar_full + 8 * s, STAGE_BYTES);
                        tma_load_2d(sbase + s * STAGE_BYTES, &tmA, bar_full + 8 * s, kb * 64, tok0);
                        tma_load_2d(sbase + s * STAGE_BYTES + A_BYTES, &tmB, bar_full + 8 * s, kb * 64, col0);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, acc = 0;              // acc counts accumulator steps across super-chunks
            const int n_sp_loop = unit_mode ? n_my_units : n_sp;
            for (int sp = 0; sp < n_sp_loop; ++sp)
            for (int nt = 0; nt < (unit_mode ? 1 : n_nt_of(sp)); ++nt, ++acc) {
                const int buf = acc & 1;
                const uint32_t use = acc >> 1;
                if (use > 0) mbar_wait(bar_acc_empty + 8 * buf, (use - 1) & 1, abort_word, p.dev_status);
                tc_fence_after();
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    if (*abort_word) break;
                    const int s = it % STAGES;
                    mbar_wait(bar_full + 8 * s, (it / STAGES) & 1, abort_word, p.dev_status);
                    tc_fence_after();
                    const uint32_t a0 = sbase + s * STAGE_BYTES, b0 = a0 + A_BYTES;
                    if (PAIR) {
                        mma_ss_chain4_pair(tmem + buf * NB, smem_desc_sw128(a0, 0, 1024), smem_desc_sw128(b0, 0, 1024),
                                           IDESC, kb ? 1u : 0u);
                        mma_commit_pair(bar_empty + 8 * s);          // the stage is free in this CTA ...
                        mma_commit_pair(peer_empty + 8 * s);         // ... and in the peer
                    } else {
                        mma_ss_chain4(tmem + buf * NB, smem_desc_sw128(a0, 0, 1024), smem_desc_sw128(b0, 0, 1024),
                                      IDESC, kb ? 1u : 0u);
                        mma_commit(bar_empty + 8 * s);
                    }
                }
                if (PAIR) {
                    mma_commit_pair(bar_acc_full + 8 * buf);
                    mma_commit_pair(peer_acc_full + 8 * buf);
                } else {
                    mma_commit(bar_acc_full + 8 * buf);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                      // TMEM lane quarter of this warp
        const int row = quarter * 32 + lane;
        long long t = static_cast<long long>(tok_fixed) + row;
        bool row_valid = t < p.T;
        int target = (!unit_mode && row_valid) ? p.target[t] : -1;
        const float it_scale = p.inv_temperature;
        uint32_t acc = 0;
        const int n_sp_loop = unit_mode ? n_my_units : n_sp;
        for (int sp = 0; sp < n_sp_loop; ++sp) {
        const int col_base = unit_mode ? unit_col(sp) : (sup0 + sp) * LP_SUPER;
        if (unit_mode) {                                   // the unit's token tile
            t = static_cast<long long>(unit_tok(sp)) + row;
            row_valid = t < p.T;
            target = row_valid ? p.target[t] : -1;
        }
        float M = -CUDART_INF_F, Lsum = 0.0f;
        bool first = true;
        for (int nt = 0; nt < (unit_mode ? 1 : n_nt_of(sp)); ++nt, ++acc) {
            const int buf = acc & 1;
            mbar_wait(bar_acc_full + 8 * buf, (acc >> 1) & 1, abort_word, p.dev_status);
            tc_fence_after();
#pragma unroll 1
            for (int half = 0; half < NB / LP_TILE; ++half) {
                const int col0 = col_base + nt * NB + half * LP_TILE;
                if (col0 >= p.V) break;                        // tile entirely past the vocabulary
                const uint32_t taddr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * NB + half * LP_TILE;
                const int vmax = p.V - 1 - col0;               // columns > vmax are past the vocabulary
                float mt = -CUDART_INF_F;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(taddr + 32 * cc, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float z = __fmul_rn(__uint_as_float(v[i]), it_scale);
                        if (32 * cc + i > vmax) z = -CUDART_INF_F;
                        mt = fmaxf(mt, z);
                    }
                }
                const float neg_mc = -__fmul_rn(mt, LOG2E_F);
                const int tcol = target - col0;                // in [0,128) when this tile owns the target
                float zt = 0.0f;
                RowSum8 rs;
                rs.reset();
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(taddr + 32 * cc, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float z = __fmul_rn(__uint_as_float(v[i]), it_scale);
                        float e = softmax_p(z, LOG2E_F, neg_mc);
                        if (32 * cc + i > vmax) e = 0.0f;
                        rowsum_add(rs, 32 * cc + i, e);
                        if (32 * cc + i == tcol) zt = z;
                    }
                }
                const float lt = rs.total();
                if (unit_mode) {
                    // the tile's own pair; folded later by the finish kernel
                    if (row_valid) {
                        const long long slot = t * p.ntile128 + (col0 >> 7);
                        p.part_ml[2 * slot] = mt;
                        p.part_ml[2 * slot + 1] = lt;
                    }
                } else if (first) {
                    M = mt;
                    Lsum = lt;
                    first = false;
                } else {
                    const FoldCoef f = fold_coef(M, mt, LOG2E_F);
                    Lsum = fold_value(Lsum, lt, f);
                    M = f.M_new;
                }
                if (row_valid && tcol >= 0 && tcol < LP_TILE && target < p.V) p.z_target[t] = zt;
            }
            // all TMEM reads of this accumulator are done: hand it back to the MMA warp
            tc_fence_before();
            if (PAIR) mbar_arrive_cluster(lead_acc_empty + 8 * buf);
            else mbar_arrive(bar_acc_empty + 8 * buf);
        }
        if (row_valid && !unit_mode) {
            p.part_ml[2 * (t * p.nsuper + sup0 + sp)] = M;
            p.part_ml[2 * (t * p.nsuper + sup0 + sp) + 1] = Lsum;
        }
        }
    }

    if (*abort_word) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 1000000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();            // neither CTA leaves while the other may still touch it
    if (warp == 1) {
        if (PAIR) tmem_dealloc_pair(tmem, TMEM_COLS);
        else tmem_dealloc(tmem, TMEM_COLS);
    }
}

// One thread per token: fold the super-chunk pairs in ascending order, write the result.
__global__ void __launch_bounds__(256) logprob_finish_kernel(const LogprobParams p) {
    pdl_wait();                        // the super-chunk pairs and target logits are complete and visible
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= p.T) return;
    const float* ml = p.part_ml + 2 * t * p.nsuper;
    float M = ml[0], Lsum = ml[1];
    for (int s = 1; s < p.nsuper; ++s) {
        const FoldCoef f = fold_coef(M, ml[2 * s], LOG2E_F);
        Lsum = fold_value(Lsum, ml[2 * s + 1], f);
        M = f.M_new;
    }
    const float lse = lp_lse(M, Lsum);
    if (p.lse) p.lse[t] = lse;
    const int target = p.target[t];
    if (target < 0 || target >= p.V) {
        atomicOr(p.dev_status, TIK_DEV_BAD_TARGET);
        p.logprob[t] = CUDART_NAN_F;
    } else {
        p.logprob[t] = __fsub_rn(p.z_target[t], lse);
    }
}

// Unit mode: one block per token.  Thread s folds the tiles of super-chunk s in ascending order
// (first tile copied, the others folded: the main kernel's in-CTA sequence), then thread 0 folds
// the super-chunks in ascending order as logprob_finish_kernel does.
__global__ void __launch_bounds__(256) logprob_finish_tiles_kernel(const LogprobParams p) {
    pdl_wait();
    __shared__ float sm[256], sl[256];
    const long long t = blockIdx.x;
    const float* ml = p.part_ml + 2 * t * p.ntile128;
    constexpr int TPS = LP_SUPER / LP_TILE;        // tiles per super-chunk
    for (int s0 = 0; s0 < p.nsuper; s0 += 256) {
        const int s = s0 + threadIdx.x;
        float M = 0.0f, Lsum = 0.0f;
        if (s < p.nsuper) {
            const int t0 = s * TPS, t1 = min(p.ntile128, t0 + TPS);
            M = ml[2 * t0];
            Lsum = ml[2 * t0 + 1];
            for (int j = t0 + 1; j < t1; ++j) {
                const FoldCoef f = fold_coef(M, ml[2 * j], LOG2E_F);
                Lsum = fold_value(Lsum, ml[2 * j + 1], f);
                M = f.M_new;
            }
        }
        __syncthreads();                            // (the previous batch of super-chunks has been consumed)
        sm[threadIdx.x] = M;
        sl[threadIdx.x] = Lsum;
        __syncthreads();
        if (threadIdx.x == 0) {
            // running total kept in sm[0] / sl[0] across batches of 256 super-chunks
            float Mt = sm[0], Lt = sl[0];
            if (s0 > 0) {
                // restore the running total saved below, then fold this batch's first entry
                const float Mr = p.part_ml[2 * t * p.ntile128], Lr = p.part_ml[2 * t * p.ntile128 + 1];
                const FoldCoef f = fold_coef(Mr, Mt, LOG2E_F);
                Lt = fold_value(Lr, Lt, f);
                Mt = f.M_new;
            }
            const int n = min(256, p.nsuper - s0);
            for (int i = 1; i < n; ++i) {
                const FoldCoef f = fold_coef(Mt, sm[i], LOG2E_F);
                Lt = fold_value(Lt, sl[i], f);
                Mt = f.M_new;
            }
            if (s0 + 256 < p.nsuper) {              // more batches follow: park the running total
                p.part_ml[2 * t * p.ntile128] = Mt;
                p.part_ml[2 * t * p.ntile128 + 1] = Lt;
            } else {
                const float lse = lp_lse(Mt, Lt);
                if (p.lse) p.lse[t] = lse;
                const int target = p.target[t];
                if (target < 0 || target >= p.V) {
                    atomicOr(p.dev_status, TIK_DEV_BAD_TARGET);
                    p.logprob[t] = CUDART_NAN_F;
                } else {
                    p.logprob[t] = __fsub_rn(p.z_target[t], lse);
                }
            }
        }
    }
}

template <bool PAIR>
static cudaError_t launch_logprob_main(const CUtensorMap& tmA, const CUtensorMap& tmB, const LogprobParams& p,
                                       cudaStream_t stream) {
    using C = lp::Cfg<PAIR>;
    auto kern = logprob_kernel<PAIR>;
    static DeviceOnce configured;     // the opt-in belongs to the (function, device) pair
    {
        cudaError_t e = configured.run([&]() {
            return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(C::ALLOC));
        });
        if (e != cudaSuccess) return e;
    }
    const long long ntile = (p.T + 127) / 128;
    const long long nband = (ntile + lp::BAND - 1) / lp::BAND;
    long long grid = nband * lp::BAND * ((p.nsuper + p.spc - 1) / p.spc);   // even: BAND is
    if (p.unit_mode) {       // persistent CTAs (pairs), one per SM (two SMs), never more than there are units
        const long long slots = PAIR ? p.sm_count / 2 : p.sm_count;
        grid = (slots < p.nunit ? slots : p.nunit) * (PAIR ? 2 : 1);
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(lp::THREADS);
    cfg.dynamicSmemBytes = C::ALLOC;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, p);
}

// pair = true: tmB must have a box of 128 rows (each CTA of a pair stages half of the 256 columns)
cudaError_t launch_logprob(const CUtensorMap& tmA, const CUtensorMap& tmB, const LogprobParams& p, bool pair,
                           cudaStream_t stream) {
    if (p.T <= 0) return cudaSuccess;
    cudaError_t e = pair ? launch_logprob_main<true>(tmA, tmB, p, stream) : launch_logprob_main<false>(tmA, tmB, p, stream);
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(p.unit_mode ? p.T : (p.T + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();  // exactly one of the launches below runs
    if (p.unit_mode) return cudaLaunchKernelEx(&cfg, logprob_finish_tiles_kernel, p);
    return cudaLaunchKernelEx(&cfg, logprob_finish_kernel, p);
}

}  // namespace tik
