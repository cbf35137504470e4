// Backward of the packed causal GQA attention (policy-update backward) for sm_100a.
//
// Deterministic by construction: no atomics and no split accumulation.  Two launches of one
// kernel body recompute the score tiles and differ in which side stays resident:
//   DQ  mode: a CTA owns one 128-row query tile of one (sequence, head) and walks the KV tiles
//             0..i:      S = Q_i K_j^T, dP = dO_i V_j^T, dS = P o (dP - delta),
//             dQ_i += dS K_j                                     (accumulator in TMEM)
//   DKV mode: a CTA owns one 128-row KV tile of one (sequence, KV head) and walks the query
//             tiles i >= j of the G query heads of that KV head, one after the other:
//             S^T = K_j Q_i^T, dP^T = V_j dO_i^T, dV_j += P^T dO_i, dK_j += dS^T Q_i
// with P = exp2(S c - lse log2 e) from the forward's log-sum-exp and delta = rowsum(dO o O)
// (a small kernel of its own).  All five products run on tcgen05: the two score products with
// both operands in shared memory (TMA, 128B swizzle), the gradient products with the bf16
// weights P / dS read from TMEM, written there in place of the fp32 scores they came from.
// One TMA warp, one MMA-issuing warp, and sixteen element-wise warps.  A step's 128 streamed rows
// are handled as two halves of 64: the eight warps of half h (two threads per tile row, 32
// columns each) turn the half's score columns into weights while the tensor pipe runs the
// gradient product of the other half and the score product of the next step, so MMAs and
// element-wise work overlap and the element-wise latency of a half stays short.
// Every wait is bounded and raises TIK_DEV_WAIT_EXPIRED instead of hanging.
#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

enum { BWD_DQ = 0, BWD_DKV = 1 };
// warp 0 TMA, warp 1 MMA (DQ: the score products), warps 2-17 element-wise (four threads per tile
// row), warp 18 DQ: the gradient products
constexpr int BWD_THREADS = 608;
constexpr int BWD_STAGES = 2;

template <int D, int MODE>
struct BwdSmem {
    static constexpr uint32_t ATOM = 128 * 128;           // 128 rows x 64 bf16
    static constexpr uint32_t TILE = (D / 64) * ATOM;
    static constexpr uint32_t OFF_R = 0;                  // two resident row-side tiles
    // streamed tiles.  DKV: BWD_STAGES stages of (Q_i, dO_i).  DQ: three K stages, then two V
    // stages (a V tile is done with after its dP product, a K tile only after the gradient product).
    static constexpr uint32_t OFF_C = 2 * TILE;
    static constexpr uint32_t N_STREAM = (MODE == 0) ? 5 : 2 * BWD_STAGES;
    static constexpr uint32_t OFF_BAR = OFF_C + N_STREAM * TILE;
    static constexpr uint32_t OFF_SC = OFF_BAR + 160;     // DKV: [half][buffer][-l2 x 64 | -delta x 64] floats of the columns
    static constexpr uint32_t BYTES = OFF_SC + ((MODE == 0) ? 0 : 2 * 2 * 2 * 64 * 4);
    static constexpr uint32_t ALLOC = BYTES + 1024;       // slack to align the base to 1 KiB
};
constexpr int DQ_KSTAGES = 3, DQ_VSTAGES = 2;

template <int D, int MODE>
__global__ void __launch_bounds__(BWD_THREADS, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO,
                const BwdParams p) {
    using L = BwdSmem<D, MODE>;
    constexpr int NATOM = D / 64;
    constexpr uint32_t TMEM_COLS = 512;
    // TMEM columns.  DKV: two score tiles (weights in place), two accumulators.  DQ: the score tile
    // S, two dP tiles used alternately (dS in place), one accumulator.
    constexpr uint32_t COL_T1 = 0, COL_T2 = 128;
    constexpr uint32_t COL_T2B = 256;                                   // DQ only
    constexpr uint32_t COL_A1 = (MODE == BWD_DQ) ? 384 : 256, COL_A2 = 256 + D;
    constexpr uint32_t IDESC_SC = mma_idesc_bf16(128, 64, false);       // one half: 64 streamed rows
    constexpr uint32_t IDESC_SC128 = mma_idesc_bf16(128, 128, false);   // DQ: all 128 streamed rows at once
    constexpr uint32_t IDESC_OUT = mma_idesc_bf16(128, D, true);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---------------------------------------------------------------- work item
    const int seq = blockIdx.z;
    const int tok0 = p.cu_seqlens[seq];
    const int len = p.cu_seqlens[seq + 1] - tok0;
    if (len <= 0) return;
    const int nq = (len + 127) / 128;                      // tiles of the sequence (query and KV alike)
    int own, head = 0, kvh, n_steps;
    if (MODE == BWD_DQ) {
        own = gridDim.x - 1 - blockIdx.x;                  // query tile, heaviest first
        if (own >= nq) return;
        head = blockIdx.y;
        kvh = head / p.G;
        n_steps = own + 1;                                 // KV tiles 0..own
    } else {
        own = blockIdx.x;                                  // KV tile, heaviest first
        if (own >= nq) return;
        kvh = blockIdx.y;
        n_steps = p.G * (nq - own);                        // (g, query tile i >= own), g outermost
    }
    // step t -> the streamed tile and (DKV) the query head
    auto step_tile = [&](int t) { return MODE == BWD_DQ ? t : own + t % (nq - own); };
    auto step_head = [&](int t) { return MODE == BWD_DQ ? head : kvh * p.G + t / (nq - own); };

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw_addr + pad;
    const uint32_t sR1 = sbase + L::OFF_R, sR2 = sR1 + L::TILE;
    const uint32_t bar0 = sbase + L::OFF_BAR;
    const uint32_t bar_r = bar0;                 // row-side tiles landed
    const uint32_t bar_cfull = bar0 + 8;         // [3] streamed tiles landed (DQ: K tiles)
    const uint32_t bar_cempty = bar0 + 32;       // [3] gradient MMAs that read the stage are done
    const uint32_t bar_vfull = bar0 + 56;        // [2] DQ: V tile landed
    const uint32_t bar_vempty = bar0 + 72;       // [2] DQ: the dP product that read the V stage is done
    const uint32_t bar_tfull = bar0 + 88;        // [2] score MMAs of a half-step done (DQ: [0] of a step,
                                                 //     [1] "score tile S is in registers", 16 warps)
    const uint32_t bar_efull = bar0 + 104;       // [2] weights of a half-step written to TMEM (8 warps; DQ:
                                                 //     [0] dS of a step written, 16 warps)
    const uint32_t bar_acc = bar0 + 120;         // all MMAs done
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_BAR + 128);
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 132);
    const uint32_t bar_gdone = bar0 + 136;       // [2] DQ: the gradient product that read a dS tile is done
    float* sc_base = reinterpret_cast<float*>(smem + L::OFF_SC);

    if (tid == 0) {
        mbar_init(bar_r, 1);
        for (int i = 0; i < 3; ++i) {
            mbar_init(bar_cfull + 8 * i, 1);
            mbar_init(bar_cempty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_vfull + 8 * i, 1);
            mbar_init(bar_vempty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_tfull + 8 * i, (MODE == BWD_DQ && i == 1) ? 16 : 1);
            mbar_init(bar_efull + 8 * i, MODE == BWD_DQ ? 16 : 8);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_gdone, 1);
        mbar_init(bar_gdone + 8, 1);
        *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmDO);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int row_own = tok0 + 128 * own;
            mbar_expect_tx(bar_r, 2 * L::TILE);
            for (int a = 0; a < NATOM; ++a) {
                if (MODE == BWD_DQ) {
                    tma_load_3d(sR1 + a * L::ATOM, &tmQ, bar_r, a * 64, head, row_own);
                    tma_load_3d(sR2 + a * L::ATOM, &tmDO, bar_r, a * 64, head, row_own);
                } else {
                    tma_load_3d(sR1 + a * L::ATOM, &tmK, bar_r, a * 64, kvh, row_own);
                    tma_load_3d(sR2 + a * L::ATOM, &tmV, bar_r, a * 64, kvh, row_own);
                }
            }
            if (MODE == BWD_DQ) {
                for (int t = 0; t < n_steps; ++t) {
                    if (*abort_word) break;          // a wait expired somewhere: stop issuing copies
                    const int row = tok0 + 128 * t;
                    const int ks = t % DQ_KSTAGES, vs = t % DQ_VSTAGES;
                    const uint32_t kuse = t / DQ_KSTAGES, vuse = t / DQ_VSTAGES;
                    if (kuse > 0) mbar_wait(bar_cempty + 8 * ks, (kuse - 1) & 1, abort_word, p.dev_status);
                    mbar_expect_tx(bar_cfull + 8 * ks, L::TILE);
                    for (int a = 0; a < NATOM; ++a)
                        tma_load_3d(sbase + L::OFF_C + ks * L::TILE + a * L::ATOM, &tmK, bar_cfull + 8 * ks, a * 64, kvh, row);
                    if (vuse > 0) mbar_wait(bar_vempty + 8 * vs, (vuse - 1) & 1, abort_word, p.dev_status);
                    mbar_expect_tx(bar_vfull + 8 * vs, L::TILE);
                    for (int a = 0; a < NATOM; ++a)
                        tma_load_3d(sbase + L::OFF_C + (DQ_KSTAGES + vs) * L::TILE + a * L::ATOM, &tmV, bar_vfull + 8 * vs,
                                    a * 64, kvh, row);
                }
            } else
            for (int t = 0; t < n_steps; ++t) {
                if (*abort_word) break;          // a wait expired somewhere: stop issuing copies
                const int st = t % BWD_STAGES;
                const uint32_t use = t / BWD_STAGES;
                if (use > 0) mbar_wait(bar_cempty + 8 * st, (use - 1) & 1, abort_word, p.dev_status);
                const uint32_t c1 = sbase + L::OFF_C + st * 2 * L::TILE, c2 = c1 + L::TILE;
                const uint32_t full = bar_cfull + 8 * st;
                const int row = tok0 + 128 * step_tile(t);
                const int h = step_head(t);
                mbar_expect_tx(full, 2 * L::TILE);
                for (int a = 0; a < NATOM; ++a) {
                    if (MODE == BWD_DQ) {
                        tma_load_3d(c1 + a * L::ATOM, &tmK, full, a * 64, kvh, row);
                        tma_load_3d(c2 + a * L::ATOM, &tmV, full, a * 64, kvh, row);
                    } else {
                        tma_load_3d(c1 + a * L::ATOM, &tmQ, full, a * 64, h, row);
                        tma_load_3d(c2 + a * L::ATOM, &tmDO, full, a * 64, h, row);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // MMAs issued by one thread execute in order: the score MMAs of half h of step t+1 overwrite
        // the columns that hold the weights of half h of step t only after the gradient MMAs that
        // read them.  Issue order per step: gradient(a,t), score(a,t+1), gradient(b,t), score(b,t+1).
        if (lane == 0) {
            mbar_wait(bar_r, 0, abort_word, p.dev_status);
            const uint64_t dr1 = smem_desc_sw128(sR1, 0, 1024), dr2 = smem_desc_sw128(sR2, 0, 1024);
            auto stage_c1 = [&](int t) { return sbase + L::OFF_C + (t % BWD_STAGES) * 2 * L::TILE; };
            auto score = [&](int t, int h) {      // T1h = R1 C1h^T, T2h = R2 C2h^T (64 streamed rows = 8 KiB)
                const uint32_t c1 = stage_c1(t) + h * 8192, c2 = c1 + L::TILE;
                if (D == 128) {
                    mma_ss_chain8_fresh(tmem + COL_T1 + 64 * h, dr1, smem_desc_sw128(c1, 0, 1024), IDESC_SC);
                    mma_ss_chain8_fresh(tmem + COL_T2 + 64 * h, dr2, smem_desc_sw128(c2, 0, 1024), IDESC_SC);
                } else {
                    mma_ss_chain4_fresh(tmem + COL_T1 + 64 * h, dr1, smem_desc_sw128(c1, 0, 1024), IDESC_SC);
                    mma_ss_chain4_fresh(tmem + COL_T2 + 64 * h, dr2, smem_desc_sw128(c2, 0, 1024), IDESC_SC);
                }
                mma_commit(bar_tfull + 8 * h);
            };
            auto gradient = [&](int t, int h) {   // A = bf16 weights of half h in TMEM, B = its 64 streamed rows
                const uint32_t c1 = stage_c1(t) + h * 8192, c2 = c1 + L::TILE;
                const uint32_t acc = (t > 0 || h > 0) ? 1u : 0u;
                mma_ts_chain4(tmem + COL_A1, tmem + COL_T2 + 64 * h, smem_desc_sw128(c1, L::ATOM, 1024), IDESC_OUT, acc);
                if (MODE == BWD_DKV)
                    mma_ts_chain4(tmem + COL_A2, tmem + COL_T1 + 64 * h, smem_desc_sw128(c2, L::ATOM, 1024), IDESC_OUT,
                                  acc);
            };
            if (MODE == BWD_DQ) {
                // DQ: only dS feeds a gradient product, so the score tile S is free again as soon as
                // the element-wise threads hold it in registers, and dP / dS alternate between two
                // tiles.  Both score products of step t+1 (128 streamed rows each, which an SS-form
                // MMA reads at the full rate; 64-row halves are bound by shared-memory bandwidth) are
                // issued while the element-wise work of step t runs, the gradient product of step t
                // right behind them.
                auto stage_k = [&](int t) { return sbase + L::OFF_C + (t % DQ_KSTAGES) * L::TILE; };
                auto score_full = [&](int t) {
                    const uint32_t c1 = stage_k(t), c2 = sbase + L::OFF_C + (DQ_KSTAGES + t % DQ_VSTAGES) * L::TILE;
                    const uint32_t t2 = tmem + ((t & 1) ? COL_T2B : COL_T2);
                    mbar_wait(bar_cfull + 8 * (t % DQ_KSTAGES), (t / DQ_KSTAGES) & 1, abort_word, p.dev_status);
                    mbar_wait(bar_vfull + 8 * (t % DQ_VSTAGES), (t / DQ_VSTAGES) & 1, abort_word, p.dev_status);
                    if (t > 0) mbar_wait(bar_tfull + 8, (t - 1) & 1, abort_word, p.dev_status);   // S of step t-1 is in registers
                    // the dP tile of this parity held dS of step t-2 (the two issuing threads have no
                    // common program order, so its gradient product is waited for)
                    if (t > 1) mbar_wait(bar_gdone + 8 * (t & 1), ((t - 2) >> 1) & 1, abort_word, p.dev_status);
                    tc_fence_after();
                    if (D == 128) {
                        mma_ss_chain8_fresh(tmem + COL_T1, dr1, smem_desc_sw128(c1, 0, 1024), IDESC_SC128);
                        mma_ss_chain8_fresh(t2, dr2, smem_desc_sw128(c2, 0, 1024), IDESC_SC128);
                    } else {
                        mma_ss_chain4_fresh(tmem + COL_T1, dr1, smem_desc_sw128(c1, 0, 1024), IDESC_SC128);
                        mma_ss_chain4_fresh(t2, dr2, smem_desc_sw128(c2, 0, 1024), IDESC_SC128);
                    }
                    mma_commit(bar_tfull);
                    mma_commit(bar_vempty + 8 * (t % DQ_VSTAGES));      // the V stage is done with
                };
                for (int t = 0; t < n_steps; ++t) {
                    if (*abort_word) break;
                    score_full(t);
                }
            } else {
            mbar_wait(bar_cfull, 0, abort_word, p.dev_status);
            tc_fence_after();
            score(0, 0);
            score(0, 1);
            for (int t = 0; t < n_steps; ++t) {
                if (*abort_word) break;
                const bool more = t + 1 < n_steps;
                if (more) mbar_wait(bar_cfull + 8 * ((t + 1) % BWD_STAGES), ((t + 1) / BWD_STAGES) & 1, abort_word,
                                    p.dev_status);
                for (int h = 0; h < 2; ++h) {
                    mbar_wait(bar_efull + 8 * h, t & 1, abort_word, p.dev_status);
                    tc_fence_after();
                    gradient(t, h);
                    if (h == 1) mma_commit(bar_cempty + 8 * (t % BWD_STAGES));     // stage of step t consumed
                    if (more) score(t + 1, h);
                }
            }
            mma_commit(bar_acc);
            }
        }
        __syncwarp();
    } else if (warp == 18) {
        // ------------------------------------------------------------ DQ: gradient-product issuer
        // A thread of its own, so that its waits and commits do not stand between two score
        // products in the other issuing thread.
        if (MODE == BWD_DQ && lane == 0) {
            for (int t = 0; t < n_steps; ++t) {
                if (*abort_word) break;
                mbar_wait(bar_efull, t & 1, abort_word, p.dev_status);
                tc_fence_after();
                // A = dS: every thread left its 32 columns' bf16 pairs in the first 16 columns of
                // its own 32-column block, so the eight 16-key steps sit at 0, 8, 32, 40, ...
                mma_ts_chain8_blocks(tmem + COL_A1, tmem + ((t & 1) ? COL_T2B : COL_T2),
                                     smem_desc_sw128(sbase + L::OFF_C + (t % DQ_KSTAGES) * L::TILE, L::ATOM, 1024),
                                     IDESC_OUT, t > 0 ? 1u : 0u);
                mma_commit(bar_cempty + 8 * (t % DQ_KSTAGES));
                mma_commit(bar_gdone + 8 * (t & 1));
            }
            mma_commit(bar_acc);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ element-wise warps
        const int quarter = warp & 3;                      // TMEM lane quarter of this warp
        const int r = quarter * 32 + lane;                 // tile row == TMEM lane
        const int hlf = (warp - 2) >> 3;                   // which half (64 streamed rows) this thread works on
        const int sub = ((warp - 2) >> 2) & 1;             // which 32 of the half's 64 columns
        const int et = ((warp - 2) & 7) * 32 + lane;       // 0..255 within the half's eight warps
        const uint32_t tlane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int row_abs = 128 * own + r;                 // position of this row in the sequence
        const float c = p.c;                               // scale * log2(e)
        float row_l2 = 0.0f, row_dl = 0.0f;
        if (MODE == BWD_DQ && row_abs < len) {
            const long long idx = (static_cast<long long>(tok0) + row_abs) * p.Hq + head;
            row_l2 = __fmul_rn(p.lse[idx], LOG2E_F);
            row_dl = p.delta[idx];
        }
        // DKV: the scalars belong to the columns (query rows of the streamed tile).  Thread `et` < 64
        // of warpgroup h fetches those of column 64 h + et one step ahead; they reach the other
        // threads of the warpgroup through shared memory (double-buffered, one named barrier per step).
        // (stored negated and as two arrays, so that two neighbouring columns' values load as one
        // 8-byte pair, ready for the two-wide arithmetic)
        float* my_sc = sc_base + hlf * (2 * 2 * 64);          // [buffer][-l2 x 64 | -delta x 64]
        auto fetch_col = [&](int t, float& l2, float& dl) {
            l2 = 0.0f;
            dl = 0.0f;
            if (t < n_steps && et < 64) {
                const int qa = 128 * step_tile(t) + 64 * hlf + et;
                if (qa < len) {
                    const long long idx = (static_cast<long long>(tok0) + qa) * p.Hq + step_head(t);
                    l2 = __fmul_rn(p.lse[idx], LOG2E_F);
                    dl = p.delta[idx];
                }
            }
        };
        if (MODE == BWD_DKV) {
            float l2, dl;
            fetch_col(0, l2, dl);
            if (et < 64) {
                my_sc[et] = -l2;
                my_sc[64 + et] = -dl;
            }
            named_bar_sync(1 + hlf, 256);
        }
        if (MODE == BWD_DQ) {
            // DQ: all sixteen warps work on the same step, four threads per row with 32 columns each
            const int cq = 2 * hlf + sub;
            const float nl2 = -row_l2, ndl = -row_dl;
            for (int t = 0; t < n_steps; ++t) {
                mbar_wait(bar_tfull, t & 1, abort_word, p.dev_status);
                tc_fence_after();
                const uint32_t t2 = tlane + ((t & 1) ? COL_T2B : COL_T2) + 32 * cq;
                uint32_t s_[32], d_[32];
                tmem_ld32(tlane + COL_T1 + 32 * cq, s_);
                tmem_ld32(t2, d_);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tfull + 8);      // S is in registers: the next QK^T may overwrite it
                uint32_t dk_[16];
                if (t != own) {               // off the diagonal nothing is masked: two-wide, no compares
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float p0, p1, ds0, ds1;
                        bwd_pds_x2(__uint_as_float(s_[i]), __uint_as_float(s_[i + 1]), __uint_as_float(d_[i]),
                                   __uint_as_float(d_[i + 1]), c, nl2, nl2, ndl, ndl, p0, p1, ds0, ds1);
                        dk_[i >> 1] = pack_bf16x2(ds0, ds1);
                    }
                } else {
                    const int col0_abs = 128 * t + 32 * cq;
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float dsv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const bool masked = col0_abs + i + e > row_abs;      // key after query
                            const float pe = bwd_p(__uint_as_float(s_[i + e]), c, row_l2);
                            dsv[e] = masked ? 0.0f : bwd_ds(pe, __uint_as_float(d_[i + e]), row_dl);
                        }
                        dk_[i >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                    }
                }
                // dS goes over the first 16 of this thread's own 32 dP columns: no other thread reads them
                tmem_st16(t2, dk_);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_efull);
            }
        } else
        for (int t = 0; t < n_steps; ++t) {
            float nl2 = 0.0f, ndl = 0.0f;
            if (MODE == BWD_DKV) fetch_col(t + 1, nl2, ndl);            // in flight during this step
            const float* csc = my_sc + (t & 1) * 128 + 32 * sub;       // -l2 of this thread's 32 columns; -delta at + 64
            mbar_wait(bar_tfull + 8 * hlf, t & 1, abort_word, p.dev_status);
            tc_fence_after();
            // column cc of the half is masked for this row when it lies in the row's future (DQ: key
            // after query; DKV: query before key) or, DKV, past the end of the sequence
            const int col0_abs = 128 * step_tile(t) + 64 * hlf + 32 * sub;
            {
                uint32_t s_[32], d_[32];
                tmem_ld32(tlane + COL_T1 + 64 * hlf + 32 * sub, s_);
                tmem_ld32(tlane + COL_T2 + 64 * hlf + 32 * sub, d_);
                tmem_wait_ld();
                // the weights go in place of the half's scores: its first 32 columns, which the
                // threads of sub-block 0 are reading until they have passed this barrier
                named_bar_sync(3 + hlf, 256);
                uint32_t pk[16], dk_[16];
                // only the diagonal tile and (DKV) the sequence's last query tile have masked columns;
                // everywhere else the two-wide path runs without compares and selects
                const bool any_mask = (step_tile(t) == own) || (MODE == BWD_DKV && col0_abs + 32 > len);
                if (!any_mask) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float nl2_0, nl2_1, ndl0, ndl1;
                        if (MODE == BWD_DQ) {
                            nl2_0 = nl2_1 = -row_l2;
                            ndl0 = ndl1 = -row_dl;
                        } else {
                            const float2 nl = *reinterpret_cast<const float2*>(&csc[i]);
                            const float2 nd = *reinterpret_cast<const float2*>(&csc[64 + i]);
                            nl2_0 = nl.x, nl2_1 = nl.y, ndl0 = nd.x, ndl1 = nd.y;
                        }
                        float p0, p1, ds0, ds1;
                        bwd_pds_x2(__uint_as_float(s_[i]), __uint_as_float(s_[i + 1]), __uint_as_float(d_[i]),
                                   __uint_as_float(d_[i + 1]), c, nl2_0, nl2_1, ndl0, ndl1, p0, p1, ds0, ds1);
                        pk[i >> 1] = pack_bf16x2(p0, p1);
                        dk_[i >> 1] = pack_bf16x2(ds0, ds1);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float pv[2], dsv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int cc = i + e;
                            const int col_abs = col0_abs + cc;
                            bool masked;
                            float l2, dl;
                            if (MODE == BWD_DQ) {
                                masked = col_abs > row_abs;
                                l2 = row_l2;
                                dl = row_dl;
                            } else {
                                masked = (row_abs > col_abs) || (col_abs >= len);
                                l2 = -csc[cc];
                                dl = -csc[64 + cc];
                            }
                            const float pe = bwd_p(__uint_as_float(s_[i + e]), c, l2);
                            pv[e] = masked ? 0.0f : pe;
                            dsv[e] = masked ? 0.0f : bwd_ds(pe, __uint_as_float(d_[i + e]), dl);
                        }
                        pk[i >> 1] = pack_bf16x2(pv[0], pv[1]);
                        dk_[i >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                    }
                }
                if (MODE == BWD_DKV) tmem_st16(tlane + COL_T1 + 64 * hlf + 16 * sub, pk);
                tmem_st16(tlane + COL_T2 + 64 * hlf + 16 * sub, dk_);
            }
            tmem_wait_st();
            if (MODE == BWD_DKV) {
                // hand the next step's column scalars over (the buffer was last read a step ago, before
                // the previous barrier)
                if (et < 64) {
                    my_sc[((t + 1) & 1) * 128 + et] = -nl2;
                    my_sc[((t + 1) & 1) * 128 + 64 + et] = -ndl;
                }
                named_bar_sync(1 + hlf, 256);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_efull + 8 * hlf);
        }
        // ---- epilogue: fp32 accumulators -> bf16 rows
        mbar_wait(bar_acc, 0, abort_word, p.dev_status);
        tc_fence_after();
        const bool valid = row_abs < len && sub == 0;     // one thread per (row, column half) stores
        const long long tok = static_cast<long long>(tok0) + row_abs;
        __nv_bfloat16* out1 = (MODE == BWD_DQ) ? p.dq + (tok * p.Hq + head) * D : p.dk + (tok * p.Hkv + kvh) * D;
        __nv_bfloat16* out2 = p.dv + (tok * p.Hkv + kvh) * D;
#pragma unroll 1
        for (int which = 0; which < (MODE == BWD_DKV ? 2 : 1); ++which) {
            const uint32_t col = which ? COL_A2 : COL_A1;
            __nv_bfloat16* out = which ? out2 : out1;
            const float osc = which ? 1.0f : p.scale;          // dQ, dK carry the softmax scale; dV does not
#pragma unroll
            for (int cc = hlf * (D / 64); cc < (hlf + 1) * (D / 64); ++cc) {
                uint32_t v[32];
                tmem_ld32(tlane + col + 32 * cc, v);
                tmem_wait_ld();
                if (valid) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        reinterpret_cast<uint4*>(out + 32 * cc)[i] = make_uint4(
                            pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * i]), osc), __fmul_rn(__uint_as_float(v[8 * i + 1]), osc)),
                            pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * i + 2]), osc), __fmul_rn(__uint_as_float(v[8 * i + 3]), osc)),
                            pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * i + 4]), osc), __fmul_rn(__uint_as_float(v[8 * i + 5]), osc)),
                            pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * i + 6]), osc), __fmul_rn(__uint_as_float(v[8 * i + 7]), osc)));
                }
            }
        }
    }

    if (*abort_word) {   // let copies and MMAs in flight finish before shared memory and TMEM are released
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 1000000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

// delta[token][head] = sum_c dO * O in fp32: one warp per (token, head), lane chain then butterfly.
template <int D>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __nv_bfloat16* __restrict__ o,
                                                       const __nv_bfloat16* __restrict__ dout,
                                                       float* __restrict__ delta, long long n_vec) {
    const long long v = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (v >= n_vec) return;
    constexpr int EPL = D / 32;                             // elements per lane (4 or 2)
    const __nv_bfloat16* op = o + v * D + EPL * lane;
    const __nv_bfloat16* dp = dout + v * D + EPL * lane;
    float part = 0.0f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) part = __fmaf_rn(__bfloat162float(dp[e]), __bfloat162float(op[e]), part);
    part = hn_warp_total(part);
    if (lane == 0) delta[v] = part;
}

template <int D, int MODE>
static cudaError_t launch_bwd_t(dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                const CUtensorMap& tmDO, const BwdParams& p, cudaStream_t stream) {
    auto kern = attn_bwd_kernel<D, MODE>;
    static DeviceOnce configured;     // the opt-in belongs to the (function, device) pair
    {
        cudaError_t e = configured.run([&]() {
            return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(BwdSmem<D, MODE>::ALLOC));
        });
        if (e != cudaSuccess) return e;
    }
    count_launch();
    kern<<<grid, BWD_THREADS, BwdSmem<D, MODE>::ALLOC, stream>>>(tmQ, tmK, tmV, tmDO, p);
    return cudaGetLastError();
}

cudaError_t launch_attn_bwd(int d, int max_tiles, int S, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                            const CUtensorMap& tmV, const CUtensorMap& tmDO, const BwdParams& p,
                            const void* o, const void* dout, long long n_vec, cudaStream_t stream) {
    const unsigned dgrid = static_cast<unsigned>((n_vec * 32 + 255) / 256);
    count_launch();  // exactly one of the launches below runs
    if (d == 128)
        bwd_delta_kernel<128><<<dgrid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(o),
                                                         static_cast<const __nv_bfloat16*>(dout), p.delta, n_vec);
    else
        bwd_delta_kernel<64><<<dgrid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(o),
                                                        static_cast<const __nv_bfloat16*>(dout), p.delta, n_vec);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const dim3 gq(max_tiles, p.Hq, S), gkv(max_tiles, p.Hkv, S);
    if (d == 128) {
        e = launch_bwd_t<128, BWD_DKV>(gkv, tmQ, tmK, tmV, tmDO, p, stream);
        if (e == cudaSuccess) e = launch_bwd_t<128, BWD_DQ>(gq, tmQ, tmK, tmV, tmDO, p, stream);
    } else {
        e = launch_bwd_t<64, BWD_DKV>(gkv, tmQ, tmK, tmV, tmDO, p, stream);
        if (e == cudaSuccess) e = launch_bwd_t<64, BWD_DQ>(gq, tmQ, tmK, tmV, tmDO, p, stream);
    }
    return e;
}

}  // namespace tik
