// Dense linear layer y = x W^T (bf16 in, fp32 accumulation in TMEM, bf16 out) for sm_100a: the
// FFN projections of the unified operator set.  Same machinery as the log-probability GEMM: one
// CTA = (128-row tile, super-chunk of 256 to 4096 output columns); a TMA warp streams 64-wide K slices of x and W
// through a four-stage shared-memory ring, an MMA warp accumulates the whole K range in ascending
// order into one of two 256-column TMEM accumulators (M128 x N256 x K16, no split-K), and four
// epilogue warps (one thread per row) round the accumulator to bf16 and send it out through
// shared memory and tiled TMA stores while the next 256 columns are being accumulated.  An output element is one fixed chain of MMAs over K, so it
// depends on its x row and its W row only: a row gives the same bits whether it is computed alone
// (decode) or inside a long batch (prefill, policy update).
#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

namespace lin {
constexpr int NB = 256;                      // output columns per MMA
constexpr uint32_t A_BYTES = 128 * 128;      // 128 rows x 64 bf16
constexpr uint32_t STG_BYTES = 128 * 128;    // output staging: 128 rows x 64 bf16, two buffers
constexpr int BAND = 32;                     // row tiles per L2 band (even: CTA pairs stay inside a band)
constexpr int THREADS = 192;                 // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
// PAIR: two CTAs on neighbouring SMs share every MMA (M = 256 rows); each stages its own 128 rows of
// x and 128 of the 256 weight rows of a step, as in the log-probability kernel.
template <bool PAIR>
struct Cfg {
    static constexpr int STAGES = PAIR ? 6 : 4;
    static constexpr uint32_t B_BYTES = (PAIR ? NB / 2 : NB) * 128;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr uint32_t OFF_STG = STAGES * STAGE_BYTES;
    static constexpr uint32_t OFF_BAR = OFF_STG + 2 * STG_BYTES;
    static constexpr uint32_t BYTES = OFF_BAR + 256;
    static constexpr uint32_t ALLOC = BYTES + 1024;
};
}  // namespace lin

template <bool PAIR>
__global__ void __launch_bounds__(lin::THREADS, 1)
linear_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmY, const LinearParams p) {
    using namespace lin;
    using C = Cfg<PAIR>;
    constexpr int STAGES = C::STAGES;
    constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES, OFF_STG = C::OFF_STG, OFF_BAR = C::OFF_BAR;
    constexpr uint32_t TMEM_COLS = 512;      // two 256-column accumulators
    constexpr uint32_t IDESC = mma_idesc_bf16(PAIR ? 256 : 128, NB, false);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;     // 0 = the CTA that issues the pair's MMAs

    // raster: bands of BAND row tiles; within a band the row tile varies fastest so the CTAs in
    // flight share one super-chunk of W in L2 and W is streamed from HBM once per band
    const int ntile = static_cast<int>((p.T + 127) / 128);
    const long long per_band = static_cast<long long>(BAND) * p.nsuper;
    const int band = static_cast<int>(blockIdx.x / per_band);
    const int band_tiles = min(BAND, ntile - band * BAND);
    const long long rem = blockIdx.x - band * per_band;
    const int sup = static_cast<int>(rem / BAND);
    const int tile_in_band = static_cast<int>(rem % BAND);
    // unit mode (up to 16 row tiles, CTA pairs only): one persistent pair per two SMs walks the
    // units q = pair index, + number of pairs, ...; unit q = (256-column step q / ntp, pair of row
    // tiles q % ntp): the pairs running at one time share a few steps of W in L2, and x (at most
    // 2048 rows) stays there throughout.  Same MMA chain per element.
    const bool unit_mode = PAIR && p.unit_mode != 0;
    const int u_first = static_cast<int>(blockIdx.x >> 1), u_stride = static_cast<int>(gridDim.x >> 1);
    if (!unit_mode && (PAIR ? (tile_in_band & ~1) : tile_in_band) >= band_tiles) return;   // a pair leaves only together
    const int row_fixed = (band * BAND + tile_in_band) * 128;
    const int col_base = sup * p.super_cols;
    const int ntp = unit_mode ? p.ntp : 1;
    auto row_of = [&](int nt) {
        return unit_mode ? (2 * ((u_first + nt * u_stride) % ntp) + static_cast<int>(rank)) * 128 : row_fixed;
    };
    auto col_of = [&](int nt) { return unit_mode ? ((u_first + nt * u_stride) / ntp) * NB : col_base + nt * NB; };
    const int n_nt = unit_mode ? (p.nunit - u_first + u_stride - 1) / u_stride
                               : min(p.super_cols / NB, (p.N - col_base + NB - 1) / NB);   // 256-column steps
    const int n_kb = p.K / 64;

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
            mbar_init(bar_acc_empty + 8 * b, PAIR ? 256 : 128);
        }
        *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmY);
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
    const uint32_t lead_full = PAIR ? mapa_cluster(bar_full, 0) : bar_full;
    const uint32_t lead_acc_empty = PAIR ? mapa_cluster(bar_acc_empty, 0) : bar_acc_empty;
    const uint32_t peer_empty = PAIR ? mapa_cluster(bar_empty, 1) : bar_empty;
    const uint32_t peer_acc_full = PAIR ? mapa_cluster(bar_acc_full, 1) : bar_acc_full;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int nt = 0; nt < n_nt; ++nt) {
                const int col0 = col_of(nt), row0 = row_of(nt);
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    if (*abort_word) break;      // a wait expired somewhere: stop issuing copies
                    const int s = it % STAGES;
                    const uint32_t use = it / STAGES;
                    if (use > 0) mbar_wait(bar_empty + 8 * s, (use - 1) & 1, abort_word, p.dev_status);
                    // rows past T and W rows past N are outside the tensor maps and arrive as zeros
                    if (PAIR) {
                        if (rank == 0) mbar_expect_tx(bar_full + 8 * s, 2 * STAGE_BYTES);   // both CTAs' bytes
                        tma_load_2d_pair(sbase + s * STAGE_BYTES, &tmA, lead_full + 8 * s, kb * 64, row0);
                        tma_load_2d_pair(sbase + s * STAGE_BYTES + A_BYTES, &tmB, lead_full + 8 * s, kb * 64,
                                         col0 + 128 * static_cast<int>(rank));
                    } else {
                        mbar_expect_tx(bar_full + 8 * s, STAGE_BYTES);
                        tma_load_2d(sbase + s * STAGE_BYTES, &tmA, bar_full + 8 * s, kb * 64, row0);
                        tma_load_2d(sbase + s * STAGE_BYTES + A_BYTES, &tmB, bar_full + 8 * s, kb * 64, col0);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            uint32_t it = 0;
            for (int nt = 0; nt < n_nt; ++nt) {
                const int buf = nt & 1;
                const uint32_t use = nt >> 1;
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
                        mma_commit_pair(bar_empty + 8 * s);
                        mma_commit_pair(peer_empty + 8 * s);
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
        // Thread per row: 64 columns at a time go from TMEM to a 128B-swizzled staging tile in
        // shared memory and leave as one tiled TMA store of 128 rows x 128 bytes (row-by-row
        // 16-byte stores from 128 threads cost a third of the kernel on wide outputs).  The store
        // clips at the tensor's bounds, so rows past T and columns past N need no guard.  Two
        // staging tiles alternate; the issuing thread lets at most one store group read behind it.
        const int quarter = warp & 3;                      // TMEM lane quarter of this warp
        const int row = quarter * 32 + lane;
        uint32_t piece = 0;
        for (int nt = 0; nt < n_nt; ++nt) {
            const int buf = nt & 1;
            mbar_wait(bar_acc_full + 8 * buf, (nt >> 1) & 1, abort_word, p.dev_status);
            tc_fence_after();
            const int col0 = col_of(nt), row0 = row_of(nt);
            const uint32_t taddr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * NB;
#pragma unroll 1
            for (int q = 0; q < NB / 64; ++q, ++piece) {
                if (col0 + 64 * q >= p.N) break;               // uniform: columns past N
                uint32_t v[64];
                tmem_ld32(taddr + 64 * q, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld32(taddr + 64 * q + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_wait_ld();
                uint8_t* stg = smem + OFF_STG + (piece & 1) * STG_BYTES;
                // the store that last read this staging tile (two pieces ago) has finished reading
                if (warp == 2 && lane == 0) tma_store_wait_read1();
                named_bar_sync(1, 128);
#pragma unroll
                for (int c16 = 0; c16 < 8; ++c16) {
                    const uint4 val = make_uint4(
                        pack_bf16x2(__uint_as_float(v[8 * c16]), __uint_as_float(v[8 * c16 + 1])),
                        pack_bf16x2(__uint_as_float(v[8 * c16 + 2]), __uint_as_float(v[8 * c16 + 3])),
                        pack_bf16x2(__uint_as_float(v[8 * c16 + 4]), __uint_as_float(v[8 * c16 + 5])),
                        pack_bf16x2(__uint_as_float(v[8 * c16 + 6]), __uint_as_float(v[8 * c16 + 7])));
                    *reinterpret_cast<uint4*>(stg + row * 128 + ((c16 ^ (row & 7)) << 4)) = val;
                }
                fence_proxy_async_smem();
                named_bar_sync(1, 128);
                if (warp == 2 && lane == 0) {
                    tma_store_2d(&tmY, smem_u32(stg), col0 + 64 * q, row0);
                    tma_store_commit();
                }
            }
            // all TMEM reads of this accumulator are done: hand it back to the MMA warp
            tc_fence_before();
            if (PAIR) mbar_arrive_cluster(lead_acc_empty + 8 * buf);
            else mbar_arrive(bar_acc_empty + 8 * buf);
        }
        if (warp == 2 && lane == 0) tma_store_wait_read();     // shared memory stays valid until the last read
    }

    if (*abort_word) {   // let copies and MMAs in flight finish before shared memory and TMEM are released
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

// ---------------------------------------------------------------------------------------------
// Decode-shaped calls (one row tile: T <= 128).  The work is one pass over W at HBM rate, so the
// schedule is built for bytes in flight and even SM load instead of tensor throughput: the grid is
// one persistent CTA per SM walking column units u = blockIdx.x, + gridDim.x, ...; a unit is
// `nu` = 64, 128 or 256 output columns (the host picks the width from a cost model);
// only `a_rows` = 32, 64 or 128 rows of x are staged per K slice (the MMA still spans 128 rows: rows
// past a_rows read whatever the stage holds, their accumulator rows are never stored); the ring
// has as many stages as fit in 192 KiB (3 .. 4) of one, two or four K slices each, and the producer runs ahead into the next unit
// while the epilogue of the last one drains.  An output element is still one chain of K16 MMAs in
// ascending K into one fp32 accumulator, so its bits equal those of the batched kernel.
namespace linu {
constexpr uint32_t RING_BYTES = 192 * 1024;
constexpr int MAX_STAGES = 12;
constexpr uint32_t OFF_STG = RING_BYTES;
constexpr uint32_t OFF_BAR = OFF_STG + 2 * lin::STG_BYTES;
constexpr uint32_t BYTES = OFF_BAR + 512;
constexpr uint32_t ALLOC = BYTES + 1024;
}  // namespace linu

__global__ void __launch_bounds__(lin::THREADS, 1)
linear_unit_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmY, const LinearParams p) {
    using namespace linu;
    constexpr uint32_t TMEM_COLS = 512;      // two accumulators, 256 columns apart
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nu = p.nu;
    const uint32_t a_bytes = static_cast<uint32_t>(p.a_rows) * 128u;
    const uint32_t slice_bytes = a_bytes + static_cast<uint32_t>(nu) * 128u;      // a multiple of 1 KiB
    // K slices per stage: the issuing thread spends ~300 cycles per stage on its barrier wait, fence,
    // descriptors and commit, more than four narrow MMAs run (N = 128: 256 cycles, N = 64: ~190);
    // 256 / nu slices per stage (as long as three stages fit) bring that share down (N = 256 MMAs run
    // 512 cycles per slice and hide it)
    int kps = 256 / nu;
    while (kps > 1 && RING_BYTES / (slice_bytes * static_cast<uint32_t>(kps)) < 3u) kps >>= 1;
    const uint32_t stage_bytes = slice_bytes * static_cast<uint32_t>(kps);
    const int nst = min(MAX_STAGES, static_cast<int>(RING_BYTES / stage_bytes));
    const int n_my = (p.nunit - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const int n_kb = p.K / 64;
    const uint32_t idesc = mma_idesc_bf16(128, nu, false);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw_addr + pad;
    const uint32_t bar_full = sbase + OFF_BAR;                   // MAX_STAGES barriers
    const uint32_t bar_empty = bar_full + 8 * MAX_STAGES;        // MAX_STAGES barriers
    const uint32_t bar_acc_full = bar_empty + 8 * MAX_STAGES;    // 2
    const uint32_t bar_acc_empty = bar_acc_full + 16;            // 2
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 8 * (2 * MAX_STAGES + 4));
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8 * (2 * MAX_STAGES + 4) + 4);

    if (tid == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, 128);
        }
        *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmY);
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
            int s = 0;
            uint32_t use = 0;                    // how often stage s has been filled before
            for (int i = 0; i < n_my; ++i) {
                const int col0 = (static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x)) * nu;
                for (int kb = 0; kb < n_kb; kb += kps) {
                    if (*abort_word) break;
                    if (use > 0) mbar_wait(bar_empty + 8 * s, (use - 1) & 1, abort_word, p.dev_status);
                    const int ns = min(kps, n_kb - kb);
                    mbar_expect_tx(bar_full + 8 * s, slice_bytes * static_cast<uint32_t>(ns));
                    for (int sl = 0; sl < ns; ++sl) {
                        const uint32_t dst = sbase + s * stage_bytes + sl * slice_bytes;
                        tma_load_2d(dst + a_bytes, &tmB, bar_full + 8 * s, (kb + sl) * 64, col0);   // W rows past N: zeros
                        tma_load_2d(dst, &tmA, bar_full + 8 * s, (kb + sl) * 64, 0);                // x rows past T: zeros
                    }
                    if (++s == nst) {
                        s = 0;
                        ++use;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t use = 0;
            for (int i = 0; i < n_my; ++i) {
                const int buf = i & 1;
                const uint32_t acc_use = i >> 1;
                if (acc_use > 0) mbar_wait(bar_acc_empty + 8 * buf, (acc_use - 1) & 1, abort_word, p.dev_status);
                tc_fence_after();
                for (int kb = 0; kb < n_kb; kb += kps) {
                    if (*abort_word) break;
                    mbar_wait(bar_full + 8 * s, use & 1, abort_word, p.dev_status);
                    tc_fence_after();
                    const uint32_t a0 = sbase + s * stage_bytes, b0 = a0 + a_bytes;
                    const int ns = min(kps, n_kb - kb);
                    for (int sl = 0; sl < ns; ++sl)
                        mma_ss_chain4(tmem + buf * 256, smem_desc_sw128(a0 + sl * slice_bytes, 0, 1024),
                                      smem_desc_sw128(b0 + sl * slice_bytes, 0, 1024), idesc, (kb + sl) ? 1u : 0u);
                    mma_commit(bar_empty + 8 * s);
                    if (++s == nst) {
                        s = 0;
                        ++use;
                    }
                }
                mma_commit(bar_acc_full + 8 * buf);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        // As in the batched kernel: a thread per accumulator row, 64 columns at a time through a
        // swizzled staging tile and one tiled TMA store, which clips rows past T and columns past N.
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        uint32_t piece = 0;
        for (int i = 0; i < n_my; ++i) {
            const int buf = i & 1;
            mbar_wait(bar_acc_full + 8 * buf, (i >> 1) & 1, abort_word, p.dev_status);
            tc_fence_after();
            const int col0 = (static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x)) * nu;
            const uint32_t taddr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256;
#pragma unroll 1
            for (int q = 0; q < nu / 64; ++q, ++piece) {
                if (col0 + 64 * q >= p.N) break;
                uint32_t v[64];
                tmem_ld32(taddr + 64 * q, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld32(taddr + 64 * q + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_wait_ld();
                uint8_t* stg = smem + OFF_STG + (piece & 1) * lin::STG_BYTES;
                if (warp == 2 && lane == 0) tma_store_wait_read1();
                named_bar_sync(1, 128);
#pragma unroll
                for (int c16 = 0; c16 < 8; ++c16) {
                    const uint4 val = make_uint4(
                        pack_bf16x2(__uint_as_float(v[8 * c16]), __uint_as_float(v[8 * c16 + 1])),
                        pack_bf16x2(__uint_as_float(v[8 * c16 + 2]), __uint_as_float(v[8 * c16 + 3])),
                        pack_bf16x2(__uint_as_float(v[8 * c16 + 4]), __uint_as_float(v[8 * c16 + 5])),
                        pack_bf16x2(__uint_as_float(v[8 * c16 + 6]), __uint_as_float(v[8 * c16 + 7])));
                    *reinterpret_cast<uint4*>(stg + row * 128 + ((c16 ^ (row & 7)) << 4)) = val;
                }
                fence_proxy_async_smem();
                named_bar_sync(1, 128);
                if (warp == 2 && lane == 0) {
                    tma_store_2d(&tmY, smem_u32(stg), col0 + 64 * q, 0);
                    tma_store_commit();
                }
            }
            tc_fence_before();
            mbar_arrive(bar_acc_empty + 8 * buf);
        }
        if (warp == 2 && lane == 0) tma_store_wait_read();
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

static cudaError_t launch_linear_unit(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                                      const LinearParams& p, cudaStream_t stream) {
    static DeviceOnce configured;
    cudaError_t e = configured.run([&]() {
        return cudaFuncSetAttribute(linear_unit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(linu::ALLOC));
    });
    if (e != cudaSuccess) return e;
    const int grid = p.nunit < p.sm_count ? p.nunit : p.sm_count;
    count_launch();
    linear_unit_kernel<<<grid, lin::THREADS, linu::ALLOC, stream>>>(tmA, tmB, tmY, p);
    return cudaGetLastError();
}

template <bool PAIR>
static cudaError_t launch_linear_t(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                                   const LinearParams& p, cudaStream_t stream) {
    using C = lin::Cfg<PAIR>;
    auto kern = linear_kernel<PAIR>;
    static DeviceOnce configured;     // the opt-in belongs to the (function, device) pair
    {
        cudaError_t e = configured.run([&]() {
            return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(C::ALLOC));
        });
        if (e != cudaSuccess) return e;
    }
    const long long ntile = (p.T + 127) / 128;
    const long long nband = (ntile + lin::BAND - 1) / lin::BAND;
    long long grid = nband * lin::BAND * p.nsuper;               // even: BAND is
    if (PAIR && p.unit_mode) {
        const int slots = p.sm_count / 2;
        grid = 2ll * (slots < p.nunit ? slots : p.nunit);
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(lin::THREADS);
    cfg.dynamicSmemBytes = C::ALLOC;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, p);
}

// pair = true: tmB must have a box of 128 rows (each CTA of a pair stages half of a step's 256)
cudaError_t launch_linear(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                          const LinearParams& p, bool pair, cudaStream_t stream) {
    if (p.T <= 0) return cudaSuccess;
    if (p.unit_mode && !pair) return launch_linear_unit(tmA, tmB, tmY, p, stream);
    return pair ? launch_linear_t<true>(tmA, tmB, tmY, p, stream) : launch_linear_t<false>(tmA, tmB, tmY, p, stream);
}

}  // namespace tik
