// Unified causal GQA attention for sm_100a: one kernel body for the packed train-forward,
// the paged prefill and the paged decode regime, plus the split-KV combine and the
// KV-cache write.
//
// One CTA owns one MMA tile of 128 query rows and walks 128-key KV tiles in ascending
// order.  S = Q K^T and O += P V run on tcgen05 (M128 x N128 x K16 and M128 x Nd x K16,
// fp32 accumulators in TMEM); Q, K, V arrive by TMA into 128B-swizzled shared memory
// (K/V of the paged regimes are gathered page by page through the block table).  The CTA
// is warp-specialised: two TMA warps (K, V), two MMA-issuing warps (QK^T, PV) and two
// softmax warpgroups that alternate over KV tiles, one thread per row, working straight out
// of TMEM with the arithmetic of tik_core.cuh.  A thread pulls its score row into registers
// and releases the score buffer at once, and the bf16 weights go to two TMEM buffers of their
// own, so the QK^T of tile j+1 and the PV of tile j-1 run under the softmax of tile j.  What differs between regimes is only where rows come from
// and where they go:
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

constexpr int ATTN_THREADS = 384;   // warp 0 TMA (Q, K), warp 1 QK^T MMA, warp 2 TMA (V), warp 3 PV MMA, warps 4-11 softmax
constexpr int KV_STAGES = 3;

template <int D>
struct AttnSmem {
    static constexpr uint32_t ATOM = 128 * 128;          // 128 rows x 64 bf16
    static constexpr uint32_t TILE = (D / 64) * ATOM;    // one Q, K or V tile
    // seven tiles: one query tile + three K stages + three V stages, or (paired mode) two query
    // tiles + two K stages + three V stages
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = TILE;                        // paired mode: 2 * TILE
    static constexpr uint32_t OFF_V = OFF_K + KV_STAGES * TILE;
    static constexpr uint32_t OFF_BAR = OFF_V + KV_STAGES * TILE;
    static constexpr uint32_t OFF_LX = OFF_BAR + 272;             // 3 x 128 floats of row state
    // decode: exchange area of the softmax warps (per warpgroup 3 x 8 x 32 float4 of weights and
    // 4 x 32 tile maxima).  Decode uses two K stages, so for D = 128 the third K stage holds it.
    static constexpr uint32_t XCH_WG = 3 * 8 * 32 * 16 + 4 * 32 * 4;
    static constexpr uint32_t OFF_XCH = (2 * XCH_WG <= TILE) ? OFF_K + 2 * TILE : OFF_LX + 3 * 512;
    static constexpr uint32_t BYTES = OFF_LX + 3 * 512 + ((2 * XCH_WG <= TILE) ? 0 : 2 * XCH_WG);
    static constexpr uint32_t ALLOC = BYTES;                      // base must be 1 KiB aligned
};

// Rarely taken paths of the softmax loops, kept out of line so that the loop bodies stay small
// (the loops of two warpgroups, the issuing threads and the producers share one instruction cache).
template <int D>
__device__ __noinline__ void rescale_o_tmem(uint32_t to, float alpha) {
#pragma unroll 1
    for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t v[32];
        tmem_ld32(to + 32 * cc, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(rescale_o(__uint_as_float(v[i]), alpha));
        tmem_st32(to + 32 * cc, v);
    }
}
template <int D>
__device__ __noinline__ void fold_o_tmem(uint32_t t_a, uint32_t t_b, FoldCoef f) {
#pragma unroll 1
    for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t a[32], b[32];
        tmem_ld32(t_a + 32 * cc, a);
        tmem_ld32(t_b + 32 * cc, b);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i)
            a[i] = __float_as_uint(fold_value(__uint_as_float(a[i]), __uint_as_float(b[i]), f));
        tmem_st32(t_a + 32 * cc, a);
    }
    tmem_wait_st();
}

template <int D, int MODE>
__global__ void __launch_bounds__(ATTN_THREADS, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnParams p) {
    using L = AttnSmem<D>;
    constexpr int NATOM = D / 64;
    constexpr int DH = D / 2;                              // O columns owned by one softmax thread
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0;                          // one score buffer of 128 columns
    constexpr uint32_t COL_P = 128;                        // two weight buffers of 64 columns (bf16 pairs)
    constexpr uint32_t COL_OA = 256, COL_OB = 256 + D;
    constexpr uint32_t IDESC_QK = mma_idesc_bf16(128, 128, false);
    constexpr uint32_t IDESC_PV = mma_idesc_bf16(128, D, true);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Launched with programmatic stream serialization: the grid may be scheduled while the kernel
    // before it in the stream (typically the cache write or the pre-attention step of the same
    // call sequence) is still draining; nothing of this kernel's input is read before this wait.
    pdl_wait();

    // ---------------------------------------------------------------- work item
    // Train / prefill: query tiles are aligned to absolute positions.  Tiles 0..15 (their KV
    // range is one chunk) are taken two at a time: a CTA owns tiles 2m (A) and 2m+1 (B) of one
    // (sequence, head), streams every K/V tile once for both, and each softmax warpgroup keeps
    // the rows of one of the two tiles from the first KV tile to the last.  Tiles >= 16, a tile
    // without a partner, and decode run one query tile per CTA.
    int seq, head, kvh, chunk = 0, ctx = 0;
    int T0 = 0, T1 = 0;        // query tile of parity 0 (single mode, or B) and of parity 1 (A)
    bool pair = false;
    long long qrow0[2] = {0, 0};   // token row of tile row 0, per query tile (may be negative)
    long long tok0 = 0;            // first token of the sequence in the packed K/V (train)
    int row_lo[2] = {0, 0}, row_hi[2] = {0, 0};   // valid tile rows [row_lo, row_hi), per query tile
    int tile_first, tile_last;
    if (MODE == MODE_TRAIN || MODE == MODE_PREFILL) {
        pdl_launch_dependents();       // a grid launched behind this one may fill the SMs that its last wave leaves
        seq = blockIdx.z;
        head = blockIdx.y;
        kvh = head / p.G;
        int pos0, qb;
        if (MODE == MODE_TRAIN) {
            tok0 = p.cu_seqlens[seq];
            ctx = p.cu_seqlens[seq + 1] - static_cast<int>(tok0);
            pos0 = 0;
            qb = static_cast<int>(tok0);
            if (ctx <= 0) return;
        } else {
            qb = p.cu_seqlens[seq];
            const int qlen = p.cu_seqlens[seq + 1] - qb;
            ctx = p.ctx_lens[seq];
            pos0 = ctx - qlen;
            if (qlen <= 0 || pos0 < 0) return;
        }
        const int t_lo = pos0 / 128, t_hi = (ctx - 1) / 128;     // first and last query tile
        const int x = p.x_base + gridDim.x - 1 - blockIdx.x;     // heaviest candidates first
        if (x >= 8) {
            T0 = 16 + (x - 8);
            if (T0 < t_lo || T0 > t_hi) return;
        } else {
            const int ta = 2 * x, tb = 2 * x + 1;
            const bool va = ta >= t_lo && ta <= t_hi, vb = tb >= t_lo && tb <= t_hi;
            if (!va && !vb) return;
            pair = va && vb;
            T0 = vb ? tb : ta;
            T1 = ta;
        }
        for (int q2 = 0; q2 < 2; ++q2) {
            const int Tq = q2 ? T1 : T0;
            qrow0[q2] = static_cast<long long>(qb) + 128ll * Tq - pos0;
            row_lo[q2] = max(0, pos0 - 128 * Tq);
            row_hi[q2] = min(128, ctx - 128 * Tq);
        }
        tile_first = 0;
        tile_last = T0;
    } else {
        pdl_launch_dependents();       // the combine kernel may be scheduled behind this grid's last wave
        seq = blockIdx.z;
        kvh = blockIdx.y;
        head = kvh * p.G;
        // a CTA streams `cpc` consecutive chunks; each still leaves its own partial
        chunk = blockIdx.x * p.cpc;
        ctx = p.ctx_lens[seq];
        if (ctx > p.max_ctx) {
            // The grid and the scratch were sized from the host's bound: a longer context is cut
            // to that bound (and flagged) instead of writing partials past the sequence's slots.
            if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) atomicOr(p.dev_status, TIK_DEV_BAD_CONTEXT);
            ctx = p.max_ctx;
        }
        if (ctx <= 0 || chunk * CHUNK >= ctx) return;
        tile_first = chunk * TILES_PER_CHUNK;
        tile_last = min(tile_first + p.cpc * TILES_PER_CHUNK - 1, (ctx - 1) / 128);
        row_lo[0] = 0;
        row_hi[0] = p.G;
    }
    const int n_tiles = tile_last - tile_first + 1;              // K/V tiles streamed by this CTA
    // One step = one (query tile, KV tile) product.  Single mode: step g is KV tile g.  Paired
    // mode: even steps belong to B (= T0), odd steps to A (= T1 = T0 - 1), step g uses KV tile g/2;
    // A has one KV tile less, so the last step (even) is B's diagonal tile.
    const int n_steps = pair ? (2 * n_tiles - 1) : n_tiles;
    const int KS = (pair || MODE == MODE_DECODE) ? 2 : KV_STAGES;   // K stages in use
    const int q_row_first[2] = {static_cast<int>(qrow0[0]), static_cast<int>(qrow0[1])};

    // ---------------------------------------------------------------- shared memory
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    const uint32_t sbase = smem_u32(smem_raw);
    if (sbase & 1023u) {     // the swizzled tiles need a 1 KiB aligned base: refuse to run otherwise
        if (tid == 0) atomicOr(p.dev_status, TIK_DEV_WAIT_EXPIRED);
        return;
    }
    const uint32_t sQ = sbase + L::OFF_Q, sK = sbase + (pair ? 2 * L::TILE : L::OFF_K), sV = sbase + L::OFF_V;
    // barriers (8 bytes each)
    const uint32_t bar0 = sbase + L::OFF_BAR;
    const uint32_t bar_q = bar0;                 // Q landed
    const uint32_t bar_kfull = bar0 + 8;         // [KV_STAGES] K tile landed
    const uint32_t bar_vfull = bar0 + 40;        // [KV_STAGES] V tile landed
    const uint32_t bar_kempty = bar0 + 72;       // [KV_STAGES] QK^T that read the stage is done
    const uint32_t bar_vempty = bar0 + 104;      // [KV_STAGES] PV that read the stage is done
    const uint32_t bar_sfull = bar0 + 136;       // [2] QK^T of an even / odd tile done: scores ready in TMEM
    const uint32_t bar_pfull = bar0 + 152;       // [2] P written over the scores, O rescaled (4 warps)
    const uint32_t bar_pempty = bar0 + 168;      // [2] PV done: O updated, weight buffer free
    const uint32_t bar_hand = bar0 + 184;        // [4] reference-maximum hand-off between the warpgroups
    const uint32_t bar_sempty = bar0 + 248;      // [2] scores of a tile are in registers (4 warps)
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_BAR + 264);
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 268);
    float* lx = reinterpret_cast<float*>(smem + L::OFF_LX);
    // values only the epilogue needs are parked in shared memory instead of living in registers
    // across the main loop: [q2][0] first token row, [q2][1] row_lo, [q2][2] row_hi
    volatile int* meta = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 216);
    if (tid == 64) {
        for (int q2 = 0; q2 < 2; ++q2) {
            meta[3 * q2] = q_row_first[q2];
            meta[3 * q2 + 1] = row_lo[q2];
            meta[3 * q2 + 2] = row_hi[q2];
        }
    }

    // ---------------------------------------------------------------- set-up
    // The two TMA warps initialise the barriers of their own rings and put the first K / V tiles
    // (and Q) in flight before the CTA-wide synchronisation: a CTA's first data then arrives while
    // TMEM is being allocated instead of ~1000 cycles later.
    const int kv = (warp == 2) ? 1 : 0;                     // producer warps: 0 streams K, 2 streams V
    const CUtensorMap* tm = kv ? &tmV : &tmK;
    int my_phys = p.num_pages;                              // paged regimes: one block-table entry per lane
    auto produce_tile = [&](int it) {                       // whole warp (paged) or lane 0 (train)
        const int j = tile_first + it;
        // (no division by a run-time stage count: this code sits between a stage's release and its
        // next request, and the issuing threads below are the pace-makers of the tensor pipe)
        const bool two = !kv && KS == 2;
        const int st = two ? (it & 1) : (it % KV_STAGES);
        const uint32_t use = two ? (it >> 1) : (it / KV_STAGES);
        const uint32_t dst = (kv ? sV : sK) + st * L::TILE;
        const uint32_t full = (kv ? bar_vfull : bar_kfull) + 8 * st;
        if (MODE != MODE_TRAIN) {
            // Paged K/V: the warp reads 32 block-table entries at a time (one per lane, coalesced),
            // so the table's latency is paid once per 32 pages instead of before every tile.
            // (page sizes are powers of two: shifts, not divisions)
            const int tpb_mask = (32 >> p.ppt_shift) - 1;             // tiles per batch - 1
            if ((it & tpb_mask) == 0) {
                const int lp = ((128 * j) >> p.page_shift) + lane;
                int ph = p.num_pages;       // out of range: the box is filled with zeros
                if ((lp << p.page_shift) < ctx) {
                    ph = (lp < p.max_blocks) ? p.block_table[static_cast<long long>(seq) * p.max_blocks + lp] : -1;
                    if (ph < 0 || ph >= p.num_pages) {
                        if (kv == 0) atomicOr(p.dev_status, TIK_DEV_BAD_BLOCK);
                        ph = p.num_pages;
                    }
                }
                my_phys = ph;
            }
        }
        // paged: lane i < pages_per_tile takes the tile's i-th page (everything that does not need
        // the stage to be free happens before the wait; after it only the copies are issued)
        int my_page = 0;
        if (MODE != MODE_TRAIN) {
            const int in_batch = it & ((32 >> p.ppt_shift) - 1);
            my_page = __shfl_sync(0xffffffffu, my_phys, (in_batch << p.ppt_shift) + (lane & (p.pages_per_tile - 1)));
        }
        // Each stage has its own release barrier with this warp as its only waiter: a barrier
        // shared with waiters of a different lag could run two phases ahead of the slowest one,
        // which a parity wait cannot tell from "not yet".
        if (use > 0)
            mbar_wait((kv ? bar_vempty : bar_kempty) + 8 * st, (use - 1) & 1, abort_word, p.dev_status);
        if (lane == 0) mbar_expect_tx(full, L::TILE);
        if (MODE == MODE_TRAIN) {
            if (lane == 0) {
                const int row = static_cast<int>(tok0) + 128 * j;
                for (int a = 0; a < NATOM; ++a) tma_load_3d(dst + a * L::ATOM, tm, full, a * 64, kvh, row);
            }
        } else {
            __syncwarp();                                 // the expected byte count is registered first
            if (lane < p.pages_per_tile) {
                const uint32_t off = static_cast<uint32_t>(lane << p.page_shift) * 128u;
                for (int a = 0; a < NATOM; ++a)
                    tma_load_4d(dst + a * L::ATOM + off, tm, full, a * 64, 0, kvh, my_page);
            }
        }
    };
    auto load_q = [&]() {                                   // lane 0 of warp 0
        if (MODE == MODE_DECODE) {
            // the G query rows go to rows 0.., 32.., 64.., 96..: every lane quarter of the score
            // tile then holds the same G rows and the four warps of a warpgroup share a row's columns
            mbar_expect_tx(bar_q, 4u * static_cast<uint32_t>(p.G) * 128u * NATOM);
            for (int q4 = 0; q4 < 4; ++q4)
                for (int a = 0; a < NATOM; ++a)
                    tma_load_3d(sQ + a * L::ATOM + q4 * 4096, &tmQ, bar_q, a * 64, head, seq);
        } else {
            mbar_expect_tx(bar_q, pair ? 2 * L::TILE : L::TILE);
            for (int q2 = 0; q2 < (pair ? 2 : 1); ++q2)
                for (int a = 0; a < NATOM; ++a)
                    tma_load_3d(sQ + q2 * L::TILE + a * L::ATOM, &tmQ, bar_q, a * 64, head,
                                static_cast<int>(qrow0[q2]));
        }
    };
    const int n_early = min(n_tiles, kv ? KV_STAGES : KS);  // tiles that need no stage release
    if (warp == 0 || warp == 2) {
        if (lane == 0) {
            tma_prefetch_desc(tm);
            if (kv == 0) {
                tma_prefetch_desc(&tmQ);
                mbar_init(bar_q, 1);
            }
            for (int i = 0; i < KV_STAGES; ++i) {
                mbar_init((kv ? bar_vfull : bar_kfull) + 8 * i, 1);
                mbar_init((kv ? bar_vempty : bar_kempty) + 8 * i, 1);
            }
            fence_barrier_init();
            if (kv == 0 && MODE != MODE_DECODE) load_q();
        }
        __syncwarp();
        if (MODE != MODE_TRAIN || lane == 0)
            for (int it = 0; it < n_early; ++it) produce_tile(it);
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            for (int i = 0; i < 2; ++i) {
                mbar_init(bar_sfull + 8 * i, 1);
                mbar_init(bar_pfull + 8 * i, 4);
                mbar_init(bar_sempty + 8 * i, 4);
                mbar_init(bar_pempty + 8 * i, 1);
            }
            for (int i = 0; i < 4; ++i) mbar_init(bar_hand + 8 * i, 1);
            fence_barrier_init();
        }
        __syncwarp();
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    } else if (warp == 3) {
        // an earlier kernel on this context may have run out of a wait: then do nothing at all
        if (lane == 0)
            *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
    }
    if (MODE == MODE_DECODE) {
        // rows >= G of the Q tile are never loaded: zero them (their scores and weights stay 0)
        const uint4 z = make_uint4(0, 0, 0, 0);
        for (uint32_t i = tid; i < L::TILE / 16; i += ATTN_THREADS)
            reinterpret_cast<uint4*>(smem + L::OFF_Q)[i] = z;
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    auto chunk_of = [&](int it) { return (tile_first + it) / TILES_PER_CHUNK; };
    auto is_chunk_start = [&](int it) { return ((tile_first + it) % TILES_PER_CHUNK) == 0; };
    auto col_o_of = [&](int it) -> uint32_t {
        // train / prefill: chunk 0 accumulates in O_A (the folded accumulator), later chunks in O_B;
        // decode: consecutive chunks alternate, each is written out as a partial of its own
        if (MODE == MODE_DECODE) return (chunk_of(it) & 1) ? COL_OB : COL_OA;
        return chunk_of(it) == 0 ? COL_OA : COL_OB;
    };

    // Register budget: the four role warps (one warpgroup) need few registers, a softmax thread
    // holds a 128-column score row.  128 x 88 + 256 x 208 = 64 512 registers.
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    if (warp == 0 || warp == 2) {
        // ------------------------------------------------------------ TMA producers
        // warp 0 streams Q and the K tiles, warp 2 the V tiles: a K tile is requested as soon as
        // the QK^T that used its stage has finished, without queueing behind a wait for PV.
        if (MODE == MODE_DECODE && kv == 0 && lane == 0) load_q();     // after the zero fill of the Q tile
        if (MODE != MODE_TRAIN || lane == 0) {
            for (int it = n_early; it < n_tiles; ++it) {
                if (*abort_word) break;      // a wait expired somewhere: stop issuing copies
                produce_tile(it);
            }
        }
        if (MODE == MODE_DECODE && !*abort_word) {
            // This warp has requested its last tile; the SM asks nothing of HBM while the CTA
            // drains and its successor sets up.  Fill that gap: pull into L2 the first K (V)
            // tiles of the CTA `lookahead` blocks later, which starts about when this one ends.
            const long long nblk = static_cast<long long>(gridDim.x) * gridDim.y * gridDim.z;
            const long long lin = (static_cast<long long>(blockIdx.z) * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
            const long long nxt = lin + p.lookahead;
            if (p.lookahead > 0 && nxt < nblk) {
                const int bx = static_cast<int>(nxt % gridDim.x);
                const int by = static_cast<int>((nxt / gridDim.x) % gridDim.y);
                const int bz = static_cast<int>(nxt / (static_cast<long long>(gridDim.x) * gridDim.y));
                const int ctx2 = p.ctx_lens[bz];
                const int pos2 = bx * p.cpc * CHUNK;                 // first key position of that CTA
                const int lp = (pos2 >> p.page_shift) + lane;
                if (lane < KV_STAGES * p.pages_per_tile && lp < p.max_blocks && (lp << p.page_shift) < ctx2) {
                    const int ph = p.block_table[static_cast<long long>(bz) * p.max_blocks + lp];
                    if (ph >= 0 && ph < p.num_pages)
                        for (int a = 0; a < NATOM; ++a) tma_prefetch_l2_4d(tm, a * 64, 0, by, ph);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ QK^T issuer
        // Two threads feed the tensor pipe (this one and the PV issuer in warp 3): whatever an
        // issuing thread executes between MMAs is time in which it queues nothing, so each
        // keeps to waits, one MMA chain and its commits per step.
        if (lane == 0) {
            mbar_wait(bar_q, 0, abort_word, p.dev_status);
            const uint64_t dq0 = smem_desc_sw128(sQ, 0, 1024);
            const uint64_t dq1 = smem_desc_sw128(sQ + L::TILE, 0, 1024);
            for (int g = 0; g < n_steps; ++g) {
                const int kt = pair ? (g >> 1) : g;                 // K tile of this step
                const int st = (KS == 2) ? (kt & 1) : (kt % KV_STAGES), b = g & 1;
                const int kuse = (KS == 2) ? (kt >> 1) : (kt / KV_STAGES);
                // the single score buffer is free once the softmax of step g-1 holds it in registers
                mbar_wait(bar_kfull + 8 * st, kuse & 1, abort_word, p.dev_status);
                if (g >= 1) mbar_wait(bar_sempty + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1, abort_word, p.dev_status);
                tc_fence_after();
                const uint64_t dq = (pair && b) ? dq1 : dq0;
                const uint64_t dk = smem_desc_sw128(sK + st * L::TILE, 0, 1024);
                if (D == 128) mma_ss_chain8_fresh(tmem + COL_S, dq, dk, IDESC_QK);
                else mma_ss_chain4_fresh(tmem + COL_S, dq, dk, IDESC_QK);
                mma_commit(bar_sfull + 8 * b);
                // the K stage is free after its last reader (paired mode: the odd step, or B's last tile)
                if (!pair || b || g == n_steps - 1) mma_commit(bar_kempty + 8 * st);
            }
        }
        __syncwarp();
    } else if (warp == 3) {
        // ------------------------------------------------------------ PV issuer
        // (done here, after the set-up synchronisation: its dependent global loads would otherwise
        // hold up every warp of the CTA, and this thread has nothing to do until the first weights)
        // Query tiles are read once, so a CTA's first load is a DRAM miss of ~1.5 us with nothing
        // to overlap it.  CTAs start roughly in block order as SMs free up: prefetch into L2 the
        // query tiles of the CTA that comes `lookahead` blocks later, which starts about when this
        // one ends.
        if (MODE != MODE_DECODE && lane == 0) {
            const long long nblk = static_cast<long long>(gridDim.x) * gridDim.y * gridDim.z;
            const long long lin = (static_cast<long long>(blockIdx.z) * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
            const long long nxt = lin + p.lookahead;
            if (nxt < nblk) {
                const int bx = static_cast<int>(nxt % gridDim.x);
                const int by = static_cast<int>((nxt / gridDim.x) % gridDim.y);
                const int bz = static_cast<int>(nxt / (static_cast<long long>(gridDim.x) * gridDim.y));
                int qb2 = p.cu_seqlens[bz], ctx2, pos2;
                if (MODE == MODE_TRAIN) {
                    ctx2 = p.cu_seqlens[bz + 1] - qb2;
                    pos2 = 0;
                } else {
                    ctx2 = p.ctx_lens[bz];
                    pos2 = ctx2 - (p.cu_seqlens[bz + 1] - qb2);
                }
                if (ctx2 > 0 && pos2 >= 0) {
                    const int x2 = p.x_base + gridDim.x - 1 - bx;
                    const int t_lo2 = pos2 / 128, t_hi2 = (ctx2 - 1) / 128;
                    for (int q2 = 0; q2 < 2; ++q2) {
                        const int Tq = (x2 >= 8) ? (16 + x2 - 8) : (2 * x2 + q2);
                        if ((x2 >= 8 && q2 == 1) || Tq < t_lo2 || Tq > t_hi2) continue;
                        const int row = qb2 + 128 * Tq - pos2;
                        for (int a = 0; a < NATOM; ++a) tma_prefetch_l2_3d(&tmQ, a * 64, by, row);
                    }
                }
            }
        }
        if (lane == 0) {
            for (int g = 0; g < n_steps; ++g) {
                const int vt = pair ? (g >> 1) : g;
                const int st = vt % KV_STAGES, b = g & 1;
                mbar_wait(bar_vfull + 8 * st, (vt / KV_STAGES) & 1, abort_word, p.dev_status);
                mbar_wait(bar_pfull + 8 * b, (g >> 1) & 1, abort_word, p.dev_status);
                tc_fence_after();
                // paired mode: B accumulates in O_A, A in O_B, each from its first KV tile on
                const uint32_t col_o = pair ? (b ? COL_OB : COL_OA) : col_o_of(g);
                const bool fresh = pair ? (vt == 0) : is_chunk_start(g);
                // A = bf16 weights in TMEM (8 columns per 16 keys), B = V tile
                mma_ts_chain8(tmem + col_o, tmem + COL_P + 64 * b,
                              smem_desc_sw128(sV + st * L::TILE, L::ATOM, 1024), IDESC_PV, fresh ? 0u : 1u);
                mma_commit(bar_pempty + 8 * b);
                if (!pair || b || g == n_steps - 1) mma_commit(bar_vempty + 8 * st);
            }
        }
        __syncwarp();
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    {
        // ------------------------------------------------------------ softmax (two warpgroups)
        // The warpgroups alternate over KV tiles: warpgroup wg owns the tiles with it % 2 == wg
        // and with them score buffer wg, one thread per row and all 128 columns of the tile.
        // While one warpgroup is in its exp2 phase the other loads scores, reduces the maximum
        // and stores weights, so the special-function unit stays busy.  The row state (running
        // maximum, the two half row sums, the folded state of earlier chunks) lives in shared
        // memory and is handed from the thread of tile it to the thread of tile it+1: the maximum
        // through an mbarrier per lane quarter, the row sums with the "weights written" barrier.
        const int wg = (warp - 4) >> 2;
        const int quarter = warp & 3;                       // TMEM lane quarter of this warp
        const int r = quarter * 32 + lane;                  // tile row == TMEM lane
        const uint32_t tlane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int qpos = 128 * T0 + r;      // train / prefill, single mode: position of this thread's row
        const float c = p.c;
        float* st_m = lx;                 // [128]    running maximum of the current chunk
        float* st_l = lx + 128;           // [2][128] half row sums of the current chunk
        const uint32_t bar_m = bar_hand + 8 * quarter;       // "maximum of tile it published"
        const uint32_t ts = tlane + COL_S;
        const uint32_t tp = tlane + COL_P + 64 * wg;
        // Folded state of the finished chunks.  Both threads of a row keep it: warpgroup 0 folds
        // at the first tile of a chunk (the state of the finished chunk is handed to it), and
        // warpgroup 1 owns every chunk's last tile, so it folds the same numbers on its own.
        float M_g = -CUDART_INF_F, Lg_lo = 0.0f, Lg_hi = 0.0f;
        float m_own = -CUDART_INF_F, l_own_lo = 0.0f, l_own_hi = 0.0f;   // state after this thread's last tile

        auto wait_pv = [&](int x) {
            mbar_wait(bar_pempty + 8 * (x & 1), (x >> 1) & 1, abort_word, p.dev_status);
            tc_fence_after();
        };
        // The other warpgroup has finished tile x (weights and row sums written): the barrier the
        // PV issuer waits on doubles as the hand-off of the row sums.
        auto wait_tile_done = [&](int x) {
            mbar_wait(bar_pfull + 8 * (x & 1), (x >> 1) & 1, abort_word, p.dev_status);
        };
        // folds a finished chunk (m_c, l_c halves) into the global row state; with_o also folds
        // its accumulator O_B into O_A (one thread per row does that, after the chunk's last PV)
        auto fold_chunk = [&](int chunk_idx, float m_c, float l_c_lo, float l_c_hi, bool with_o) {
            if (chunk_idx == 0) {            // chunk 0 accumulated in place in O_A
                M_g = m_c;
                Lg_lo = l_c_lo;
                Lg_hi = l_c_hi;
            } else {
                const FoldCoef f = fold_coef(M_g, m_c, c);
                Lg_lo = fold_value(Lg_lo, l_c_lo, f);
                Lg_hi = fold_value(Lg_hi, l_c_hi, f);
                M_g = f.M_new;
                if (with_o) fold_o_tmem<D>(tlane + COL_OA, tlane + COL_OB, f);
            }
        };
        // decode: the partial of a finished chunk; the accumulator columns [col0, col0 + ncol)
        auto write_partial_ml = [&](int chunk_idx, float m_c, float l_c_lo, float l_c_hi) {
            if (r < p.G) {
                const long long slot = (static_cast<long long>(seq) * p.Hq + head + r) * p.nchunk_max + chunk_idx;
                p.part_ml[4 * slot] = m_c;
                p.part_ml[4 * slot + 1] = l_c_lo;
                p.part_ml[4 * slot + 2] = l_c_hi;
            }
        };
        auto write_partial_o = [&](int chunk_idx, int col0, int ncol) {
            const uint32_t to = tlane + ((chunk_idx & 1) ? COL_OB : COL_OA);
            for (int cc = 0; cc < ncol / 32; ++cc) {
                uint32_t v[32];
                tmem_ld32(to + col0 + 32 * cc, v);
                tmem_wait_ld();
                if (r < p.G) {
                    const long long slot =
                        (static_cast<long long>(seq) * p.Hq + head + r) * p.nchunk_max + chunk_idx;
                    float4* dst = reinterpret_cast<float4*>(p.part_o + slot * D + col0 + 32 * cc);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                             __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                }
            }
        };
        const int last = n_tiles - 1;

        if (MODE == MODE_DECODE) {
            // ---- decode: only G rows are real, and one warp per row block would leave the exp2
            // work of a tile on a single scheduler.  The query rows are replicated into every
            // lane quarter instead, and warp `quarter` takes columns [32 quarter, 32 quarter + 32)
            // of every row: tile maximum and reference maximum by an exchange through shared
            // memory, exponentials on all four warps, and then warp 0 alone sums the 128 weights
            // of a row in the contract's order, packs them and writes them to TMEM, so the
            // numbers are those of the one-thread-per-row path.
            float4* xs = reinterpret_cast<float4*>(smem + L::OFF_XCH + wg * L::XCH_WG);   // [3][8][32]
            float* xm = reinterpret_cast<float*>(smem + L::OFF_XCH + wg * L::XCH_WG + 3 * 8 * 32 * 16);   // [4][32]
            const uint32_t bar_m0 = bar_hand;
            for (int it = wg; it < n_tiles; it += 2) {
                const int j = tile_first + it;
                const bool chunk_start = is_chunk_start(it);
                const bool fold_now = chunk_start && it > 0;      // a finished chunk precedes this tile
                mbar_wait(bar_sfull + 8 * wg, (it >> 1) & 1, abort_word, p.dev_status);
                tc_fence_after();
                uint32_t sc[32];
                tmem_ld32(ts + 32 * quarter, sc);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_sempty + 8 * wg);
                const int kmax = (ctx - 1) - 128 * j - 32 * quarter;    // own columns > kmax are masked
                if (kmax < 31) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i > kmax) sc[i] = 0xff800000u;              // -inf
                }
                float mx[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) mx[k] = fmaxf(__uint_as_float(sc[2 * k]), __uint_as_float(sc[2 * k + 1]));
#pragma unroll
                for (int i = 8; i < 32; i += 8) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mx[k] = fmax3(mx[k], __uint_as_float(sc[i + 2 * k]), __uint_as_float(sc[i + 2 * k + 1]));
                }
                xm[quarter * 32 + lane] = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                // state handed over by the warpgroup that processed tile it-1
                float m_old = -CUDART_INF_F, l_old_lo = 0.0f, l_old_hi = 0.0f;
                float m_prev = 0.0f, l_prev_lo = 0.0f, l_prev_hi = 0.0f;   // finished chunk, if any
                if (it > 0) {
                    mbar_wait(bar_m0, (it - 1) & 1, abort_word, p.dev_status);
                    if (!chunk_start) {
                        m_old = st_m[lane];
                    } else if (quarter == 0) {
                        wait_tile_done(it - 1);
                        m_prev = st_m[lane];
                        l_prev_lo = st_l[lane];
                        l_prev_hi = st_l[128 + lane];
                    }
                }
                named_bar_sync(2 + wg, 128);                 // maxima exchanged, old reference read by all
                const float mt = fmaxf(fmaxf(xm[lane], xm[32 + lane]), fmaxf(xm[64 + lane], xm[96 + lane]));
                const float m_new = softmax_next_max(m_old, mt, c);
                if (quarter == 0) {
                    st_m[lane] = m_new;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_m0);
                }
                const float neg_mc = -__fmul_rn(m_new, c);
                float x[128];                                // warps 1-3 use the first 32 only
#pragma unroll
                for (int i = 0; i < 32; i += 8) softmax_x8(&sc[i], c, neg_mc, &x[i]);
                if (quarter != 0) {
#pragma unroll
                    for (int c4 = 0; c4 < 8; ++c4)
                        xs[((quarter - 1) * 8 + c4) * 32 + lane] =
                            make_float4(x[4 * c4], x[4 * c4 + 1], x[4 * c4 + 2], x[4 * c4 + 3]);
                }
                named_bar_sync(2 + wg, 128);                 // weights of columns 32..127 are in shared memory
                if (quarter == 0) {
#pragma unroll
                    for (int k = 0; k < 24; ++k) {
                        const float4 v4 = xs[k * 32 + lane];
                        x[32 + 4 * k] = v4.x;
                        x[32 + 4 * k + 1] = v4.y;
                        x[32 + 4 * k + 2] = v4.z;
                        x[32 + 4 * k + 3] = v4.w;
                    }
                    RowSum4 rs_lo, rs_hi;
                    rs_lo.reset();
                    rs_hi.reset();
                    uint32_t pk[64];
#pragma unroll
                    for (int i = 0; i < 64; i += 8) softmax_sum_pack8(&x[i], rs_lo, &pk[i >> 1]);
                    // the weight buffer of this warpgroup was last read by the PV of tile it-2
                    if (it >= 2) wait_pv(it - 2);
                    tmem_st32(tp, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
#pragma unroll
                    for (int i = 0; i < 64; i += 8) softmax_sum_pack8(&x[64 + i], rs_hi, &pk[32 + (i >> 1)]);
                    tmem_st32(tp + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]));
                    const float alpha = softmax_alpha(m_old, m_new, c);
                    if (it > 0 && !chunk_start) {
                        wait_tile_done(it - 1);
                        l_old_lo = st_l[lane];
                        l_old_hi = st_l[128 + lane];
                    }
                    m_own = m_new;
                    l_own_lo = __fmaf_rn(l_old_lo, alpha, rs_lo.total());
                    l_own_hi = __fmaf_rn(l_old_hi, alpha, rs_hi.total());
                    st_l[lane] = l_own_lo;
                    st_l[128 + lane] = l_own_hi;
                    if (fold_now) {
                        wait_pv(it - 1);
                        write_partial_ml(chunk_of(it - 1), m_prev, l_prev_lo, l_prev_hi);
                        write_partial_o(chunk_of(it - 1), 0, D);
                    } else if (!chunk_start && !__all_sync(0xffffffffu, alpha == 1.0f)) {
                        wait_pv(it - 1);
                        rescale_o_tmem<D>(tlane + col_o_of(it), alpha);
                    }
                    tmem_wait_st();
                } else if (it >= 2) {
                    wait_pv(it - 2);     // every warp passes this wait before it arrives for tile it
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pfull + 8 * wg);
            }
            // ---- the last chunk's partial: state by warp 0 of the warpgroup that owned the last
            // tile, accumulator columns half by each warpgroup's warp 0
            if (wg == (last & 1)) {
                wait_pv(last);
                if (quarter == 0 && !p.direct_out) write_partial_ml(chunk_of(last), m_own, l_own_lo, l_own_hi);
                tc_fence_before();
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            tc_fence_after();
            if (quarter == 0 && !p.direct_out) write_partial_o(chunk_of(last), DH * wg, DH);
            if (quarter == 0 && p.direct_out) {
                // One chunk per sequence: its state is the global state (the combine would copy it),
                // so the rows are normalised and stored here, by the combine's own operations; the
                // row sums of the last tile's owner are in shared memory since its hand-over.
                const float Ltot = finalize_l(st_l[lane], st_l[128 + lane]);
                const float inv = finalize_inv(Ltot);
                const long long orow = static_cast<long long>(seq) * p.Hq + head + r;
                __nv_bfloat16* const og = reinterpret_cast<__nv_bfloat16*>(p.o) + orow * D + DH * wg;
                for (int cc = 0; cc < DH / 32; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(tlane + COL_OA + DH * wg + 32 * cc, v);
                    tmem_wait_ld();
                    if (r < p.G) {
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
                if (wg == (last & 1) && r < p.G && p.lse) p.lse[orow] = finalize_lse(m_own, Ltot, c);
            }
        } else if (pair) {
            // ---- paired mode: this warpgroup keeps the rows of one query tile (wg 0: tile B = T0,
            // wg 1: tile A = T1) through all of that tile's KV tiles; nothing is handed over.
            const int Tq = wg ? T1 : T0;
            const int qpos_p = 128 * Tq + r;
            const uint32_t to = tlane + (wg ? COL_OB : COL_OA);
            float m_run = -CUDART_INF_F, l_lo = 0.0f, l_hi = 0.0f;
            int g_last = wg;
            for (int g = wg; g < n_steps; g += 2) {
                g_last = g;
                const int j = g >> 1;
                mbar_wait(bar_sfull + 8 * wg, (g >> 1) & 1, abort_word, p.dev_status);
                tc_fence_after();
                const int kmax = qpos_p - 128 * j;              // columns > kmax are masked
                uint32_t sc[128];
                tmem_ld32(ts, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
                tmem_ld32(ts + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                tmem_ld32(ts + 64, *reinterpret_cast<uint32_t(*)[32]>(&sc[64]));
                tmem_ld32(ts + 96, *reinterpret_cast<uint32_t(*)[32]>(&sc[96]));
                tmem_wait_ld();
                // the scores are in registers: the next QK^T may overwrite the buffer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_sempty + 8 * wg);
                if (kmax < 127) {
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (i > kmax) sc[i] = 0xff800000u;          // -inf
                }
                float mx[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) mx[k] = fmaxf(__uint_as_float(sc[2 * k]), __uint_as_float(sc[2 * k + 1]));
#pragma unroll
                for (int i = 16; i < 128; i += 16) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mx[k] = fmax3(mx[k], __uint_as_float(sc[i + 2 * k]), __uint_as_float(sc[i + 2 * k + 1]));
                }
                const float mt = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmax3(fmax3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
                const float m_new = softmax_next_max(m_run, mt, c);
                const float neg_mc = -__fmul_rn(m_new, c);
                const float alpha = softmax_alpha(m_run, m_new, c);
                m_run = m_new;
                RowSum4 rs_lo, rs_hi;
                rs_lo.reset();
                rs_hi.reset();
#pragma unroll
                for (int i = 0; i < 64; i += 8) softmax_p8(&sc[i], c, neg_mc, rs_lo, &sc[i >> 1]);
                // The PV of step g-2 read this warpgroup's weight buffer and updated its
                // accumulator.  It is waited for here, right before the first store: in front of
                // the score load the same wait sat inside both the softmax chain and the
                // load -> QK^T -> load cycle of the score buffer (measured: 7-9 % of the kernel).
                if (g >= 2) wait_pv(g - 2);
                tmem_st32(tp, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
#pragma unroll
                for (int i = 0; i < 64; i += 8) softmax_p8(&sc[64 + i], c, neg_mc, rs_hi, &sc[32 + (i >> 1)]);
                tmem_st32(tp + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                l_lo = __fmaf_rn(l_lo, alpha, rs_lo.total());
                l_hi = __fmaf_rn(l_hi, alpha, rs_hi.total());
                if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.0f)) {
                    // rescale this tile's accumulator (its last PV, step g-2, is complete)
                    rescale_o_tmem<D>(to, alpha);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pfull + 8 * wg);
            }
            // ---- this tile is complete after its last PV: normalise and store its rows
            wait_pv(g_last);
            const float Ltot = finalize_l(l_lo, l_hi);
            const float inv = finalize_inv(Ltot);
            const int e_row0 = meta[3 * wg], e_lo = meta[3 * wg + 1], e_hi = meta[3 * wg + 2];
            const bool valid = (r >= e_lo) && (r < e_hi);
            const long long orow = (static_cast<long long>(e_row0) + r) * p.Hq + head;
            if (valid && p.lse) p.lse[orow] = finalize_lse(m_run, Ltot, c);
            __nv_bfloat16* optr = reinterpret_cast<__nv_bfloat16*>(p.o) + orow * D;
            // A complete tile leaves through shared memory (the tile's own, now idle, query
            // buffer) and one tiled TMA store; a ragged tile is written row by row.
            const bool full_tile = e_lo == 0 && e_hi == 128;
            uint8_t* stage = smem + L::OFF_Q + wg * L::TILE;
            // 64 columns (one swizzle atom) at a time: both TMEM loads of an atom are in flight
            // together, and the atom's TMA store reads shared memory while the next one is staged
#pragma unroll
            for (int a = 0; a < NATOM; ++a) {
                uint32_t v[64];
                tmem_ld32(to + 64 * a, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld32(to + 64 * a + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i) {                 // 16-byte chunks of the atom's 128-byte row
                    uint32_t w4[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        w4[j] = pack_bf16x2(finalize_o(__uint_as_float(v[8 * i + 2 * j]), inv),
                                            finalize_o(__uint_as_float(v[8 * i + 2 * j + 1]), inv));
                    const uint4 val = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                    if (full_tile) {
                        *reinterpret_cast<uint4*>(stage + a * L::ATOM + r * 128 + ((i ^ (r & 7)) << 4)) = val;
                    } else if (valid) {
                        reinterpret_cast<uint4*>(optr + 64 * a)[i] = val;
                    }
                }
                if (full_tile) {
                    fence_proxy_async_smem();
                    named_bar_sync(2 + wg, 128);
                    if (quarter == 0 && lane == 0) {
                        tma_store_3d(&p.tmO, smem_u32(stage) + a * L::ATOM, a * 64, head, e_row0);
                        tma_store_commit();
                    }
                }
            }
            if (full_tile && quarter == 0 && lane == 0) tma_store_wait_read();
        } else {
        for (int it = wg; it < n_tiles; it += 2) {
            const int j = tile_first + it;
            const bool chunk_start = is_chunk_start(it);
            mbar_wait(bar_sfull + 8 * wg, (it >> 1) & 1, abort_word, p.dev_status);
            tc_fence_after();
            {
                const int kmax = qpos - 128 * j;            // columns > kmax are masked
                uint32_t sc[128];
                tmem_ld32(ts, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
                tmem_ld32(ts + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                tmem_ld32(ts + 64, *reinterpret_cast<uint32_t(*)[32]>(&sc[64]));
                tmem_ld32(ts + 96, *reinterpret_cast<uint32_t(*)[32]>(&sc[96]));
                tmem_wait_ld();
                // the scores are in registers: the next QK^T may overwrite the buffer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_sempty + 8 * wg);
                if (kmax < 127) {
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (i > kmax) sc[i] = 0xff800000u;          // -inf
                }
                float mx[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) mx[k] = fmaxf(__uint_as_float(sc[2 * k]), __uint_as_float(sc[2 * k + 1]));
#pragma unroll
                for (int i = 16; i < 128; i += 16) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mx[k] = fmax3(mx[k], __uint_as_float(sc[i + 2 * k]), __uint_as_float(sc[i + 2 * k + 1]));
                }
                const float mt = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmax3(fmax3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
                // state handed over by the thread that processed tile it-1
                float m_old = -CUDART_INF_F, l_old_lo = 0.0f, l_old_hi = 0.0f;
                float m_prev = 0.0f, l_prev_lo = 0.0f, l_prev_hi = 0.0f;   // finished chunk, if any
                const bool fold_now = chunk_start && it > 0;     // a finished chunk precedes this tile
                if (it > 0) {
                    mbar_wait(bar_m, (it - 1) & 1, abort_word, p.dev_status);
                    if (fold_now) {
                        wait_tile_done(it - 1);
                        m_prev = st_m[r];
                        l_prev_lo = st_l[r];
                        l_prev_hi = st_l[128 + r];
                    } else {
                        m_old = st_m[r];
                    }
                }
                const float m_new = softmax_next_max(m_old, mt, c);
                st_m[r] = m_new;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_m);
                const float neg_mc = -__fmul_rn(m_new, c);
                const float alpha = softmax_alpha(m_old, m_new, c);
                RowSum4 rs_lo, rs_hi;
                rs_lo.reset();
                rs_hi.reset();
                // a masked score is -inf: the fma gives -inf and ex2 gives +0 exactly
#pragma unroll
                for (int i = 0; i < 64; i += 8) softmax_p8(&sc[i], c, neg_mc, rs_lo, &sc[i >> 1]);
                // The weight buffer of this warpgroup was last read by the PV of tile it-2: waited
                // for right before the first store, not in front of the score load.  Every warp
                // passes this wait before it arrives for tile it, so no arrival can land in the
                // barrier phase of tile it-2.
                if (it >= 2) wait_pv(it - 2);
                tmem_st32(tp, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
#pragma unroll
                for (int i = 0; i < 64; i += 8) softmax_p8(&sc[64 + i], c, neg_mc, rs_hi, &sc[32 + (i >> 1)]);
                tmem_st32(tp + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                if (it > 0 && !fold_now) {
                    wait_tile_done(it - 1);
                    if (!chunk_start) {
                        l_old_lo = st_l[r];
                        l_old_hi = st_l[128 + r];
                    }
                }
                m_own = m_new;
                l_own_lo = __fmaf_rn(l_old_lo, alpha, rs_lo.total());
                l_own_hi = __fmaf_rn(l_old_hi, alpha, rs_hi.total());
                st_l[r] = l_own_lo;
                st_l[128 + r] = l_own_hi;
                if (fold_now) {
                    wait_pv(it - 1);
                    fold_chunk(chunk_of(it - 1), m_prev, l_prev_lo, l_prev_hi, true);
                } else if (!chunk_start && !__all_sync(0xffffffffu, alpha == 1.0f)) {
                    // rescale the chunk accumulator of this row
                    wait_pv(it - 1);
                    rescale_o_tmem<D>(tlane + col_o_of(it), alpha);
                }
                tmem_wait_st();
                // this thread closed a chunk that is not the row's last: fold its scalars here too
                if (it != last && ((tile_first + it) % TILES_PER_CHUNK) == TILES_PER_CHUNK - 1)
                    fold_chunk(chunk_of(it), m_own, l_own_lo, l_own_hi, false);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull + 8 * wg);
        }

        // ---- the warpgroup that owned the last tile finishes the row state
        if (wg == (last & 1)) {
            wait_pv(last);
            fold_chunk(chunk_of(last), m_own, l_own_lo, l_own_hi, true);
            const float Ltot = finalize_l(Lg_lo, Lg_hi);
            st_m[r] = finalize_inv(Ltot);       // the hand-off slots are free now
            const bool valid = (r >= meta[1]) && (r < meta[2]);
            if (valid && p.lse) p.lse[(static_cast<long long>(meta[0]) + r) * p.Hq + head] = finalize_lse(M_g, Ltot, c);
            tc_fence_before();
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        tc_fence_after();
        // both warpgroups write half of the output columns each
        {
            {
                const float inv = st_m[r];
                const int e_row0 = meta[0], e_lo = meta[1], e_hi = meta[2];
                const bool valid = (r >= e_lo) && (r < e_hi);
                const long long orow = (static_cast<long long>(e_row0) + r) * p.Hq + head;
                __nv_bfloat16* optr = reinterpret_cast<__nv_bfloat16*>(p.o) + orow * D + DH * wg;
                const bool full_tile = e_lo == 0 && e_hi == 128;
                uint8_t* stage = smem + L::OFF_Q;            // the query tile is no longer needed
#pragma unroll
                for (int cc = 0; cc < DH / 32; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(tlane + COL_OA + DH * wg + 32 * cc, v);
                    tmem_wait_ld();
                    uint32_t o16[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        o16[i] = pack_bf16x2(finalize_o(__uint_as_float(v[2 * i]), inv),
                                             finalize_o(__uint_as_float(v[2 * i + 1]), inv));
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint4 val = make_uint4(o16[4 * i], o16[4 * i + 1], o16[4 * i + 2], o16[4 * i + 3]);
                        if (full_tile) {
                            const int c16 = (DH * wg) / 8 + 4 * cc + i;     // 16-byte chunk of the row
                            *reinterpret_cast<uint4*>(stage + (c16 >> 3) * L::ATOM + r * 128 + (((c16 & 7) ^ (r & 7)) << 4)) = val;
                        } else if (valid) {
                            reinterpret_cast<uint4*>(optr + 32 * cc)[i] = val;
                        }
                    }
                }
                if (full_tile) {
                    // a complete tile leaves through shared memory and one tiled TMA store
                    fence_proxy_async_smem();
                    named_bar_sync(1, 256);
                    if (warp == 4 && lane == 0) {
                        for (int a = 0; a < NATOM; ++a)
                            tma_store_3d(&p.tmO, smem_u32(stage) + a * L::ATOM, a * 64, head, e_row0);
                        tma_store_commit();
                        tma_store_wait_read();
                    }
                }
            }
        }
        }
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

// ------------------------------------------------------------------ split-KV combine
// One block per (sequence, query head), one thread per head_dim column; folds the chunk
// partials (m, l_lo, l_hi, O) in ascending chunk order and normalises.
template <int D>
__global__ void __launch_bounds__(D) combine_kernel(const AttnParams p) {
    pdl_wait();                        // the decode kernel's partials are complete and visible
    const int b = blockIdx.x / p.Hq;
    const int ctx = min(p.ctx_lens[b], p.max_ctx);     // as the decode kernel: never beyond the host's bound
    if (ctx <= 0) return;
    const int nc = (ctx + CHUNK - 1) / CHUNK;
    const long long slot0 = static_cast<long long>(blockIdx.x) * p.nchunk_max;
    const int col = threadIdx.x;
    float M = p.part_ml[4 * slot0], L_lo = p.part_ml[4 * slot0 + 1], L_hi = p.part_ml[4 * slot0 + 2];
    float O = p.part_o[slot0 * D + col];
    for (int ch = 1; ch < nc; ++ch) {
        const float* ml = p.part_ml + 4 * (slot0 + ch);
        const float o_c = p.part_o[(slot0 + ch) * D + col];
        const FoldCoef f = fold_coef(M, ml[0], p.c);
        L_lo = fold_value(L_lo, ml[1], f);
        L_hi = fold_value(L_hi, ml[2], f);
        O = fold_value(O, o_c, f);
        M = f.M_new;
    }
    const float Ltot = finalize_l(L_lo, L_hi);
    const float inv = finalize_inv(Ltot);
    reinterpret_cast<__nv_bfloat16*>(p.o)[static_cast<long long>(blockIdx.x) * D + col] =
        __float2bfloat16_rn(finalize_o(O, inv));
    if (p.lse && col == 0) p.lse[blockIdx.x] = finalize_lse(M, Ltot, p.c);
}

// ------------------------------------------------------------------ KV-cache write
// A block copies KVW_TOK (8 or 1) consecutive new tokens (K and V rows of all KV heads: 16-byte vectors).
// Threads 0 .. KVW_TOK-1 find their token's sequence (binary search over cu_new), position and
// physical page; then all threads copy, every thread's loads issued before its stores.  (One token
// per 128-thread block, each doing its own search before 32 bytes of copying per thread, reached
// 0.76 of the copy bandwidth.)
constexpr int KVW_THREADS = 256;
template <int KVW_TOK>       // 8 for prompts, 1 for a decode step's handful of tokens (more blocks, shorter chains)
__global__ void __launch_bounds__(KVW_THREADS)
kv_write_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                const int32_t* __restrict__ cu_new, const int32_t* __restrict__ ctx_lens,
                uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                const int32_t* __restrict__ block_table, int max_blocks, int S, long long total_new, int Hkv,
                int vec_per_head /* d*2/16 */, int page_size, int num_pages, int* dev_status) {
    pdl_launch_dependents();       // an attention kernel launched next may be scheduled behind this grid
    __shared__ long long dst_base[KVW_TOK];     // vector index of (page, head 0, row, 0), or -1
    const long long tok0 = static_cast<long long>(blockIdx.x) * KVW_TOK;
    if (threadIdx.x < KVW_TOK) {
        const long long token = tok0 + threadIdx.x;
        long long base = -1;
        if (token < total_new) {
            int lo = 0, hi = S;            // find s with cu_new[s] <= token < cu_new[s+1]
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (cu_new[mid] <= token) lo = mid; else hi = mid;
            }
            const int s = lo;
            const int n_s = cu_new[s + 1] - cu_new[s];
            const int pos = ctx_lens[s] - n_s + static_cast<int>(token - cu_new[s]);
            if (token < cu_new[s + 1] && pos >= 0) {
                const int lp = pos / page_size, row = pos % page_size;
                const int phys = (lp < max_blocks) ? block_table[static_cast<long long>(s) * max_blocks + lp] : -1;
                if (phys < 0 || phys >= num_pages) atomicOr(dev_status, TIK_DEV_BAD_BLOCK);
                else base = (static_cast<long long>(phys) * Hkv * page_size + row) * vec_per_head;
            }
        }
        dst_base[threadIdx.x] = base;
    }
    __syncthreads();
    const int nvec = Hkv * vec_per_head;                 // vectors per token and tensor
    const int per_block = KVW_TOK * nvec;
    const long long head_pitch = static_cast<long long>(page_size) * vec_per_head;
    for (int i0 = threadIdx.x; i0 < per_block; i0 += 4 * KVW_THREADS) {
        uint4 kv[4], vv[4];
        long long dst[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * KVW_THREADS;
            dst[u] = -1;
            if (i < per_block) {
                const int j = i / nvec, r = i - j * nvec;          // token of the block, vector of the token
                const long long base = dst_base[j];
                if (base >= 0) {
                    const int hh = r / vec_per_head, e = r - hh * vec_per_head;
                    dst[u] = base + hh * head_pitch + e;
                    const long long src = (tok0 + j) * nvec + r;
                    kv[u] = k_new[src];
                    vv[u] = v_new[src];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (dst[u] >= 0) {
                k_cache[dst[u]] = kv[u];
                v_cache[dst[u]] = vv[u];
            }
    }
}

// ------------------------------------------------------------------ launchers
template <int D, int MODE>
static cudaError_t launch_attn_t(dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                                 const CUtensorMap& tmV, const AttnParams& p, cudaStream_t stream) {
    auto kern = attn_kernel<D, MODE>;
    // The opt-in to more than 48 KiB of dynamic shared memory belongs to the (function, device)
    // pair: one flag per device that has launched this instantiation.
    static DeviceOnce configured;
    cudaError_t e = configured.run([&]() {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(AttnSmem<D>::ALLOC));
    });
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(ATTN_THREADS);
    cfg.dynamicSmemBytes = AttnSmem<D>::ALLOC;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, p);
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
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(B) * p.Hq);
    cfg.blockDim = dim3(d);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();  // exactly one of the launches below runs
    if (d == 128) return cudaLaunchKernelEx(&cfg, combine_kernel<128>, p);
    return cudaLaunchKernelEx(&cfg, combine_kernel<64>, p);
}

cudaError_t launch_kv_write(const void* k_new, const void* v_new, const int32_t* cu_new,
                            const int32_t* ctx_lens, void* k_cache, void* v_cache,
                            const int32_t* block_table, int max_blocks, int S, int64_t total_new,
                            int Hkv, int d, int page_size, int num_pages, int* dev_status,
                            cudaStream_t stream) {
    if (total_new <= 0) return cudaSuccess;
    count_launch();  // exactly one of the launches below runs
    if (total_new >= 4096)
        kv_write_kernel<8><<<static_cast<unsigned>((total_new + 7) / 8), KVW_THREADS, 0, stream>>>(
            static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), cu_new, ctx_lens,
            static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), block_table, max_blocks, S, total_new, Hkv,
            d * 2 / 16, page_size, num_pages, dev_status);
    else
        kv_write_kernel<1><<<static_cast<unsigned>(total_new), KVW_THREADS, 0, stream>>>(
            static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), cu_new, ctx_lens,
            static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), block_table, max_blocks, S, total_new, Hkv,
            d * 2 / 16, page_size, num_pages, dev_status);
    return cudaGetLastError();
}

}  // namespace tik
