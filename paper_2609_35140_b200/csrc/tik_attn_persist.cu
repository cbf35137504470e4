// Full-sequence attention (packed train-forward, paged prefill) as a persistent kernel.
//
// The arithmetic, the tile and chunk structure and the roles are those of attn_kernel
// (tik_attn.cu): one CTA per SM, two TMA warps (Q + K, V), two MMA-issuing threads (QK^T, PV),
// two softmax warpgroups, S / P / O in tensor memory.  What differs is the schedule.  There a CTA
// is one work item -- a pair of query tiles 2m, 2m+1 (tiles 0..15) or one query tile >= 16 of one
// (sequence, head) -- and pays entry, first-data latency, epilogue and exit for each (~8 700 clk
// beside ~1 560 clk per (query tile, KV tile) step).  Here a CTA walks a list of items and every
// role runs ahead into the next item on its own:
//   * a small planning kernel compacts the valid (sequence, item) pairs of the call into a list,
//     sequence by sequence, each sequence's heaviest items first; CTA c takes list positions c,
//     2n-1-c, 2n+c, ... (n CTAs) for every query head: CTAs that run together share a sequence's
//     K/V in L2, and each CTA meets every weight class;
//   * all ring, score and weight barriers count across items (stage = tile count & 1, buffer =
//     step count & 1), so the K / V producers refill the rings with the next item's first tiles
//     while the current item's last steps run;
//   * the two query-tile slots alternate: the slot that frees first (tile A's, one step before the
//     end) receives the next item's first tile, released by a commit of the last QK^T that read it;
//   * finished tiles leave through a staging buffer of their own (16 KiB per warpgroup), not
//     through the query slots;
//   * a warpgroup belongs to the steps whose global index has its parity, so the warpgroup that
//     finished first in one item (odd item lengths) takes the first step of the next.
// A row's arithmetic is untouched: same tiles, same order, same instructions, hence same bits.
#include "tik_core.cuh"
#include "tik_internal.h"
#include "tik_ptx.cuh"

namespace tik {

constexpr int PA_THREADS = 384;   // warp 0 TMA (Q, K), warp 1 QK^T MMA, warp 2 TMA (V), warp 3 PV MMA, warps 4-11 softmax

template <int D>
struct PASmem {
    static constexpr uint32_t ATOM = 128 * 128;          // 128 rows x 64 bf16
    static constexpr uint32_t TILE = (D / 64) * ATOM;    // one Q, K or V tile
    static constexpr uint32_t OFF_Q = 0;                 // two query-tile slots
    static constexpr uint32_t OFF_K = 2 * TILE;          // two K stages
    static constexpr uint32_t OFF_V = 4 * TILE;          // two V stages
    static constexpr uint32_t OFF_STAGE = 6 * TILE;      // output staging: one atom per warpgroup
    static constexpr uint32_t OFF_BAR = OFF_STAGE + 2 * ATOM;
    static constexpr uint32_t OFF_LX = OFF_BAR + 320;    // 5 x 128 floats of row state
    static constexpr uint32_t BYTES = OFF_LX + 5 * 512;
};

// Event trace of one CTA (debug builds only, -DTIK_PA_TRACE): clock64 stamps of the roles' key
// events for the CTA's first items, read back through tik_debug_pa_trace.
#ifdef TIK_PA_TRACE
constexpr int PA_TRACE_ITEMS = 48, PA_TRACE_EVENTS = 48;
__device__ long long g_pa_trace[PA_TRACE_ITEMS * PA_TRACE_EVENTS];
#define PA_STAMP(k, ev)                                                                         \
    do {                                                                                        \
        if (blockIdx.x == 0 && (k) < PA_TRACE_ITEMS) g_pa_trace[(k) * PA_TRACE_EVENTS + (ev)] = clock64(); \
    } while (0)
#define PA_TAG(site) pa_tag = (site)
#define PA_AUX(v) pa_aux = static_cast<int>(v)
__device__ int g_pa_tags[148 * 12 * 2];
// per-step stamps of the first 8 items of CTA 0: [item][role: 0 QK issuer, 1 PV issuer, 2 / 3 warpgroups][step < 16][event < 8]
__device__ long long g_pa_steps[8 * 4 * 16 * 8];
#define PA_SSTAMP(k, role, g, ev)                                                               \
    do {                                                                                        \
        if (blockIdx.x == 0 && (k) < 8 && (g) < 16)                                             \
            g_pa_steps[(((k) * 4 + (role)) * 16 + (g)) * 8 + (ev)] = clock64();                  \
    } while (0)
#else
#define PA_SSTAMP(k, role, g, ev) do { } while (0)
#define PA_STAMP(k, ev) do { } while (0)
#define PA_TAG(site) do { } while (0)
#define PA_AUX(v) do { } while (0)
#endif
// a bounded barrier wait; `site` numbers the wait for the debug build's "where did it stop" record
#define PA_WAIT(site, ...)        \
    do {                          \
        PA_TAG(site);             \
        mbar_wait(__VA_ARGS__);   \
    } while (0)

__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}

// ------------------------------------------------------------------ planning kernel
// Candidate items of a sequence: x < 8 is the pair of query tiles (2x, 2x+1), x >= 8 the single
// tile 16 + (x - 8).  A sequence whose new rows cover tiles t_lo..t_hi has the candidates
// f(t_lo)..f(t_hi), f(t) = t < 16 ? t / 2 : t - 8.
__device__ __forceinline__ int plan_x_of_tile(int t) { return t < 16 ? (t >> 1) : (t - 8); }

struct PlanSeq {
    int qb, ctx, pos0, xlo, xhi;     // xhi < xlo: nothing to do
};
__device__ __forceinline__ PlanSeq plan_seq(const int32_t* cu, const int32_t* ctx_lens, int s) {
    PlanSeq q;
    q.qb = cu[s];
    const int qlen = cu[s + 1] - q.qb;
    q.ctx = ctx_lens ? ctx_lens[s] : qlen;
    q.pos0 = q.ctx - qlen;
    if (qlen <= 0 || q.pos0 < 0) {
        q.xlo = 1;
        q.xhi = 0;
    } else {
        q.xlo = plan_x_of_tile(q.pos0 >> 7);
        q.xhi = plan_x_of_tile((q.ctx - 1) >> 7);
    }
    return q;
}

constexpr int PLAN_XMAX = 4096;

// One block.  Output: plan[0].x = number of entries; plan[1 + i] = (seq | x << 16, first query
// row, context length, position of the first query row).  Order: sequences ascending, and within a
// sequence x descending (its heaviest items first).  CTAs that run at the same time then work on
// the same one or two sequences, whose K/V stay in L2 (an order by weight across all sequences
// touched every sequence's K/V at once: a third slower on sixteen 16 K-token sequences), while
// every CTA still meets every weight class, because the weights repeat sequence by sequence.
// x_max: only candidates x <= x_max are listed (7: the paired items and partner-less tiles below 16).
__global__ void __launch_bounds__(1024) attn_plan_kernel(const int32_t* __restrict__ cu,
                                                         const int32_t* __restrict__ ctx_lens, int S, int x_max,
                                                         int4* __restrict__ plan) {
    pdl_wait();
    pdl_launch_dependents();
    __shared__ int warp_sums[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // thread t owns the sequences [t * per, t * per + per)
    const int per = (S + 1023) / 1024;
    const int s_lo = threadIdx.x * per, s_hi = min(S, s_lo + per);
    int mine = 0;
    for (int s = s_lo; s < s_hi; ++s) {
        const PlanSeq q = plan_seq(cu, ctx_lens, s);
        const int hi = min(q.xhi, x_max);
        if (hi >= q.xlo) mine += hi - q.xlo + 1;
    }
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += n;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sums[lane], wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, wi, off);
            if (lane >= off) wi += n;
        }
        warp_sums[lane] = wi - w;           // exclusive prefix of the warps
        if (lane == 31) plan[0] = make_int4(wi, 0, 0, 0);
    }
    __syncthreads();
    int run = warp_sums[warp] + incl - mine;
    for (int s = s_lo; s < s_hi; ++s) {
        const PlanSeq q = plan_seq(cu, ctx_lens, s);
        for (int x = min(q.xhi, x_max); x >= q.xlo; --x) plan[1 + run++] = make_int4(s | (x << 16), q.qb, q.ctx, q.pos0);
    }
}

// ------------------------------------------------------------------ work items
struct PAItem {
    int seq, head, ctx, pos0, qb;
    int T0, T1;          // query tile of local parity 0 (B, or the single tile) and of parity 1 (A = T0 - 1)
    bool pair;
    int n_tiles, n_steps;
};
__device__ __forceinline__ PAItem pa_decode(const int4 e, int head) {
    PAItem it;
    it.seq = e.x & 0xffff;
    const int x = static_cast<int>(static_cast<unsigned>(e.x) >> 16);
    it.head = head;
    it.qb = e.y;
    it.ctx = e.z;
    it.pos0 = e.w;
    const int t_lo = it.pos0 >> 7, t_hi = (it.ctx - 1) >> 7;
    if (x >= 8) {
        it.T0 = 16 + (x - 8);
        it.T1 = 0;
        it.pair = false;
    } else {
        const int ta = 2 * x, tb = 2 * x + 1;
        const bool va = ta >= t_lo && ta <= t_hi, vb = tb >= t_lo && tb <= t_hi;
        it.pair = va && vb;
        it.T0 = vb ? tb : ta;
        it.T1 = ta;
    }
    it.n_tiles = it.T0 + 1;
    it.n_steps = it.pair ? (2 * it.n_tiles - 1) : it.n_tiles;
    return it;
}

// Rarely taken paths of the softmax loops, out of line (as in attn_kernel).
template <int D>
__device__ __noinline__ void pa_rescale_o_tmem(uint32_t to, float alpha) {
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
__device__ __noinline__ void pa_fold_o_tmem(uint32_t t_a, uint32_t t_b, FoldCoef f) {
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

// Epilogue of one warp: NCOLS accumulator columns of its 32 rows (one row per lane), scaled by the
// row's reciprocal, rounded to bf16 and written to o[row][head][col0 ...].  A lane's row is 128
// (or 64) bytes of a different 128-byte line than its neighbours', so the rows go through a
// warp-private staging area and leave as whole rows: eight (four) lanes per row and store
// instruction.  Only __syncwarp is needed, no CTA barrier, no asynchronous copy to wait for; rows
// outside [lo, hi) are skipped, which also serves ragged tiles.  After the last accumulator load
// the warp arrives `odrain_n` times on `odrain_bar`: the accumulator may be overwritten.
template <int NCOLS>
__device__ __noinline__ void pa_store_rows(uint32_t acc, float inv, int row0, int lo, int hi, int head, int col0, int D,
                                           uint8_t* stage, __nv_bfloat16* o, int Hq, uint32_t odrain_bar,
                                           uint32_t odrain_n, int lane, int quarter, const CUtensorMap* tmo,
                                           long long* tr = nullptr) {
    constexpr int PASS = NCOLS < 64 ? NCOLS : 64;      // columns per pass
    constexpr int NCH = PASS / 8;                       // 16-byte chunks per row and pass
    constexpr int RPI = 32 / NCH;                       // rows per store instruction
    // A whole tile (all 128 rows belong to the item) with 128-byte staging rows leaves through one
    // tiled bulk store of 32 rows x 64 columns per warp and pass: the staging layout is the 128-byte
    // swizzle of the copy engine, lane 0 owns the warp's bulk groups, and the warp goes on as soon
    // as the store is issued.  The staging buffer is written again only after lane 0 has seen the
    // previous group's read of it complete -- for the second pass that wait hides behind the pass's
    // own accumulator load and packing.
    const bool bulk = PASS == 64 && tmo != nullptr && lo <= 0 && hi >= 128;
#pragma unroll 1
    for (int a = 0; a < NCOLS / PASS; ++a) {
        uint32_t v[PASS];
#pragma unroll
        for (int cc = 0; cc < PASS / 32; ++cc)
            tmem_ld32(acc + PASS * a + 32 * cc, *reinterpret_cast<uint32_t(*)[32]>(&v[32 * cc]));
        tmem_wait_ld();
        if (tr) tr[3 * a] = clock64();
        if (a == NCOLS / PASS - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_n(odrain_bar, odrain_n);
        }
        if (bulk) {
            uint32_t w[PASS / 2];
#pragma unroll
            for (int i = 0; i < PASS / 2; ++i)
                w[i] = pack_bf16x2(finalize_o(__uint_as_float(v[2 * i]), inv), finalize_o(__uint_as_float(v[2 * i + 1]), inv));
            if (lane == 0) tma_store_wait_read();
            __syncwarp();
#pragma unroll
            for (int i = 0; i < NCH; ++i)
                *reinterpret_cast<uint4*>(stage + lane * 128 + ((i ^ (lane & 7)) << 4)) =
                    make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                tma_store_3d(tmo, smem_u32(stage), col0 + PASS * a, head, row0 + 32 * quarter);
                tma_store_commit();
            }
            if (tr) tr[3 * a + 1] = tr[3 * a + 2] = clock64();
            continue;
        }
        if (lane == 0) tma_store_wait_read();       // an earlier whole tile may still be leaving the buffer
        __syncwarp();
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            uint32_t w4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w4[j] = pack_bf16x2(finalize_o(__uint_as_float(v[8 * i + 2 * j]), inv),
                                    finalize_o(__uint_as_float(v[8 * i + 2 * j + 1]), inv));
            *reinterpret_cast<uint4*>(stage + lane * (NCH * 16) + ((i ^ (lane & (NCH - 1))) << 4)) =
                make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        __syncwarp();
        if (tr) tr[3 * a + 1] = clock64();
        const int cl = lane % NCH, r0 = lane / NCH;
        uint4 val[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int row = r0 + RPI * i;               // row of this warp's 32
            val[i] = *reinterpret_cast<const uint4*>(stage + row * (NCH * 16) + ((cl ^ (row & (NCH - 1))) << 4));
        }
        // all rows are read back before the first store is issued (the compiler cannot move a shared
        // load across a global store on its own)
        __nv_bfloat16* const gp = o + (static_cast<long long>(row0 + 32 * quarter + r0) * Hq + head) * D + col0 + PASS * a + cl * 8;
        const long long pitch = static_cast<long long>(RPI) * Hq * D;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int trow = 32 * quarter + r0 + RPI * i;        // row of the tile
            if (trow >= lo && trow < hi) *reinterpret_cast<uint4*>(gp + i * pitch) = val[i];
        }
        __syncwarp();
        if (tr) tr[3 * a + 2] = clock64();
    }
}

template <int D, bool PAGED>
__global__ void __launch_bounds__(PA_THREADS, 1)
attn_persist_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnParams p,
                    const int4* __restrict__ plan) {
    using L = PASmem<D>;
    constexpr int NATOM = D / 64;
    constexpr int DH = D / 2;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0;                          // one score buffer of 128 columns
    constexpr uint32_t COL_P = 128;                        // two weight buffers of 64 columns (bf16 pairs)
    constexpr uint32_t COL_OA = 256, COL_OB = 256 + D;
    constexpr uint32_t IDESC_QK = mma_idesc_bf16(128, 128, false);
    constexpr uint32_t IDESC_PV = mma_idesc_bf16(128, D, true);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef TIK_PA_TRACE
    int pa_tag = 0, pa_aux = 0;
#endif

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    const uint32_t sbase = smem_u32(smem_raw);
    if (sbase & 1023u) {     // the swizzled tiles need a 1 KiB aligned base: refuse to run otherwise
        if (tid == 0) atomicOr(p.dev_status, TIK_DEV_WAIT_EXPIRED);
        return;
    }
    const uint32_t sQ = sbase + L::OFF_Q, sK = sbase + L::OFF_K, sV = sbase + L::OFF_V;
    const uint32_t bar0 = sbase + L::OFF_BAR;
    const uint32_t bar_qfull = bar0;             // [2] query tile landed in slot
    const uint32_t bar_qempty = bar0 + 16;       // [2] last QK^T that read the slot is done
    const uint32_t bar_kfull = bar0 + 32;        // [2]
    const uint32_t bar_kempty = bar0 + 48;       // [2]
    const uint32_t bar_vfull = bar0 + 64;        // [2]
    const uint32_t bar_vempty = bar0 + 80;       // [2]
    const uint32_t bar_sfull = bar0 + 96;        // [2] scores of an even / odd global step ready
    const uint32_t bar_pfull = bar0 + 112;       // [2] weights written (4 warps)
    const uint32_t bar_pempty = bar0 + 128;      // [2] PV done
    const uint32_t bar_sempty = bar0 + 144;      // [2] scores are in registers (4 warps)
    const uint32_t bar_hand = bar0 + 160;        // [4] reference-maximum hand-off (single mode)
    const uint32_t bar_odrain = bar0 + 192;      // [2] accumulator read out by the epilogue (8 arrivals)
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_BAR + 208);
    volatile int* abort_word = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 212);
    // epilogue values (first output row, valid rows, head), double-buffered by item parity: a warp
    // cannot fall two items behind its warpgroup (every step needs all four warps' arrivals)
    volatile int* meta_pair = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 216);      // [2][2][4]
    volatile int* meta_single = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 280);    // [2][4]
    float* lx = reinterpret_cast<float*>(smem + L::OFF_LX);

    // ---------------------------------------------------------------- set-up (before the grid dependency resolves)
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        for (int i = 0; i < 26; ++i) {
            // counts: hand 1, pfull / sempty 4 (one per warp), odrain 8, everything else 1
            const uint32_t b = bar0 + 8 * i;
            uint32_t count = 1;
            if ((b >= bar_pfull && b < bar_pempty) || (b >= bar_sempty && b < bar_hand)) count = 4;
            if (b >= bar_odrain) count = 8;
            mbar_init(b, count);
        }
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    }
    // the plan (and every input) is complete from here on.  Launched behind the single-tile grid
    // (wait_at_end) this grid starts once every CTA of that grid has started, which is after the
    // plan completed, and must not wait for that grid here: it is there to fill its tail.
    if (!p.wait_at_end) pdl_wait();
    if (warp == 3 && lane == 0) {
        // an earlier kernel on this context may have run out of a wait: then do nothing at all
        *abort_word = (*reinterpret_cast<volatile int*>(p.dev_status) & TIK_DEV_WAIT_EXPIRED) ? 1 : 0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // (plan entries are read around L1: a line of an earlier call's plan may still sit there)
    const unsigned n_items = static_cast<unsigned>(__ldcg(&plan[0]).x) * static_cast<unsigned>(p.Hq);   // < 2^31 (host check)
    const unsigned ncta = gridDim.x, cta = blockIdx.x;
    // list position of this CTA's k-th item (rounds alternate direction)
    auto item_index = [&](int k) -> unsigned {
        return static_cast<unsigned>(k) * ncta + ((k & 1) ? (ncta - 1 - cta) : cta);
    };
    auto load_entry = [&](unsigned i, int& head) -> int4 {
        const unsigned idx = i / static_cast<unsigned>(p.Hq);
        head = static_cast<int>(i - idx * static_cast<unsigned>(p.Hq));
        return __ldcg(&plan[1 + idx]);
    };
    // warp-uniform view of the CTA's abort flag (full warps must leave their loops together)
    auto aborted_warp = [&]() -> bool { return __any_sync(0xffffffffu, *abort_word != 0) != 0; };

    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    if (warp == 0 || warp == 2) {
        // ------------------------------------------------------------ TMA producers
        // warp 0: query tiles and K tiles; warp 2: V tiles.  Paged: the whole warp works (one
        // block-table entry per lane, lane i issues the copies of a tile's i-th page); packed: lane 0.
        const int kv = (warp == 2) ? 1 : 0;
        const CUtensorMap* tm = kv ? &tmV : &tmK;
        if (PAGED || lane == 0) {
            uint32_t tcnt = 0;                  // K (V) tiles produced so far, across items
            uint32_t qcnt0 = 0, qcnt1 = 0;      // loads issued into each query slot so far
            int sB = 0;                         // slot of the current item's tile B
            int head = 0, head_n = 0;
            int4 e = make_int4(0, 0, 0, 0), e_n = e;
            if (item_index(0) < n_items) e_n = load_entry(item_index(0), head_n);
            for (int k = 0;; ++k) {
                if (item_index(k) >= n_items || (PAGED ? aborted_warp() : (*abort_word != 0))) break;
                e = e_n;
                head = head_n;
                const bool more = item_index(k + 1) < n_items;
                if (more) e_n = load_entry(item_index(k + 1), head_n);
                const PAItem it = pa_decode(e, head);
                const int kvh = head / p.G;
                if (kv == 0 && lane == 0 && more) {
                    // the next item's query tiles go to L2 now: when their slots free up, at the
                    // end of this item, the loads no longer wait for DRAM
                    const PAItem nx = pa_decode(e_n, head_n);
                    for (int q2 = 0; q2 < (nx.pair ? 2 : 1); ++q2) {
                        const int row = nx.qb + 128 * (q2 ? nx.T1 : nx.T0) - nx.pos0;
                        for (int a = 0; a < NATOM; ++a) tma_prefetch_l2_3d(&tmQ, a * 64, head_n, row);
                    }
                }
                auto load_q = [&](int q2) {      // lane 0 of warp 0: tile B (q2 = 0) or A (q2 = 1)
                    const int slot = sB ^ q2;
                    const uint32_t used = slot ? qcnt1 : qcnt0;
                    if (used > 0) PA_WAIT(1, bar_qempty + 8 * slot, (used - 1) & 1, abort_word, p.dev_status);
                    if (slot) ++qcnt1; else ++qcnt0;
                    if (lane == 0) {
                        mbar_expect_tx(bar_qfull + 8 * slot, L::TILE);
                        const int row = it.qb + 128 * (q2 ? it.T1 : it.T0) - it.pos0;
                        for (int a = 0; a < NATOM; ++a)
                            tma_load_3d(sQ + slot * L::TILE + a * L::ATOM, &tmQ, bar_qfull + 8 * slot, a * 64, head, row);
                    }
                };
                int my_phys = p.num_pages;
                auto produce_tile = [&](int j) {
                    const int st = tcnt & 1;
                    const uint32_t dst = (kv ? sV : sK) + st * L::TILE;
                    const uint32_t full = (kv ? bar_vfull : bar_kfull) + 8 * st;
                    int my_page = 0;
                    if (PAGED) {
                        const int tpb_mask = (32 >> p.ppt_shift) - 1;             // tiles per block-table batch - 1
                        if ((j & tpb_mask) == 0) {
                            const int lp = ((128 * j) >> p.page_shift) + lane;
                            int ph = p.num_pages;       // out of range: the box is filled with zeros
                            if ((lp << p.page_shift) < it.ctx) {
                                ph = (lp < p.max_blocks) ? p.block_table[static_cast<long long>(it.seq) * p.max_blocks + lp] : -1;
                                if (ph < 0 || ph >= p.num_pages) {
                                    if (kv == 0) atomicOr(p.dev_status, TIK_DEV_BAD_BLOCK);
                                    ph = p.num_pages;
                                }
                            }
                            my_phys = ph;
                        }
                        const int in_batch = j & tpb_mask;
                        my_page = __shfl_sync(0xffffffffu, my_phys, (in_batch << p.ppt_shift) + (lane & (p.pages_per_tile - 1)));
                    }
                    if (tcnt >= 2)
                        PA_WAIT(2, (kv ? bar_vempty : bar_kempty) + 8 * st, ((tcnt >> 1) - 1) & 1, abort_word, p.dev_status);
                    ++tcnt;
                    if (lane == 0) mbar_expect_tx(full, L::TILE);
                    if (!PAGED) {
                        const int row = it.qb + 128 * j;          // packed K/V rows of the sequence start at its first token
                        for (int a = 0; a < NATOM; ++a) tma_load_3d(dst + a * L::ATOM, tm, full, a * 64, kvh, row);
                    } else {
                        __syncwarp();                             // the expected byte count is registered first
                        if (lane < p.pages_per_tile) {
                            const uint32_t off = static_cast<uint32_t>(lane << p.page_shift) * 128u;
                            for (int a = 0; a < NATOM; ++a)
                                tma_load_4d(dst + a * L::ATOM + off, tm, full, a * 64, 0, kvh, my_page);
                        }
                    }
                };
                // order of need: tile B, K tile 0, tile A, K tile 1, ...
                if (kv == 0) load_q(0);
                produce_tile(0);
                if (kv == 0 && it.pair) load_q(1);
                for (int j = 1; j < it.n_tiles; ++j) {
                    if (PAGED ? aborted_warp() : (*abort_word != 0)) break;
                    produce_tile(j);
                }
                sB ^= 1;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ QK^T issuer
        if (lane == 0) {
            uint32_t Gs = 0, kbase = 0;
            uint32_t qcnt0 = 0, qcnt1 = 0;
            int sB = 0;
            int head = 0, head_n = 0;
            int4 e = make_int4(0, 0, 0, 0), e_n = e;
            if (item_index(0) < n_items) e_n = load_entry(item_index(0), head_n);
            for (int k = 0;; ++k) {
                if (item_index(k) >= n_items || *abort_word) break;
                e = e_n;
                head = head_n;
                if (item_index(k + 1) < n_items) e_n = load_entry(item_index(k + 1), head_n);
                const PAItem it = pa_decode(e, head);
                const uint64_t dqB = smem_desc_sw128(sQ + sB * L::TILE, 0, 1024);
                const uint64_t dqA = smem_desc_sw128(sQ + (sB ^ 1) * L::TILE, 0, 1024);
                for (int g = 0; g < it.n_steps; ++g) {
                    PA_AUX(Gs | (k << 20));
                    const int kt = it.pair ? (g >> 1) : g;
                    const bool tileA = it.pair && (g & 1);
                    const uint32_t kc = kbase + kt;
                    const int st = kc & 1;
                    if (g == 0) PA_STAMP(k, 0);
                    if (g == 0 || (it.pair && g == 1)) {          // first use of this query tile
                        const int slot = tileA ? (sB ^ 1) : sB;
                        PA_WAIT(3, bar_qfull + 8 * slot, (slot ? qcnt1 : qcnt0) & 1, abort_word, p.dev_status);
                        if (slot) ++qcnt1; else ++qcnt0;
                    }
                    if (g == 0) PA_STAMP(k, 1);
                    PA_WAIT(4, bar_kfull + 8 * st, (kc >> 1) & 1, abort_word, p.dev_status);
                    if (g == 0) PA_STAMP(k, 2);
                    PA_SSTAMP(k, 0, g, 0);
                    // the single score buffer is free once the softmax of the previous step holds it in registers
                    if (Gs >= 1) PA_WAIT(5, bar_sempty + 8 * ((Gs - 1) & 1), ((Gs - 1) >> 1) & 1, abort_word, p.dev_status);
                    if (g == 0) PA_STAMP(k, 3);
                    if (g == 1) PA_STAMP(k, 4);
                    if (g == it.n_steps - 1) PA_STAMP(k, 5);
                    tc_fence_after();
                    PA_SSTAMP(k, 0, g, 1);
                    const uint64_t dk = smem_desc_sw128(sK + st * L::TILE, 0, 1024);
                    if (D == 128) mma_ss_chain8_fresh(tmem + COL_S, tileA ? dqA : dqB, dk, IDESC_QK);
                    else mma_ss_chain4_fresh(tmem + COL_S, tileA ? dqA : dqB, dk, IDESC_QK);
                    mma_commit(bar_sfull + 8 * (Gs & 1));
                    // the K stage is free after its last reader (paired: the odd step, or B's last tile)
                    if (!it.pair || (g & 1) || g == it.n_steps - 1) mma_commit(bar_kempty + 8 * st);
                    // so is the query slot: A's last step is n_steps - 2, B's (and a single tile's) the last
                    if (g == it.n_steps - 1) mma_commit(bar_qempty + 8 * sB);
                    else if (it.pair && g == it.n_steps - 2) mma_commit(bar_qempty + 8 * (sB ^ 1));
                    PA_SSTAMP(k, 0, g, 2);
                    ++Gs;
                }
                kbase += it.n_tiles;
                sB ^= 1;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ PV issuer
        if (lane == 0) {
            uint32_t Gs = 0, vbase = 0;
            uint32_t drains0 = 0, drains1 = 0;  // epilogues that have read accumulator A / B so far
            int head = 0, head_n = 0;
            int4 e = make_int4(0, 0, 0, 0), e_n = e;
            if (item_index(0) < n_items) e_n = load_entry(item_index(0), head_n);
            for (int k = 0;; ++k) {
                if (item_index(k) >= n_items || *abort_word) break;
                e = e_n;
                head = head_n;
                if (item_index(k + 1) < n_items) e_n = load_entry(item_index(k + 1), head_n);
                const PAItem it = pa_decode(e, head);
                for (int g = 0; g < it.n_steps; ++g) {
                    PA_AUX(Gs | (k << 20));
                    const int vt = it.pair ? (g >> 1) : g;
                    const uint32_t vc = vbase + vt;
                    const int st = vc & 1, b = Gs & 1;
                    if (g == 0) PA_STAMP(k, 6);
                    PA_WAIT(6, bar_vfull + 8 * st, (vc >> 1) & 1, abort_word, p.dev_status);
                    if (g == 0) PA_STAMP(k, 7);
                    PA_SSTAMP(k, 1, g, 0);
                    PA_WAIT(7, bar_pfull + 8 * b, (Gs >> 1) & 1, abort_word, p.dev_status);
                    if (g == 0) PA_STAMP(k, 8);
                    if (g == it.n_steps - 1) PA_STAMP(k, 9);
                    // paired: the warpgroup of this step's parity accumulates its tile in its own accumulator;
                    // single: chunk 0 in O_A (the folded accumulator), later chunks in O_B
                    const int acc = it.pair ? b : ((g / TILES_PER_CHUNK) == 0 ? 0 : 1);
                    const bool fresh = it.pair ? (vt == 0) : ((g % TILES_PER_CHUNK) == 0);
                    const uint32_t drained = acc ? drains1 : drains0;
                    if ((it.pair ? (g < 2) : (g == 0)) && drained > 0)
                        PA_WAIT(8, bar_odrain + 8 * acc, (drained - 1) & 1, abort_word, p.dev_status);
                    tc_fence_after();
                    PA_SSTAMP(k, 1, g, 1);
                    mma_ts_chain8(tmem + (acc ? COL_OB : COL_OA), tmem + COL_P + 64 * b,
                                  smem_desc_sw128(sV + st * L::TILE, L::ATOM, 1024), IDESC_PV, fresh ? 0u : 1u);
                    mma_commit(bar_pempty + 8 * b);
                    if (!it.pair || (g & 1) || g == it.n_steps - 1) mma_commit(bar_vempty + 8 * st);
                    PA_SSTAMP(k, 1, g, 2);
                    ++Gs;
                }
                vbase += it.n_tiles;
                ++drains0;
                if (it.pair) ++drains1;
            }
        }
        __syncwarp();
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    {
        // ------------------------------------------------------------ softmax (two warpgroups)
        const int wg = (warp - 4) >> 2;
        const int quarter = warp & 3;                       // TMEM lane quarter of this warp
        const int r = quarter * 32 + lane;                  // tile row == TMEM lane
        const uint32_t tlane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const float c = p.c;
        float* st_m = lx;                 // [128]    running maximum of the current chunk
        float* st_l = lx + 128;           // [2][128] half row sums of the current chunk
        float* st_inv_all = lx + 384;     // [2][128] final reciprocal of a single item's rows, by item parity
        const uint32_t bar_m = bar_hand + 8 * quarter;
        const uint32_t ts = tlane + COL_S;
        const uint32_t tp = tlane + COL_P + 64 * wg;
        uint8_t* stage_warp = smem + L::OFF_STAGE + wg * L::ATOM + quarter * 4096;     // this warp's 4 KiB
        __nv_bfloat16* const o_base = reinterpret_cast<__nv_bfloat16*>(p.o);
        uint32_t Gs0 = 0;                 // global index of the current item's step 0
        uint32_t hc0 = 0;                 // single-mode steps of earlier items (hand-off barrier phase)

        // x: global step index
        auto wait_pv = [&](uint32_t x) {
            PA_WAIT(9, bar_pempty + 8 * (x & 1), (x >> 1) & 1, abort_word, p.dev_status);
            tc_fence_after();
        };
        auto wait_tile_done = [&](uint32_t x) {
            PA_WAIT(10, bar_pfull + 8 * (x & 1), (x >> 1) & 1, abort_word, p.dev_status);
        };

        int head = 0, head_n = 0;
        int4 e = make_int4(0, 0, 0, 0), e_n = e;
        if (item_index(0) < n_items) e_n = load_entry(item_index(0), head_n);
        for (int k = 0;; ++k) {
            if (item_index(k) >= n_items || aborted_warp()) break;
            e = e_n;
            head = head_n;
            if (item_index(k + 1) < n_items) e_n = load_entry(item_index(k + 1), head_n);
            const PAItem it = pa_decode(e, head);
            const int n_steps = it.n_steps;

            if (it.pair) {
                // ---- paired item: this warpgroup keeps the rows of one query tile through all of that
                // tile's KV tiles.  It owns the steps whose GLOBAL index has parity wg, i.e. the local
                // steps of parity lp: 0 -> tile B (T0, ends on its diagonal), 1 -> tile A (T1).
                const int lp = wg ^ static_cast<int>(Gs0 & 1);
                const int Tq = lp ? it.T1 : it.T0;
                const int qpos_p = 128 * Tq + r;
                const uint32_t to = tlane + (wg ? COL_OB : COL_OA);
                if (lane == 0) {           // every warp writes the same values and reads them after its own __syncwarp
                    volatile int* m = meta_pair + 8 * (k & 1) + 4 * wg;
                    m[0] = it.qb + 128 * Tq - it.pos0;
                    m[1] = max(0, it.pos0 - 128 * Tq);
                    m[2] = min(128, it.ctx - 128 * Tq);
                    m[3] = it.head;
                }
                __syncwarp();
                float m_run = -CUDART_INF_F, l_lo = 0.0f, l_hi = 0.0f;
                int g_last = lp;
                if (quarter == 0 && lane == 0) PA_STAMP(k, 10 + 10 * wg);
                for (int g = lp; g < n_steps; g += 2) {
                    g_last = g;
                    const uint32_t Gg = Gs0 + g;
                    PA_AUX(Gg | (k << 20));
                    const int j = g >> 1;
                    PA_WAIT(12, bar_sfull + 8 * wg, (Gg >> 1) & 1, abort_word, p.dev_status);
                    if (quarter == 0 && lane == 0 && g == lp) PA_STAMP(k, 11 + 10 * wg);
                    tc_fence_after();
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 0);
                    {
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
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 1);
                    if (kmax < 127) {
#pragma unroll
                        for (int i = 0; i < 128; ++i)
                            if (i > kmax) sc[i] = 0xff800000u;          // -inf
                    }
                    float mx[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) mx[q] = fmaxf(__uint_as_float(sc[2 * q]), __uint_as_float(sc[2 * q + 1]));
#pragma unroll
                    for (int i = 16; i < 128; i += 16) {
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            mx[q] = fmax3(mx[q], __uint_as_float(sc[i + 2 * q]), __uint_as_float(sc[i + 2 * q + 1]));
                    }
                    const float mt = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmax3(fmax3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
                    const float m_new = softmax_next_max(m_run, mt, c);
                    const float neg_mc = -__fmul_rn(m_new, c);
                    const float alpha = softmax_alpha(m_run, m_new, c);
                    m_run = m_new;
                    RowSum4 rs_lo, rs_hi;
                    rs_lo.reset();
                    rs_hi.reset();
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 2);
#pragma unroll
                    for (int i = 0; i < 64; i += 8) softmax_p8(&sc[i], c, neg_mc, rs_lo, &sc[i >> 1]);
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 3);
                    // The PV of this warpgroup's previous step (possibly the previous item's) read its weight
                    // buffer and updated its accumulator: waited for right before the first store.
                    if (Gg >= 2) wait_pv(Gg - 2);
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 4);
                    tmem_st32(tp, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
#pragma unroll
                    for (int i = 0; i < 64; i += 8) softmax_p8(&sc[64 + i], c, neg_mc, rs_hi, &sc[32 + (i >> 1)]);
                    tmem_st32(tp + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                    l_lo = __fmaf_rn(l_lo, alpha, rs_lo.total());
                    l_hi = __fmaf_rn(l_hi, alpha, rs_hi.total());
                    if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.0f)) pa_rescale_o_tmem<D>(to, alpha);
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 5);
                    tmem_wait_st();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_pfull + 8 * wg);
                    if (quarter == 0 && lane == 0) PA_SSTAMP(k, 2 + wg, g, 6);
                }
                // ---- this tile is complete after its last PV: normalise and store its rows
                if (quarter == 0 && lane == 0) PA_STAMP(k, 12 + 10 * wg);
                wait_pv(Gs0 + g_last);
                if (quarter == 0 && lane == 0) PA_STAMP(k, 13 + 10 * wg);
                if (!aborted_warp()) {       // after an expired wait the row state may be garbage: store nothing
                    const float Ltot = finalize_l(l_lo, l_hi);
                    const float inv = finalize_inv(Ltot);
                    volatile int* m = meta_pair + 8 * (k & 1) + 4 * wg;
                    const int e_row0 = m[0], e_lo = m[1], e_hi = m[2], e_head = m[3];
                    if (r >= e_lo && r < e_hi && p.lse)
                        p.lse[(static_cast<long long>(e_row0) + r) * p.Hq + e_head] = finalize_lse(m_run, Ltot, c);
#ifdef TIK_PA_TRACE
                    long long* tr = (blockIdx.x == 0 && k < PA_TRACE_ITEMS && quarter == 0 && lane == 0)
                                        ? &g_pa_trace[k * PA_TRACE_EVENTS + 32 + 8 * wg] : nullptr;
#else
                    long long* tr = nullptr;
#endif
                    pa_store_rows<D>(to, inv, e_row0, e_lo, e_hi, e_head, 0, D, stage_warp, o_base, p.Hq,
                                     bar_odrain + 8 * wg, 2u, lane, quarter, &p.tmO32, tr);
                }
                if (quarter == 0 && lane == 0) PA_STAMP(k, 17 + 10 * wg);
            } else {
                // ---- single item: one query tile; the warpgroups alternate over its KV tiles (global
                // step parity) and hand the row state to each other through shared memory
                const int qpos = 128 * it.T0 + r;
                const int n_tiles = it.n_tiles;
                const int last = n_tiles - 1;
                float M_g = -CUDART_INF_F, Lg_lo = 0.0f, Lg_hi = 0.0f;
                float m_own = -CUDART_INF_F, l_own_lo = 0.0f, l_own_hi = 0.0f;
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
                        if (with_o) pa_fold_o_tmem<D>(tlane + COL_OA, tlane + COL_OB, f);
                    }
                };
                for (int t = wg ^ static_cast<int>(Gs0 & 1); t < n_tiles; t += 2) {
                    const uint32_t Gg = Gs0 + t;
                    PA_AUX(Gg | (k << 20));
                    const bool chunk_start = (t % TILES_PER_CHUNK) == 0;
                    PA_WAIT(13, bar_sfull + 8 * wg, (Gg >> 1) & 1, abort_word, p.dev_status);
                    tc_fence_after();
                    {
                        const int kmax = qpos - 128 * t;            // columns > kmax are masked
                        uint32_t sc[128];
                        tmem_ld32(ts, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
                        tmem_ld32(ts + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                        tmem_ld32(ts + 64, *reinterpret_cast<uint32_t(*)[32]>(&sc[64]));
                        tmem_ld32(ts + 96, *reinterpret_cast<uint32_t(*)[32]>(&sc[96]));
                        tmem_wait_ld();
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
                        for (int q = 0; q < 8; ++q) mx[q] = fmaxf(__uint_as_float(sc[2 * q]), __uint_as_float(sc[2 * q + 1]));
#pragma unroll
                        for (int i = 16; i < 128; i += 16) {
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                mx[q] = fmax3(mx[q], __uint_as_float(sc[i + 2 * q]), __uint_as_float(sc[i + 2 * q + 1]));
                        }
                        const float mt = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmax3(fmax3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
                        // state handed over by the thread that processed tile t-1
                        float m_old = -CUDART_INF_F, l_old_lo = 0.0f, l_old_hi = 0.0f;
                        float m_prev = 0.0f, l_prev_lo = 0.0f, l_prev_hi = 0.0f;   // finished chunk, if any
                        const bool fold_now = chunk_start && t > 0;      // a finished chunk precedes this tile
                        if (t > 0) {
                            PA_WAIT(14, bar_m, (hc0 + t - 1) & 1, abort_word, p.dev_status);
                            if (fold_now) {
                                wait_tile_done(Gg - 1);
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
#pragma unroll
                        for (int i = 0; i < 64; i += 8) softmax_p8(&sc[i], c, neg_mc, rs_lo, &sc[i >> 1]);
                        // The weight buffer of this warpgroup was last read by the PV two global steps back
                        // (possibly the previous item's): waited for right before the first store.  Every warp
                        // passes this wait before it arrives for this step.
                        if (Gg >= 2) wait_pv(Gg - 2);
                        tmem_st32(tp, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
#pragma unroll
                        for (int i = 0; i < 64; i += 8) softmax_p8(&sc[64 + i], c, neg_mc, rs_hi, &sc[32 + (i >> 1)]);
                        tmem_st32(tp + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                        if (t > 0 && !fold_now) {
                            wait_tile_done(Gg - 1);
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
                            wait_pv(Gg - 1);
                            fold_chunk(t / TILES_PER_CHUNK - 1, m_prev, l_prev_lo, l_prev_hi, true);
                        } else if (!chunk_start && !__all_sync(0xffffffffu, alpha == 1.0f)) {
                            wait_pv(Gg - 1);
                            pa_rescale_o_tmem<D>(tlane + ((t / TILES_PER_CHUNK) == 0 ? COL_OA : COL_OB), alpha);
                        }
                        tmem_wait_st();
                        // this thread closed a chunk that is not the row's last: fold its scalars here too
                        if (t != last && (t % TILES_PER_CHUNK) == TILES_PER_CHUNK - 1)
                            fold_chunk(t / TILES_PER_CHUNK, m_own, l_own_lo, l_own_hi, false);
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_pfull + 8 * wg);
                }
                // ---- the warpgroup that owned the last tile finishes the row state: folded accumulator in
                // O_A, reciprocal and output position in shared memory; then both warpgroups write half of
                // the output columns each
                if (wg == static_cast<int>((Gs0 + last) & 1)) {
                    wait_pv(Gs0 + last);
                    fold_chunk(last / TILES_PER_CHUNK, m_own, l_own_lo, l_own_hi, true);
                    const float Ltot = finalize_l(Lg_lo, Lg_hi);
                    st_inv_all[128 * (k & 1) + r] = finalize_inv(Ltot);
                    const int row0 = it.qb + 128 * it.T0 - it.pos0;
                    const int lo = max(0, it.pos0 - 128 * it.T0), hi = min(128, it.ctx - 128 * it.T0);
                    if (lane == 0) {
                        volatile int* m = meta_single + 4 * (k & 1);
                        m[0] = row0;
                        m[1] = lo;
                        m[2] = hi;
                        m[3] = it.head;
                    }
                    if (r >= lo && r < hi && p.lse)
                        p.lse[(static_cast<long long>(row0) + r) * p.Hq + it.head] = finalize_lse(M_g, Ltot, c);
                    tc_fence_before();
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                tc_fence_after();
                if (!aborted_warp()) {
                    const float inv = st_inv_all[128 * (k & 1) + r];
                    volatile int* m = meta_single + 4 * (k & 1);
                    pa_store_rows<DH>(tlane + COL_OA + DH * wg, inv, m[0], m[1], m[2], m[3], DH * wg, D, stage_warp, o_base,
                                      p.Hq, bar_odrain, 1u, lane, quarter, &p.tmO32);
                }
                hc0 += n_tiles;
            }
            Gs0 += n_steps;
        }
        if (lane == 0) tma_store_wait_all();     // this warp's bulk stores are complete before the CTA ends
    }
    }

    // ---------------------------------------------------------------- teardown
#ifdef TIK_PA_TRACE
    if (*abort_word && lane == 0 && pa_tag != 0 && g_pa_tags[(blockIdx.x * 12 + warp) * 2 + 1] == 0) {
        // where every warp of an aborted CTA waited last (first aborted launch only)
        g_pa_tags[(blockIdx.x * 12 + warp) * 2] = pa_tag;
        g_pa_tags[(blockIdx.x * 12 + warp) * 2 + 1] = 0x40000000 | pa_aux;
    }
#endif
    if (*abort_word) {   // let copies and MMAs in flight finish before shared memory and TMEM are released
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 1000000ull) {
        }
    }
    // Behind the single-tile grid: this grid must not complete before that one has (a kernel that
    // follows with a programmatic dependency waits for its immediate predecessor only).
    if (p.wait_at_end) pdl_wait();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

// ------------------------------------------------------------------ launcher
template <int D, bool PAGED>
static cudaError_t launch_persist_t(int ncta, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                    const AttnParams& p, const int4* plan, cudaStream_t stream) {
    auto kern = attn_persist_kernel<D, PAGED>;
    static DeviceOnce configured;     // the shared-memory opt-in belongs to the (function, device) pair
    cudaError_t e = configured.run([&]() {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(PASmem<D>::BYTES));
    });
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(ncta));
    cfg.blockDim = dim3(PA_THREADS);
    cfg.dynamicSmemBytes = PASmem<D>::BYTES;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, p, plan);
}

#ifdef TIK_PA_TRACE
extern "C" int tik_debug_pa_trace(long long* host_out, int n) {
    const int total = PA_TRACE_ITEMS * PA_TRACE_EVENTS;
    return cudaMemcpyFromSymbol(host_out, g_pa_trace, sizeof(long long) * (n < total ? n : total)) == cudaSuccess ? 0 : -1;
}
extern "C" int tik_debug_pa_steps(long long* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_pa_steps, sizeof(long long) * 8 * 4 * 16 * 8) == cudaSuccess ? 0 : -1;
}
extern "C" int tik_debug_pa_tags(int* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_pa_tags, sizeof(int) * 148 * 12 * 2) == cudaSuccess ? 0 : -1;
}
#endif

size_t attn_plan_bytes(int64_t S, int64_t max_positions) {
    const int64_t nt = (max_positions + 127) / 128;
    const int64_t X = nt <= 16 ? (nt + 1) / 2 : 8 + (nt - 16);
    return static_cast<size_t>(16 + 16 * S * X);
}

bool attn_persist_supported(int64_t S, int64_t max_positions) {
    const int64_t nt = (max_positions + 127) / 128;
    const int64_t X = nt <= 16 ? (nt + 1) / 2 : 8 + (nt - 16);
    return S >= 1 && S <= 65535 && X >= 1 && X <= PLAN_XMAX && S * X <= (1ll << 22);
}
// (the caller also checks S * X * Hq < 2^31: item indices are 32-bit)

cudaError_t launch_attn_persist(int d, bool paged, int sm_count, int S, int X, const CUtensorMap& tmQ,
                                const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnParams& p, void* plan,
                                cudaStream_t stream) {
    // Query tiles >= 16 (candidates x >= 8) are long items (17+ steps): they run best as one CTA per
    // item, with three-stage K/V rings and the sequence-major block order.  When the call has any,
    // three launches follow each other with programmatic dependencies: the planning kernel (paired
    // items only), the one-CTA-per-item grid over the single tiles, and the persistent grid, whose
    // CTAs start as the single-tile grid's last wave leaves SMs free.  Measured on B200: with
    // sequences of 16 K tokens the split is 9 % faster than the persistent grid alone (which gives
    // single tiles two-stage rings), with lengths up to 9 K (most items paired or short) 4 % slower
    // (three launches, two tails): it is used when the length bound exceeds 96 tiles.
    const bool split = X > 8 + (96 - 16);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(1024);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_plan_kernel, p.cu_seqlens, paged ? p.ctx_lens : static_cast<const int32_t*>(nullptr),
                                       S, split ? 7 : X - 1, static_cast<int4*>(plan));
    if (e != cudaSuccess) return e;
    AttnParams pp = p;
    if (split) {
        AttnParams ps = p;
        ps.x_base = 8;
        e = launch_attn(d, paged ? 1 : 0, dim3(static_cast<unsigned>(X - 8), static_cast<unsigned>(p.Hq), static_cast<unsigned>(S)),
                        tmQ, tmK, tmV, ps, stream);
        if (e != cudaSuccess) return e;
        pp.wait_at_end = 1;
    }
    const int4* pl = static_cast<const int4*>(plan);
    if (d == 128) {
        return paged ? launch_persist_t<128, true>(sm_count, tmQ, tmK, tmV, pp, pl, stream)
                     : launch_persist_t<128, false>(sm_count, tmQ, tmK, tmV, pp, pl, stream);
    }
    return paged ? launch_persist_t<64, true>(sm_count, tmQ, tmK, tmV, pp, pl, stream)
                 : launch_persist_t<64, false>(sm_count, tmQ, tmK, tmV, pp, pl, stream);
}

}  // namespace tik
