// Host-side declarations shared by the translation units of libtik (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <string>

struct tik_ctx {
    int device = 0;
    int sm_count = 0;
    int* dev_status = nullptr;          // one int of device flags (TIK_DEV_*)
    void* encode_tiled = nullptr;       // cuTensorMapEncodeTiled from the driver
    std::string last_error;
};

namespace tik {

// Kernel launches issued by the library in this process (every launch site counts itself): what
// tik_kernel_launches() reports, so that a caller can state how many kernels a region launched.
extern std::atomic<unsigned long long> g_kernel_launches;
inline void count_launch() { g_kernel_launches.fetch_add(1, std::memory_order_relaxed); }


// Runs a per-device set-up step (typically cudaFuncSetAttribute, whose effect belongs to the
// current device's context) once for every device that reaches it.  One flag per device ordinal;
// a failed step is retried by the next call.  Two threads racing on a device's first call may
// both run the step, which is harmless for idempotent set-up.
struct DeviceOnce {
    static constexpr int MAX_DEVICES = 64;
    std::atomic<bool> done[MAX_DEVICES] = {};
    bool is_done(int device) const {
        return device >= 0 && device < MAX_DEVICES && done[device].load(std::memory_order_acquire);
    }
    void mark(int device) {
        if (device >= 0 && device < MAX_DEVICES) done[device].store(true, std::memory_order_release);
    }
    // `device` < 0: use the current CUDA device.  Ordinals beyond the table run the step every time.
    template <class F>
    cudaError_t run(F&& step, int device = -1) {
        if (device < 0) {
            cudaError_t e = cudaGetDevice(&device);
            if (e != cudaSuccess) return e;
        }
        if (is_done(device)) return cudaSuccess;
        cudaError_t e = step();
        if (e == cudaSuccess) mark(device);
        return e;
    }
};

// Builds a bf16 tiled tensor map with 128-byte swizzle; dims/box innermost first, strides
// in bytes for dims 1..rank-1.  Returns false (and fills err) on failure.
bool make_tmap_bf16(tik_ctx* ctx, CUtensorMap* out, const void* base, int rank,
                    const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                    std::string* err);

struct AttnParams {
    alignas(64) CUtensorMap tmO; // train / prefill: tiled map of the output (same shape and box as Q)
    alignas(64) CUtensorMap tmO32;   // the same tensor with a box of 32 rows (persistent kernel: one warp's rows)
    void* o;                     // bf16 output rows
    float* lse;                  // optional
    const int32_t* cu_seqlens;   // train: per sequence; prefill: per sequence, query tokens
    const int32_t* ctx_lens;     // prefill / decode
    const int32_t* block_table;  // prefill / decode
    int max_blocks;
    int Hq, Hkv, G;
    int page_size, pages_per_tile, num_pages;
    float c;                     // softmax_scale * log2(e)
    float* part_o;               // decode: [B][Hq][nchunk_max][d]
    float* part_ml;              // decode: [B][Hq][nchunk_max][4] = m, l_lo, l_hi, unused
    int page_shift, ppt_shift;   // log2(page_size), log2(pages_per_tile)
    int nchunk_max;
    int max_ctx;                 // decode: the host's bound on ctx_lens (sized the grid and the scratch)
    int cpc;                     // decode: consecutive chunks streamed by one CTA
    int direct_out;              // decode: one chunk per sequence by the host's bound -- the chunk's partial is
                                 // the result, normalised and stored by the decode kernel itself (no combine)
    int* dev_status;
    int lookahead;               // train / prefill: block distance of the query-tile L2 prefetch
    int x_base;                  // train / prefill, one CTA per item: candidate index of the grid's last block (0, or 8: single tiles only)
    int wait_at_end;             // persistent kernel: 1 = launched behind the single-tile grid (see launch_attn_persist)
};

// mode: 0 train (packed K/V), 1 prefill (paged K/V), 2 decode (paged K/V, chunk partials)
cudaError_t launch_attn(int d, int mode, dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                        const CUtensorMap& tmV, const AttnParams& p, cudaStream_t stream);
cudaError_t launch_combine(int d, const AttnParams& p, int B, cudaStream_t stream);
// Decode for query groups of at most DECODE2_MAX_G heads (tik_decode.cu): two small CTAs per SM,
// same grid, scratch layout and output bits as launch_attn in decode mode.
constexpr int DECODE2_MAX_G = 8;
cudaError_t launch_decode2(int d, dim3 grid, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                           const AttnParams& p, cudaStream_t stream);

// Persistent full-sequence attention (tik_attn_persist.cu): a planning kernel writes the list of
// work items of the call into `plan` (attn_plan_bytes bytes, 16-byte aligned), then one CTA per SM
// walks it.  X = candidate items per sequence for the host's length bound (as the grid's x extent
// of the one-CTA-per-item kernel).  Same output bits as launch_attn.
size_t attn_plan_bytes(int64_t S, int64_t max_positions);
bool attn_persist_supported(int64_t S, int64_t max_positions);
cudaError_t launch_attn_persist(int d, bool paged, int sm_count, int S, int X, const CUtensorMap& tmQ,
                                const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnParams& p, void* plan,
                                cudaStream_t stream);

struct PrepParams {
    __nv_bfloat16* q;            // [total_new][Hq][d], in place
    __nv_bfloat16* k;            // [total_new][Hkv][d], in place
    const __nv_bfloat16* v;      // [total_new][Hkv][d] or null
    const __nv_bfloat16* q_weight;   // [d] or null (no Q norm)
    const __nv_bfloat16* k_weight;   // [d] or null (no K norm)
    float eps;
    const float* cos_sin;        // [max_pos][d]: cos | sin
    int max_pos;
    const int32_t* cu_new;       // [S+1]
    const int32_t* ctx_lens;     // [S] context after the write, or null (positions start at 0)
    __nv_bfloat16* k_cache;      // [num_pages][Hkv][page_size][d] or null (no cache write)
    __nv_bfloat16* v_cache;
    const int32_t* block_table;
    int max_blocks, S, Hq, Hkv, page_size, num_pages;
    long long total_new;
    int* dev_status;
};
cudaError_t launch_prep(int d, const PrepParams& p, int64_t total_new, cudaStream_t stream);

// Decode: how many consecutive chunks one CTA streams.  A CTA's set-up and drain cost about a
// third of one chunk's streaming time, so several chunks per CTA pay as long as the grid still
// covers every CTA slot several times over.  Chunk partials do not depend on this choice.
// With two resident CTAs per SM (tik_decode.cu) a CTA's rate is bound by its own serial chain and
// short ring (measured ~22 GB/s per CTA), so what counts is that all slots stay busy and that no
// CTA is long: many one-chunk CTAs that the hardware deals out dynamically do that better than few
// long ones (a batch of ragged contexts is as slow as its longest CTA).  Chunks are grouped only
// when the grid stays above four waves.
inline int decode_chunks_per_cta(long long B, int Hkv, int nchunk, int sm_count, int ctas_per_sm = 1) {
    const long long slots = static_cast<long long>(ctas_per_sm) * (sm_count > 0 ? sm_count : 148);
    for (int c = 4; c > 1; --c)
        if (c <= nchunk && B * Hkv * ((nchunk + c - 1) / c) >= 4 * slots) return c;
    return 1;
}
cudaError_t launch_kv_write(const void* k_new, const void* v_new, const int32_t* cu_new,
                            const int32_t* ctx_lens, void* k_cache, void* v_cache,
                            const int32_t* block_table, int max_blocks, int S, int64_t total_new,
                            int Hkv, int d, int page_size, int num_pages, int* dev_status,
                            cudaStream_t stream);

struct LogprobParams {
    const int32_t* target;
    float* logprob;
    float* lse;                  // optional
    float* part_ml;              // [T][nsuper][2]
    float* z_target;             // [T]
    int64_t T;
    int H, V, nsuper;
    int spc;                     // consecutive 1024-column super-chunks walked by one CTA
    int unit_mode;               // 1: T <= LP_UNIT_MODE_ROWS: persistent CTAs over 256-column steps, one (max, sum) pair per 128-column tile
    int nunit, ntile128;         // units = ceil(V / 256) x ntp, ceil(V / 128)
    int ntp;                     // unit mode: pairs of token tiles (single CTAs: 1)
    int sm_count;
    float inv_temperature;
    int* dev_status;
};
cudaError_t launch_logprob(const CUtensorMap& tmA, const CUtensorMap& tmB, const LogprobParams& p, bool pair,
                           cudaStream_t stream);

struct NormParams {
    const __nv_bfloat16* x;      // [T][H]
    __nv_bfloat16* residual;     // [T][H] in/out, or null (plain RMSNorm)
    const __nv_bfloat16* weight; // [H]
    __nv_bfloat16* y;            // [T][H] (may be x)
    float eps;
    long long T;
    int H;
};
cudaError_t launch_rmsnorm(const NormParams& p, cudaStream_t stream);
cudaError_t launch_swiglu(const void* gate_up, void* out, long long T, int I, cudaStream_t stream);

struct LinearParams {
    __nv_bfloat16* y;            // [T][N]
    int64_t T;
    int K, N, nsuper;
    int super_cols;              // output columns per CTA: a multiple of 256, at most 4096
    int unit_mode;               // T <= 128: persistent CTAs over column units (tmA box a_rows, tmB box nu rows)
    int ntp;                     // pair unit mode: pairs of row tiles (1 .. 8)
    int nu, nunit, a_rows;       // unit width 64 / 128 / 256, ceil(N / nu), staged x rows 32 / 64 / 128
    int sm_count;
    int* dev_status;
};
// Unit width of the decode-shaped linear kernel, from a cost model of one 64-wide K slice of one
// unit on a B200: its four MMAs (N = 256: 270 ns, 128: 135 ns, 64: 100 ns -- shared-memory bound) plus
// the issuing thread's ~170 ns per stage spread over the stage's slices; or the slice's bytes (x
// rows and W rows) into one SM at ~95 GB/s; or its W bytes at the CTA's share of ~6.5 TB/s -- whichever
// is longest; a CTA runs `waves` units one after the other.  The cheapest width wins, the wider one
// on ties (x is staged once per unit).
inline int linear_unit_cols(int N, int a_rows, int sm_count) {
    int best = 256;
    double best_cost = -1.0;
    for (int nu = 256; nu >= 64; nu /= 2) {
        const long long units = (N + nu - 1) / nu;
        const long long waves = (units + sm_count - 1) / sm_count;
        const double active = static_cast<double>(units < sm_count ? units : sm_count);
        const double mma_ns = nu == 256 ? 270.0 : nu == 128 ? 135.0 : 100.0;
        int kps = 256 / nu;
        while (kps > 1 && (192 * 1024) / ((a_rows + nu) * 128 * kps) < 3) kps >>= 1;
        double slice_ns = mma_ns + 170.0 / kps;
        const double fill_ns = (a_rows + nu) * 128.0 / 95.0;
        const double hbm_ns = nu * 128.0 / (6500.0 / active);
        if (fill_ns > slice_ns) slice_ns = fill_ns;
        if (hbm_ns > slice_ns) slice_ns = hbm_ns;
        const double cost = waves * slice_ns;
        if (best_cost < 0.0 || cost < best_cost * 0.999) {
            best_cost = cost;
            best = nu;
        }
    }
    return best;
}
cudaError_t launch_linear(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                          const LinearParams& p, bool pair, cudaStream_t stream);

struct BwdParams {
    const int32_t* cu_seqlens;   // [S+1]
    const float* lse;            // [total][Hq], natural log, from the forward
    float* delta;                // [total][Hq] scratch: rowsum(dO o O)
    __nv_bfloat16* dq;           // [total][Hq][d]
    __nv_bfloat16* dk;           // [total][Hkv][d]
    __nv_bfloat16* dv;           // [total][Hkv][d]
    int Hq, Hkv, G;
    float c;                     // softmax_scale * log2(e)
    float scale;
    int* dev_status;
};
cudaError_t launch_attn_bwd(int d, int max_tiles, int S, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                            const CUtensorMap& tmV, const CUtensorMap& tmDO, const BwdParams& p,
                            const void* o, const void* dout, long long n_vec, cudaStream_t stream);

}  // namespace tik
