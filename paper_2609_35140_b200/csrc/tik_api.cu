// C ABI of libtik: argument checks, tensor maps, grid sizing from host upper bounds, launches.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "../../include/tik.h"
#include "tik_core.cuh"
#include "tik_internal.h"

namespace tik {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

bool make_tmap_bf16(tik_ctx* ctx, CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                    const uint64_t* strides_bytes, const uint32_t* box, std::string* err) {
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bdim[5], estr[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estr[i] = 1;
        if (i > 0) gstr[i - 1] = strides_bytes[i - 1];
    }
    CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
        out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank), const_cast<void*>(base), gdim,
        gstr, bdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char buf[256];
        snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled failed (CUresult %d, rank %d, dims %llu %llu %llu)",
                 static_cast<int>(r), rank, (unsigned long long)dims[0], (unsigned long long)dims[1],
                 (unsigned long long)(rank > 2 ? dims[2] : 0));
        *err = buf;
        return false;
    }
    return true;
}

static tik_status fail(tik_ctx* ctx, tik_status s, const char* msg) {
    if (ctx) ctx->last_error = msg;
    return s;
}
static tik_status cuda_fail(tik_ctx* ctx, cudaError_t e, const char* where) {
    ctx->last_error = std::string(where) + ": " + cudaGetErrorString(e);
    return TIK_ERR_CUDA;
}
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool page_ok(int page) { return page == 16 || page == 32 || page == 64 || page == 128; }
static float scale_to_c(float softmax_scale) { return softmax_scale * LOG2E_F; }
// Candidate work items per (sequence, head) for the full-sequence kernels: query tiles 0..15 go
// in pairs (x = 0..7), tiles >= 16 one by one (x = 8 + tile - 16); see attn_kernel.
static unsigned attn_grid_x(int max_positions) {
    const int nt = (max_positions + 127) / 128;
    return static_cast<unsigned>(nt <= 16 ? (nt + 1) / 2 : 8 + (nt - 16));
}

// The persistent kernel runs when the caller passed a large enough, 16-byte aligned plan buffer and
// the call is within what the planning kernel handles; otherwise one CTA per work item.
static bool use_persistent(const void* ws, size_t ws_bytes, int S, int max_positions, int Hq, int sm_count) {
    if (!ws || !aligned16(ws) || !attn_persist_supported(S, max_positions)) return false;
    const long long nt = (static_cast<long long>(max_positions) + 127) / 128;
    const long long X = nt <= 16 ? (nt + 1) / 2 : 8 + (nt - 16);
    if (static_cast<long long>(S) * X * Hq >= (1ll << 31)) return false;
    // fewer work items than two per SM: nothing to amortise, the planning launch only adds latency
    if (static_cast<long long>(S) * X * Hq <= 2ll * sm_count) return false;
    return ws_bytes >= attn_plan_bytes(S, max_positions);
}

static tik_status check_heads(tik_ctx* ctx, int Hq, int Hkv, int d, float scale) {
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return fail(ctx, TIK_ERR_INVALID_ARG, "Hq must be a positive multiple of Hkv");
    if (!(scale > 0.0f) || !std::isfinite(scale)) return fail(ctx, TIK_ERR_INVALID_ARG, "softmax_scale must be finite and > 0");
    if (d != 64 && d != 128) return fail(ctx, TIK_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
    if (Hq / Hkv > 32) return fail(ctx, TIK_ERR_UNSUPPORTED, "Hq/Hkv must be <= 32");
    return TIK_OK;
}

}  // namespace tik

using namespace tik;

namespace tik {
std::atomic<unsigned long long> g_kernel_launches{0};
}

extern "C" {

unsigned long long tik_kernel_launches(void) { return tik::g_kernel_launches.load(std::memory_order_relaxed); }


tik_status tik_create(tik_ctx** out, int device) {
    if (!out) return TIK_ERR_INVALID_ARG;
    *out = nullptr;
    tik_ctx* ctx = new (std::nothrow) tik_ctx();
    if (!ctx) return TIK_ERR_CUDA;
    ctx->device = device;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    int major = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e == cudaSuccess && major != 10) {
        delete ctx;
        return TIK_ERR_UNSUPPORTED;   // built for sm_100a only
    }
    if (e == cudaSuccess) e = cudaMalloc(&ctx->dev_status, 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->dev_status, 0, 256);
    if (e == cudaSuccess) {
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault, &qres);
        if (e == cudaSuccess && (qres != cudaDriverEntryPointSuccess || !ctx->encode_tiled)) e = cudaErrorNotSupported;
    }
    if (e != cudaSuccess) {
        if (ctx->dev_status) cudaFree(ctx->dev_status);
        delete ctx;
        return TIK_ERR_CUDA;
    }
    *out = ctx;
    return TIK_OK;
}

tik_status tik_destroy(tik_ctx* ctx) {
    if (!ctx) return TIK_OK;
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    delete ctx;
    return TIK_OK;
}

const char* tik_status_str(tik_status s) {
    switch (s) {
        case TIK_OK: return "ok";
        case TIK_ERR_INVALID_ARG: return "invalid argument";
        case TIK_ERR_UNSUPPORTED: return "outside the supported domain";
        case TIK_ERR_WORKSPACE: return "workspace too small";
        case TIK_ERR_CUDA: return "CUDA error";
        default: return "unknown status";
    }
}

const char* tik_last_error(const tik_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

int tik_selftest_host(void) {
    // Per-device set-up bookkeeping (DeviceOnce) with stand-in device ordinals and steps: the step
    // runs once per device, a failed step is retried, a second device is not skipped because the
    // first one is done, and ordinals outside the table run every time.
    DeviceOnce once;
    int runs = 0;
    auto ok_step = [&]() { ++runs; return cudaSuccess; };
    auto bad_step = [&]() { ++runs; return cudaErrorInvalidValue; };
    if (once.run(bad_step, 0) != cudaErrorInvalidValue || runs != 1 || once.is_done(0)) return 1;
    if (once.run(ok_step, 0) != cudaSuccess || runs != 2 || !once.is_done(0)) return 2;
    if (once.run(ok_step, 0) != cudaSuccess || runs != 2) return 3;            // done: not run again
    if (once.is_done(1)) return 4;
    if (once.run(ok_step, 1) != cudaSuccess || runs != 3 || !once.is_done(1)) return 5;   // second device
    if (once.run(ok_step, 1) != cudaSuccess || runs != 3) return 6;
    if (once.run(ok_step, DeviceOnce::MAX_DEVICES + 5) != cudaSuccess || runs != 4) return 7;
    if (once.run(ok_step, DeviceOnce::MAX_DEVICES + 5) != cudaSuccess || runs != 5) return 8;
    return 0;
}
const char* tik_contract_id(void) { return TIK_CONTRACT_ID; }

size_t tik_workspace_bytes(int op, int64_t rows_or_batch, int Hq, int Hkv, int d, int64_t max_ctx, int H,
                           int V) {
    (void)Hkv;
    (void)H;
    if (op == TIK_OP_ATTN_TRAIN_FWD || op == TIK_OP_ATTN_PREFILL) {
        // rows_or_batch = number of sequences S, max_ctx = the host's bound on a sequence's positions
        if (rows_or_batch <= 0 || max_ctx <= 0 || !attn_persist_supported(rows_or_batch, max_ctx)) return 0;
        return attn_plan_bytes(rows_or_batch, max_ctx);
    }
    if (op == TIK_OP_ATTN_DECODE) {
        if (rows_or_batch <= 0 || max_ctx <= 0) return 0;
        const int64_t nchunk = (max_ctx + CHUNK - 1) / CHUNK;
        return static_cast<size_t>(rows_or_batch) * Hq * nchunk * (d + 4) * sizeof(float);
    }
    if (op == TIK_OP_TOKEN_LOGPROB) {
        if (rows_or_batch <= 0 || V <= 0) return 0;
        // partial (max, sum) pairs: per 1024-column super-chunk, or per 128-column tile for calls of
        // at most LP_UNIT_MODE_ROWS rows (decode-sized batches), plus one target logit per row
        const int64_t nsuper = (V + LP_SUPER - 1) / LP_SUPER, ntile = (V + LP_TILE - 1) / LP_TILE;
        const int64_t npart = rows_or_batch <= LP_UNIT_MODE_ROWS ? ntile : nsuper;
        return static_cast<size_t>(rows_or_batch) * (2 * npart + 1) * sizeof(float);
    }
    if (op == TIK_OP_ATTN_TRAIN_BWD) {      // rows_or_batch = total tokens: delta [tokens][Hq]
        if (rows_or_batch <= 0) return 0;
        return static_cast<size_t>(rows_or_batch) * Hq * sizeof(float);
    }
    return 0;
}

tik_status tik_device_status(tik_ctx* ctx, void* stream, int* out_flags) {
    if (!ctx || !out_flags) return TIK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int flags = 0;
    cudaError_t e = cudaMemcpyAsync(&flags, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->dev_status, 0, sizeof(int), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "tik_device_status");
    *out_flags = flags;
    return TIK_OK;
}

tik_status tik_attn_train_fwd(tik_ctx* ctx, const void* q, const void* k, const void* v, void* o, float* lse,
                              const int32_t* cu_seqlens, int S, int64_t total_tokens, int max_seqlen, int Hq,
                              int Hkv, int d, float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (S < 0 || total_tokens < 0 || max_seqlen < 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative size");
    tik_status s = check_heads(ctx, Hq, Hkv, d, softmax_scale);
    if (s != TIK_OK) return s;
    if (S == 0 || total_tokens == 0 || max_seqlen == 0) return TIK_OK;
    if (!q || !k || !v || !o || !cu_seqlens) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (total_tokens >= (1ll << 31)) return fail(ctx, TIK_ERR_UNSUPPORTED, "total_tokens must be < 2^31");

    CUtensorMap tmQ, tmK, tmV;
    std::string err;
    const uint64_t ud = static_cast<uint64_t>(d);
    uint64_t qd[3] = {ud, static_cast<uint64_t>(Hq), static_cast<uint64_t>(total_tokens)};
    uint64_t qs[2] = {ud * 2, ud * 2 * Hq};
    uint64_t kd[3] = {ud, static_cast<uint64_t>(Hkv), static_cast<uint64_t>(total_tokens)};
    uint64_t ks[2] = {ud * 2, ud * 2 * Hkv};
    uint32_t box[3] = {64, 1, 128};
    if (!make_tmap_bf16(ctx, &tmQ, q, 3, qd, qs, box, &err) || !make_tmap_bf16(ctx, &tmK, k, 3, kd, ks, box, &err) ||
        !make_tmap_bf16(ctx, &tmV, v, 3, kd, ks, box, &err))
        return fail(ctx, TIK_ERR_CUDA, err.c_str());

    AttnParams p{};
    if (!make_tmap_bf16(ctx, &p.tmO, o, 3, qd, qs, box, &err)) return fail(ctx, TIK_ERR_CUDA, err.c_str());
    uint32_t box32[3] = {64, 1, 32};
    if (!make_tmap_bf16(ctx, &p.tmO32, o, 3, qd, qs, box32, &err)) return fail(ctx, TIK_ERR_CUDA, err.c_str());
    p.o = o;
    p.lse = lse;
    p.cu_seqlens = cu_seqlens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.c = scale_to_c(softmax_scale);
    p.dev_status = ctx->dev_status;
    p.lookahead = ctx->sm_count;
    dim3 grid(attn_grid_x(max_seqlen), Hq, S);
    if (grid.y > 65535 || grid.z > 65535) return fail(ctx, TIK_ERR_UNSUPPORTED, "Hq and S must be <= 65535");
    cudaError_t e;
    if (use_persistent(ws, ws_bytes, S, max_seqlen, Hq, ctx->sm_count))
        e = launch_attn_persist(d, false, ctx->sm_count, S, static_cast<int>(grid.x), tmQ, tmK, tmV, p, ws,
                                static_cast<cudaStream_t>(stream));
    else
        e = launch_attn(d, 0, grid, tmQ, tmK, tmV, p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_attn_train_fwd");
}

tik_status tik_kv_cache_write(tik_ctx* ctx, const void* k_new, const void* v_new, const int32_t* cu_seqlens_new,
                              const int32_t* ctx_lens, void* k_cache, void* v_cache, const int32_t* block_table,
                              int max_blocks, int S, int64_t total_new, int Hkv, int d, int page_size,
                              int num_pages, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (S < 0 || total_new < 0 || max_blocks < 0 || num_pages < 0 || Hkv <= 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative size");
    if (d != 64 && d != 128) return fail(ctx, TIK_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
    if (!page_ok(page_size)) return fail(ctx, TIK_ERR_UNSUPPORTED, "page_size must be 16, 32, 64 or 128");
    if (S == 0 || total_new == 0) return TIK_OK;
    if (!k_new || !v_new || !cu_seqlens_new || !ctx_lens || !k_cache || !v_cache || !block_table)
        return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (total_new >= (1ll << 31)) return fail(ctx, TIK_ERR_UNSUPPORTED, "total_new must be < 2^31");
    cudaError_t e = launch_kv_write(k_new, v_new, cu_seqlens_new, ctx_lens, k_cache, v_cache, block_table,
                                    max_blocks, S, total_new, Hkv, d, page_size, num_pages, ctx->dev_status,
                                    static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_kv_cache_write");
}

static tik_status make_cache_maps(tik_ctx* ctx, const void* k_cache, const void* v_cache, int Hkv, int d,
                                  int page_size, int num_pages, CUtensorMap* tmK, CUtensorMap* tmV) {
    std::string err;
    const uint64_t ud = static_cast<uint64_t>(d);
    uint64_t cd[4] = {ud, static_cast<uint64_t>(page_size), static_cast<uint64_t>(Hkv),
                      static_cast<uint64_t>(num_pages)};
    uint64_t cs[3] = {ud * 2, ud * 2 * page_size, ud * 2 * page_size * Hkv};
    uint32_t box[4] = {64, static_cast<uint32_t>(page_size), 1, 1};
    if (!make_tmap_bf16(ctx, tmK, k_cache, 4, cd, cs, box, &err) ||
        !make_tmap_bf16(ctx, tmV, v_cache, 4, cd, cs, box, &err))
        return fail(ctx, TIK_ERR_CUDA, err.c_str());
    return TIK_OK;
}

tik_status tik_attn_prefill(tik_ctx* ctx, const void* q, void* o, float* lse, const int32_t* cu_seqlens_q,
                            const int32_t* ctx_lens, const void* k_cache, const void* v_cache,
                            const int32_t* block_table, int max_blocks, int S, int64_t total_q, int max_q_len,
                            int max_ctx_len, int Hq, int Hkv, int d, int page_size, int num_pages,
                            float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (S < 0 || total_q < 0 || max_q_len < 0 || max_ctx_len < 0 || max_blocks < 0 || num_pages < 0)
        return fail(ctx, TIK_ERR_INVALID_ARG, "negative size");
    tik_status s = check_heads(ctx, Hq, Hkv, d, softmax_scale);
    if (s != TIK_OK) return s;
    if (!page_ok(page_size)) return fail(ctx, TIK_ERR_UNSUPPORTED, "page_size must be 16, 32, 64 or 128");
    if (S == 0 || total_q == 0 || max_q_len == 0) return TIK_OK;
    if (!q || !o || !cu_seqlens_q || !ctx_lens || !k_cache || !v_cache || !block_table || num_pages == 0)
        return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(q) || !aligned16(o) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (total_q >= (1ll << 31)) return fail(ctx, TIK_ERR_UNSUPPORTED, "total_q must be < 2^31");

    CUtensorMap tmQ, tmK, tmV;
    std::string err;
    const uint64_t ud = static_cast<uint64_t>(d);
    uint64_t qd[3] = {ud, static_cast<uint64_t>(Hq), static_cast<uint64_t>(total_q)};
    uint64_t qs[2] = {ud * 2, ud * 2 * Hq};
    uint32_t box[3] = {64, 1, 128};
    if (!make_tmap_bf16(ctx, &tmQ, q, 3, qd, qs, box, &err)) return fail(ctx, TIK_ERR_CUDA, err.c_str());
    s = make_cache_maps(ctx, k_cache, v_cache, Hkv, d, page_size, num_pages, &tmK, &tmV);
    if (s != TIK_OK) return s;

    AttnParams p{};
    if (!make_tmap_bf16(ctx, &p.tmO, o, 3, qd, qs, box, &err)) return fail(ctx, TIK_ERR_CUDA, err.c_str());
    uint32_t box32[3] = {64, 1, 32};
    if (!make_tmap_bf16(ctx, &p.tmO32, o, 3, qd, qs, box32, &err)) return fail(ctx, TIK_ERR_CUDA, err.c_str());
    p.o = o;
    p.lse = lse;
    p.cu_seqlens = cu_seqlens_q;
    p.ctx_lens = ctx_lens;
    p.block_table = block_table;
    p.max_blocks = max_blocks;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.page_size = page_size;
    p.pages_per_tile = 128 / page_size;
    p.page_shift = page_size == 16 ? 4 : page_size == 32 ? 5 : page_size == 64 ? 6 : 7;
    p.ppt_shift = 7 - p.page_shift;
    p.num_pages = num_pages;
    p.c = scale_to_c(softmax_scale);
    p.dev_status = ctx->dev_status;
    p.lookahead = ctx->sm_count;
    // query tiles are aligned to absolute positions 0 .. ctx-1 (tiles before the first new token exit)
    dim3 grid(attn_grid_x(max_ctx_len), Hq, S);
    if (grid.y > 65535 || grid.z > 65535) return fail(ctx, TIK_ERR_UNSUPPORTED, "Hq and S must be <= 65535");
    cudaError_t e;
    if (use_persistent(ws, ws_bytes, S, max_ctx_len, Hq, ctx->sm_count))
        e = launch_attn_persist(d, true, ctx->sm_count, S, static_cast<int>(grid.x), tmQ, tmK, tmV, p, ws,
                                static_cast<cudaStream_t>(stream));
    else
        e = launch_attn(d, 1, grid, tmQ, tmK, tmV, p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_attn_prefill");
}

tik_status tik_attn_prefill_kv(tik_ctx* ctx, const void* q, const void* k_new, const void* v_new, void* o,
                               float* lse, const int32_t* cu_seqlens_q, const int32_t* ctx_lens, void* k_cache,
                               void* v_cache, const int32_t* block_table, int max_blocks, int S, int64_t total_q,
                               int max_q_len, int max_ctx_len, int Hq, int Hkv, int d, int page_size,
                               int num_pages, float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
    // argument checks of both halves run before anything is queued: a refused call writes nothing
    if (!ctx) return TIK_ERR_INVALID_ARG;
    tik_status s = check_heads(ctx, Hq, Hkv, d, softmax_scale);
    if (s != TIK_OK) return s;
    if (S > 0 && total_q > 0 && (!q || !o)) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(q) || !aligned16(o)) return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    s = tik_kv_cache_write(ctx, k_new, v_new, cu_seqlens_q, ctx_lens, k_cache, v_cache, block_table, max_blocks, S,
                           total_q, Hkv, d, page_size, num_pages, stream);
    if (s != TIK_OK) return s;
    return tik_attn_prefill(ctx, q, o, lse, cu_seqlens_q, ctx_lens, k_cache, v_cache, block_table, max_blocks, S,
                            total_q, max_q_len, max_ctx_len, Hq, Hkv, d, page_size, num_pages, softmax_scale, ws,
                            ws_bytes, stream);
}

tik_status tik_attn_decode(tik_ctx* ctx, const void* q, void* o, float* lse, const int32_t* ctx_lens,
                           const void* k_cache, const void* v_cache, const int32_t* block_table, int max_blocks,
                           int B, int max_ctx_len, int Hq, int Hkv, int d, int page_size, int num_pages,
                           float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (B < 0 || max_ctx_len < 0 || max_blocks < 0 || num_pages < 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative size");
    tik_status s = check_heads(ctx, Hq, Hkv, d, softmax_scale);
    if (s != TIK_OK) return s;
    if (!page_ok(page_size)) return fail(ctx, TIK_ERR_UNSUPPORTED, "page_size must be 16, 32, 64 or 128");
    if (B == 0 || max_ctx_len == 0) return TIK_OK;
    if (!q || !o || !ctx_lens || !k_cache || !v_cache || !block_table || num_pages == 0)
        return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(q) || !aligned16(o) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    const size_t need = tik_workspace_bytes(TIK_OP_ATTN_DECODE, B, Hq, Hkv, d, max_ctx_len, 0, 0);
    if (!ws || ws_bytes < need) return fail(ctx, TIK_ERR_WORKSPACE, "decode workspace too small");

    CUtensorMap tmQ, tmK, tmV;
    std::string err;
    const uint64_t ud = static_cast<uint64_t>(d);
    const int G = Hq / Hkv;
    uint64_t qd[3] = {ud, static_cast<uint64_t>(Hq), static_cast<uint64_t>(B)};
    uint64_t qs[2] = {ud * 2, ud * 2 * Hq};
    uint32_t box[3] = {64, static_cast<uint32_t>(G), 1};
    if (!make_tmap_bf16(ctx, &tmQ, q, 3, qd, qs, box, &err)) return fail(ctx, TIK_ERR_CUDA, err.c_str());
    s = make_cache_maps(ctx, k_cache, v_cache, Hkv, d, page_size, num_pages, &tmK, &tmV);
    if (s != TIK_OK) return s;

    const int nchunk = (max_ctx_len + CHUNK - 1) / CHUNK;
    AttnParams p{};
    p.o = o;
    p.lse = lse;
    p.ctx_lens = ctx_lens;
    p.block_table = block_table;
    p.max_blocks = max_blocks;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = G;
    p.page_size = page_size;
    p.pages_per_tile = 128 / page_size;
    p.page_shift = page_size == 16 ? 4 : page_size == 32 ? 5 : page_size == 64 ? 6 : 7;
    p.ppt_shift = 7 - p.page_shift;
    p.num_pages = num_pages;
    p.c = scale_to_c(softmax_scale);
    p.nchunk_max = nchunk;
    p.direct_out = nchunk == 1 ? 1 : 0;     // contexts of at most one chunk: no partials, no combine launch
    p.max_ctx = max_ctx_len;
    p.part_o = static_cast<float*>(ws);
    p.part_ml = p.part_o + static_cast<size_t>(B) * Hq * nchunk * d;
    p.dev_status = ctx->dev_status;
    // Two kernels give the same bits.  The small CTA of tik_decode.cu (two per SM) wins where CTAs
    // are short or few per SM: at most one (sequence, KV head) pair per SM but about as many chunks
    // as SMs or more (the one-CTA-per-SM kernel runs a ragged second wave there), and any number of
    // pairs with contexts of at most two chunks (a CTA streams <= 32 tiles; two co-resident CTAs hide
    // each other's set-up and tail: 64 x 4096 keys 103 -> 93 us, 256 x 2048 395 -> 313 us, also
    // right after a seconds-long GEMM).  With fewer chunks than SMs every CTA has an SM to itself
    // either way and the big kernel's faster per-CTA pipeline (two softmax warpgroups, five K/V
    // stages) gives the shorter latency; with many pairs of long contexts the same pipeline streams
    // faster per SM (the paper's decode grid, Sec. 6 Q3, covers both ends).
    const long long pairs = static_cast<long long>(B) * Hkv;
    const bool small_group = G <= DECODE2_MAX_G && (pairs <= ctx->sm_count || nchunk <= 2) && 4 * pairs * nchunk >= 3ll * ctx->sm_count;
    p.cpc = decode_chunks_per_cta(B, Hkv, nchunk, ctx->sm_count, small_group ? 2 : 1);
    p.lookahead = ctx->sm_count;
    dim3 grid((nchunk + p.cpc - 1) / p.cpc, Hkv, B);
    if (grid.y > 65535 || grid.z > 65535) return fail(ctx, TIK_ERR_UNSUPPORTED, "Hkv and B must be <= 65535");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = small_group ? launch_decode2(d, grid, tmQ, tmK, tmV, p, st) : launch_attn(d, 2, grid, tmQ, tmK, tmV, p, st);
    if (e == cudaSuccess && !p.direct_out) e = launch_combine(d, p, B, st);
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_attn_decode");
}

tik_status tik_qk_norm_rope_kv_write(tik_ctx* ctx, void* q, void* k, const void* v, const void* q_weight,
                                     const void* k_weight, float eps, const float* cos_sin, int max_pos,
                                     const int32_t* cu_seqlens_new, const int32_t* ctx_lens, void* k_cache,
                                     void* v_cache, const int32_t* block_table, int max_blocks, int S,
                                     int64_t total_new, int Hq, int Hkv, int d, int page_size, int num_pages,
                                     void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (S < 0 || total_new < 0 || max_pos < 0 || max_blocks < 0 || num_pages < 0)
        return fail(ctx, TIK_ERR_INVALID_ARG, "negative size");
    if (Hq <= 0 || Hkv <= 0) return fail(ctx, TIK_ERR_INVALID_ARG, "Hq and Hkv must be positive");
    if (!(eps >= 0.0f) || !std::isfinite(eps)) return fail(ctx, TIK_ERR_INVALID_ARG, "eps must be finite and >= 0");
    if (d != 64 && d != 128) return fail(ctx, TIK_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
    const bool cache = k_cache != nullptr || v_cache != nullptr;
    if (cache && !page_ok(page_size)) return fail(ctx, TIK_ERR_UNSUPPORTED, "page_size must be 16, 32, 64 or 128");
    if (S == 0 || total_new == 0) return TIK_OK;
    if (!q || !k || !cos_sin || !cu_seqlens_new || max_pos == 0) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (cache && (!k_cache || !v_cache || !v || !block_table || num_pages == 0))
        return fail(ctx, TIK_ERR_INVALID_ARG, "cache write needs k_cache, v_cache, v and block_table");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(q_weight) || !aligned16(k_weight) || !aligned16(cos_sin))
        return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (total_new >= (1ll << 31)) return fail(ctx, TIK_ERR_UNSUPPORTED, "total_new must be < 2^31");
    PrepParams p{};
    p.q = static_cast<__nv_bfloat16*>(q);
    p.k = static_cast<__nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.q_weight = static_cast<const __nv_bfloat16*>(q_weight);
    p.k_weight = static_cast<const __nv_bfloat16*>(k_weight);
    p.eps = eps;
    p.cos_sin = cos_sin;
    p.max_pos = max_pos;
    p.cu_new = cu_seqlens_new;
    p.ctx_lens = ctx_lens;
    p.k_cache = static_cast<__nv_bfloat16*>(k_cache);
    p.v_cache = static_cast<__nv_bfloat16*>(v_cache);
    p.block_table = block_table;
    p.max_blocks = max_blocks;
    p.S = S;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.page_size = page_size;
    p.num_pages = num_pages;
    p.total_new = total_new;
    p.dev_status = ctx->dev_status;
    cudaError_t e = launch_prep(d, p, total_new, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_qk_norm_rope_kv_write");
}

tik_status tik_token_logprob(tik_ctx* ctx, const void* hidden, const void* lm_head, const int32_t* target_ids,
                             float* logprob, float* lse, int64_t T, int H, int V, float inv_temperature, void* ws,
                             size_t ws_bytes, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (T < 0 || H <= 0 || V <= 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative or zero size");
    if (!(inv_temperature > 0.0f) || !std::isfinite(inv_temperature))
        return fail(ctx, TIK_ERR_INVALID_ARG, "inv_temperature must be finite and > 0");
    if (H % 64 != 0) return fail(ctx, TIK_ERR_UNSUPPORTED, "H must be a multiple of 64");
    if (T == 0) return TIK_OK;
    if (!hidden || !lm_head || !target_ids || !logprob) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(hidden) || !aligned16(lm_head) || !aligned16(ws)) return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (T >= (1ll << 31) - 128) return fail(ctx, TIK_ERR_UNSUPPORTED, "T must be < 2^31 - 128");
    const size_t need = tik_workspace_bytes(TIK_OP_TOKEN_LOGPROB, T, 0, 0, 0, 0, H, V);
    if (!ws || ws_bytes < need) return fail(ctx, TIK_ERR_WORKSPACE, "log-prob workspace too small");

    CUtensorMap tmA, tmB;
    std::string err;
    uint64_t ad[2] = {static_cast<uint64_t>(H), static_cast<uint64_t>(T)};
    uint64_t bd[2] = {static_cast<uint64_t>(H), static_cast<uint64_t>(V)};
    uint64_t st1[1] = {static_cast<uint64_t>(H) * 2};
    uint32_t box[2] = {64, 128};
    // More than one token tile: CTA pairs (two-SM MMAs), each CTA staging 128 of the 256 vocabulary
    // rows of an MMA step; a single tile (decode-sized calls) runs on single CTAs with all 256.
    // A log-probability has the same bits either way (same K order, same 128-column tiles).
    const bool pair = T > 128;
    uint32_t boxB[2] = {64, pair ? 128u : 256u};
    if (!make_tmap_bf16(ctx, &tmA, hidden, 2, ad, st1, box, &err) ||
        !make_tmap_bf16(ctx, &tmB, lm_head, 2, bd, st1, boxB, &err))
        return fail(ctx, TIK_ERR_CUDA, err.c_str());

    LogprobParams p{};
    p.target = target_ids;
    p.logprob = logprob;
    p.lse = lse;
    p.T = T;
    p.H = H;
    p.V = V;
    p.nsuper = (V + LP_SUPER - 1) / LP_SUPER;
    // A CTA's last accumulator is reduced after its MMAs have ended, so several super-chunks per
    // CTA amortise that tail (measured: 1360 -> 1455 TFLOP/s on workload 1 from 1 to 8); the partial
    // (m, l) pairs stay per 1024 columns.  The grid keeps four CTAs per SM or more.
    p.spc = 1;
    {
        const long long ntile = (T + 127) / 128;
        while (p.spc < 8 && ntile * ((p.nsuper + 2 * p.spc - 1) / (2 * p.spc)) >= 4ll * ctx->sm_count) p.spc *= 2;
    }
    p.unit_mode = T <= LP_UNIT_MODE_ROWS ? 1 : 0;
    p.ntp = pair ? static_cast<int>((T + 255) / 256) : 1;
    p.nunit = ((V + 255) / 256) * p.ntp;
    p.ntile128 = (V + LP_TILE - 1) / LP_TILE;
    p.sm_count = ctx->sm_count;
    p.part_ml = static_cast<float*>(ws);
    p.z_target = p.part_ml + static_cast<size_t>(T) * (p.unit_mode ? p.ntile128 : p.nsuper) * 2;
    p.inv_temperature = inv_temperature;
    p.dev_status = ctx->dev_status;
    cudaError_t e = launch_logprob(tmA, tmB, p, pair, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_token_logprob");
}

tik_status tik_rmsnorm(tik_ctx* ctx, const void* x, void* residual, const void* weight, void* y, float eps,
                       int64_t T, int H, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (T < 0 || H <= 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative or zero size");
    if (!(eps >= 0.0f) || !std::isfinite(eps)) return fail(ctx, TIK_ERR_INVALID_ARG, "eps must be finite and >= 0");
    if (H % 8 != 0 || H > 8192) return fail(ctx, TIK_ERR_UNSUPPORTED, "H must be a multiple of 8 and <= 8192");
    if (T == 0) return TIK_OK;
    if (!x || !weight || !y) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(x) || !aligned16(residual) || !aligned16(weight) || !aligned16(y))
        return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (T >= (1ll << 31)) return fail(ctx, TIK_ERR_UNSUPPORTED, "T must be < 2^31");
    NormParams p{};
    p.x = static_cast<const __nv_bfloat16*>(x);
    p.residual = static_cast<__nv_bfloat16*>(residual);
    p.weight = static_cast<const __nv_bfloat16*>(weight);
    p.y = static_cast<__nv_bfloat16*>(y);
    p.eps = eps;
    p.T = T;
    p.H = H;
    cudaError_t e = launch_rmsnorm(p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_rmsnorm");
}

tik_status tik_swiglu(tik_ctx* ctx, const void* gate_up, void* out, int64_t T, int I, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (T < 0 || I <= 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative or zero size");
    if (I % 8 != 0) return fail(ctx, TIK_ERR_UNSUPPORTED, "I must be a multiple of 8");
    if (T == 0) return TIK_OK;
    if (!gate_up || !out) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(gate_up) || !aligned16(out)) return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (T * (I / 8) >= (1ll << 39)) return fail(ctx, TIK_ERR_UNSUPPORTED, "T * I too large");
    cudaError_t e = launch_swiglu(gate_up, out, T, I, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_swiglu");
}

tik_status tik_linear(tik_ctx* ctx, const void* x, const void* weight, void* y, int64_t T, int K, int N,
                      void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (T < 0 || K <= 0 || N <= 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative or zero size");
    if (K % 64 != 0) return fail(ctx, TIK_ERR_UNSUPPORTED, "K must be a multiple of 64");
    if (N % 8 != 0) return fail(ctx, TIK_ERR_UNSUPPORTED, "N must be a multiple of 8");
    if (T == 0) return TIK_OK;
    if (!x || !weight || !y) return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(x) || !aligned16(weight) || !aligned16(y)) return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (T >= (1ll << 31) - 128) return fail(ctx, TIK_ERR_UNSUPPORTED, "T must be < 2^31 - 128");
    CUtensorMap tmA, tmB;
    std::string err;
    uint64_t ad[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(T)};
    uint64_t bd[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(N)};
    uint64_t st1[1] = {static_cast<uint64_t>(K) * 2};
    uint32_t box[2] = {64, 128};
    const bool pair = T > 128;           // CTA pairs (two-SM MMAs) as soon as there is more than one row tile
    // one row tile: the decode-shaped schedule (persistent CTAs over column units, only the rows
    // that exist staged); same MMA chain per output element, so the same bits
    const bool unit_mode = !pair;
    const int a_rows = T <= 32 ? 32 : T <= 64 ? 64 : 128;
    const int nu = unit_mode ? linear_unit_cols(N, a_rows, ctx->sm_count) : 0;
    uint32_t boxA[2] = {64, unit_mode ? static_cast<uint32_t>(a_rows) : 128u};
    uint32_t boxB[2] = {64, unit_mode ? static_cast<uint32_t>(nu) : pair ? 128u : 256u};
    CUtensorMap tmY;
    uint64_t yd[2] = {static_cast<uint64_t>(N), static_cast<uint64_t>(T)};
    uint64_t ys[1] = {static_cast<uint64_t>(N) * 2};
    if (!make_tmap_bf16(ctx, &tmA, x, 2, ad, st1, boxA, &err) || !make_tmap_bf16(ctx, &tmB, weight, 2, bd, st1, boxB, &err) ||
        !make_tmap_bf16(ctx, &tmY, y, 2, yd, ys, box, &err))
        return fail(ctx, TIK_ERR_CUDA, err.c_str());
    LinearParams p{};
    p.y = static_cast<__nv_bfloat16*>(y);
    p.T = T;
    p.K = K;
    p.N = N;
    // Columns per CTA (a "super-chunk" of 256-column steps): up to 16 steps amortise a CTA's set-up
    // and its last epilogue, which runs after the MMAs have ended; with few row tiles that would leave
    // SMs idle, so the number of super-chunks doubles until the grid covers the SMs four times.  The
    // steps are then dealt evenly (N = 5120: two super-chunks of 10 steps, not 16 + 4, whose short
    // CTAs left a quarter of the last wave idle).  An output element is one 256-column accumulator's
    // chain over K either way: its bits do not depend on this choice.
    const long long ntile = (T + 127) / 128;
    const int steps = (N + 255) / 256;
    int nsup = (steps + 15) / 16;
    while (nsup < steps && ntile * nsup < 4ll * ctx->sm_count) nsup = nsup * 2 < steps ? nsup * 2 : steps;
    const int per = (steps + nsup - 1) / nsup;
    p.super_cols = per * 256;
    p.nsuper = (steps + per - 1) / per;
    // two to sixteen row tiles (decode batches up to 256, prefill-sized calls up to 2048 rows): the pair
    // kernel, persistent over (256-column step, pair of row tiles) units -- a grid of one CTA pair per
    // unit spends as long on set-up as on a unit's 56 .. 432 K slices, and x fits L2
    const bool pair_units = pair && ntile <= 16;
    p.unit_mode = (unit_mode || pair_units) ? 1 : 0;
    p.nu = nu;
    p.ntp = static_cast<int>((ntile + 1) / 2);
    p.nunit = unit_mode ? (N + nu - 1) / nu : pair_units ? steps * p.ntp : 0;
    p.a_rows = a_rows;
    p.sm_count = ctx->sm_count;
    p.dev_status = ctx->dev_status;
    cudaError_t e = launch_linear(tmA, tmB, tmY, p, pair, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_linear");
}

tik_status tik_attn_train_bwd(tik_ctx* ctx, const void* q, const void* k, const void* v, const void* o,
                              const void* d_o, const float* lse, void* dq, void* dk, void* dv,
                              const int32_t* cu_seqlens, int S, int64_t total_tokens, int max_seqlen, int Hq,
                              int Hkv, int d, float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
    if (!ctx) return TIK_ERR_INVALID_ARG;
    if (S < 0 || total_tokens < 0 || max_seqlen < 0) return fail(ctx, TIK_ERR_INVALID_ARG, "negative size");
    tik_status st = check_heads(ctx, Hq, Hkv, d, softmax_scale);
    if (st != TIK_OK) return st;
    if (S == 0 || total_tokens == 0 || max_seqlen == 0) return TIK_OK;
    if (!q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv || !cu_seqlens)
        return fail(ctx, TIK_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv) || !aligned16(ws))
        return fail(ctx, TIK_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (total_tokens >= (1ll << 31)) return fail(ctx, TIK_ERR_UNSUPPORTED, "total_tokens must be < 2^31");
    const size_t need = tik_workspace_bytes(TIK_OP_ATTN_TRAIN_BWD, total_tokens, Hq, Hkv, d, 0, 0, 0);
    if (!ws || ws_bytes < need) return fail(ctx, TIK_ERR_WORKSPACE, "backward workspace too small");
    if (S > 65535 || Hq > 65535) return fail(ctx, TIK_ERR_UNSUPPORTED, "S and Hq must be <= 65535");

    CUtensorMap tmQ, tmK, tmV, tmDO;
    std::string err;
    const uint64_t ud = static_cast<uint64_t>(d);
    uint64_t qd[3] = {ud, static_cast<uint64_t>(Hq), static_cast<uint64_t>(total_tokens)};
    uint64_t qs[2] = {ud * 2, ud * 2 * Hq};
    uint64_t kd[3] = {ud, static_cast<uint64_t>(Hkv), static_cast<uint64_t>(total_tokens)};
    uint64_t ks[2] = {ud * 2, ud * 2 * Hkv};
    uint32_t box[3] = {64, 1, 128};
    if (!make_tmap_bf16(ctx, &tmQ, q, 3, qd, qs, box, &err) || !make_tmap_bf16(ctx, &tmDO, d_o, 3, qd, qs, box, &err) ||
        !make_tmap_bf16(ctx, &tmK, k, 3, kd, ks, box, &err) || !make_tmap_bf16(ctx, &tmV, v, 3, kd, ks, box, &err))
        return fail(ctx, TIK_ERR_CUDA, err.c_str());
    BwdParams p{};
    p.cu_seqlens = cu_seqlens;
    p.lse = lse;
    p.delta = static_cast<float*>(ws);
    p.dq = static_cast<__nv_bfloat16*>(dq);
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dv = static_cast<__nv_bfloat16*>(dv);
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.c = scale_to_c(softmax_scale);
    p.scale = softmax_scale;
    p.dev_status = ctx->dev_status;
    cudaError_t e = launch_attn_bwd(d, (max_seqlen + 127) / 128, S, tmQ, tmK, tmV, tmDO, p, o, d_o,
                                    total_tokens * Hq, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TIK_OK : cuda_fail(ctx, e, "tik_attn_train_bwd");
}

}  // extern "C"
