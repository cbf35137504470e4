// tik_attn_decode_static: decode attention for callers that cannot allocate device memory.
//
// Some users of this library run where a device allocation is not an option: a serving
// process that handed every free byte of the GPU to its KV-cache pool at start-up (a later
// cudaMalloc simply fails), or a latency-critical decode loop that must not hit the
// device-wide synchronisation that cudaMalloc / cudaFree imply.  tik_create needs one small
// allocation and tik_attn_decode needs a caller-allocated workspace; this entry point needs
// neither.  Its split-KV scratch (the per-chunk partial results that the combine kernel
// folds) lives in a file-scope __device__ array of TIK_STATIC_SCRATCH_BYTES, and so does its
// device flag word.  Every GPU that loads the library holds those bytes until the process
// exits.
//
// The kernels are the ones tik_attn_decode launches, so the output bits are the same.
#include <cmath>
#include <mutex>

#include "../../include/tik.h"
#include "tik_core.cuh"
#include "tik_internal.h"

namespace {

constexpr size_t kScratchBytes = TIK_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// In host code these names are only host-side stand-ins for the device symbols: their
// device addresses come from cudaGetSymbolAddress below, never from `&` or decay.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];
static __device__ __align__(256) int g_static_flags[64];

struct DeviceSetup {
    bool ready = false;
    void* scratch = nullptr;     // device address of g_static_scratch on this device
    int* flags = nullptr;        // device address of g_static_flags on this device
    void* encode_tiled = nullptr;
    int sm_count = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current: resolve the device addresses of the static
// arrays and the driver's tensor-map encoder.  Allocates nothing.
cudaError_t setup_device(int device, DeviceSetup** out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[device];
    if (!s.ready) {
        void* scratch = nullptr;
        void* flags = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&scratch, g_static_scratch);
        if (e != cudaSuccess) return e;
        e = cudaGetSymbolAddress(&flags, g_static_flags);
        if (e != cudaSuccess) return e;
        cudaDriverEntryPointQueryResult qres;
        void* fn = nullptr;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        s.scratch = scratch;
        s.flags = static_cast<int*>(flags);
        s.encode_tiled = fn;
        if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) s.sm_count = 0;
        s.ready = true;
    }
    *out = &s;
    return cudaSuccess;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" tik_status tik_attn_decode_static(const void* q, void* o, float* lse, const int32_t* ctx_lens,
                                             const void* k_cache, const void* v_cache,
                                             const int32_t* block_table, int max_blocks, int B,
                                             int max_ctx_len, int Hq, int Hkv, int d, int page_size,
                                             int num_pages, float softmax_scale, int* dev_flags,
                                             void* stream) {
    using namespace tik;
    if (B < 0 || max_ctx_len < 0 || max_blocks < 0 || num_pages < 0) return TIK_ERR_INVALID_ARG;
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return TIK_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.0f) || !std::isfinite(softmax_scale)) return TIK_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TIK_ERR_UNSUPPORTED;
    if (Hq / Hkv > 32) return TIK_ERR_UNSUPPORTED;
    if (page_size != 16 && page_size != 32 && page_size != 64 && page_size != 128) return TIK_ERR_UNSUPPORTED;
    if (B == 0 || max_ctx_len == 0) return TIK_OK;
    if (!q || !o || !ctx_lens || !k_cache || !v_cache || !block_table || num_pages == 0) return TIK_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(o) || !aligned16(k_cache) || !aligned16(v_cache)) return TIK_ERR_UNSUPPORTED;
    if (B > 65535 || Hkv > 65535) return TIK_ERR_UNSUPPORTED;

    // the scratch has a fixed size: larger problems are refused, never truncated
    const size_t need = tik_workspace_bytes(TIK_OP_ATTN_DECODE, B, Hq, Hkv, d, max_ctx_len, 0, 0);
    if (need > kScratchBytes) return TIK_ERR_WORKSPACE;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return TIK_ERR_CUDA;
    DeviceSetup* s = nullptr;
    if (setup_device(device, &s) != cudaSuccess) return TIK_ERR_CUDA;

    tik_ctx local;                       // host-only carrier for the encoder pointer
    local.device = device;
    local.encode_tiled = s->encode_tiled;
    CUtensorMap tmQ, tmK, tmV;
    std::string err;
    const uint64_t ud = static_cast<uint64_t>(d);
    const int G = Hq / Hkv;
    uint64_t qd[3] = {ud, static_cast<uint64_t>(Hq), static_cast<uint64_t>(B)};
    uint64_t qs[2] = {ud * 2, ud * 2 * Hq};
    uint32_t qbox[3] = {64, static_cast<uint32_t>(G), 1};
    uint64_t cd[4] = {ud, static_cast<uint64_t>(page_size), static_cast<uint64_t>(Hkv),
                      static_cast<uint64_t>(num_pages)};
    uint64_t cs[3] = {ud * 2, ud * 2 * page_size, ud * 2 * page_size * Hkv};
    uint32_t cbox[4] = {64, static_cast<uint32_t>(page_size), 1, 1};
    if (!make_tmap_bf16(&local, &tmQ, q, 3, qd, qs, qbox, &err) ||
        !make_tmap_bf16(&local, &tmK, k_cache, 4, cd, cs, cbox, &err) ||
        !make_tmap_bf16(&local, &tmV, v_cache, 4, cd, cs, cbox, &err))
        return TIK_ERR_CUDA;

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
    p.c = softmax_scale * LOG2E_F;
    p.nchunk_max = nchunk;
    p.direct_out = nchunk == 1 ? 1 : 0;
    p.max_ctx = max_ctx_len;
    // Every chunk partial that the combine kernel reads is written by the decode kernel of
    // this same call first, so stale contents of the shared scratch are never consumed.
    p.part_o = static_cast<float*>(s->scratch);
    p.part_ml = p.part_o + static_cast<size_t>(B) * Hq * nchunk * d;
    p.dev_status = dev_flags ? dev_flags : s->flags;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    // The library's own flag word keeps the last call's flags; a stale "wait expired" would
    // make every later kernel bail out, so it is cleared (stream-ordered) before each use.
    if (!dev_flags) e = cudaMemsetAsync(s->flags, 0, sizeof(int), st);
    p.cpc = 1;
    if (e == cudaSuccess)
        e = (G <= DECODE2_MAX_G && (B * Hkv <= s->sm_count || nchunk <= 2) && 4ll * B * Hkv * nchunk >= 3ll * s->sm_count) ? launch_decode2(d, dim3(nchunk, Hkv, B), tmQ, tmK, tmV, p, st)
                               : launch_attn(d, 2, dim3(nchunk, Hkv, B), tmQ, tmK, tmV, p, st);
    if (e == cudaSuccess && !p.direct_out) e = launch_combine(d, p, B, st);
    return e == cudaSuccess ? TIK_OK : TIK_ERR_CUDA;
}
