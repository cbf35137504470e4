// The numerical contract shared by every regime (packed train-forward, paged prefill,
// paged decode, split-KV combine) and by the log-probability kernels.
//
// Section 5.3 of the paper lists what decides the bits of unified attention: the
// reduction orders of QK^T, PV, online softmax and final normalisation; where and in
// which precision scaling and masking happen; the exact exp / reciprocal instructions
// and flush-to-zero behaviour; the bf16<->fp32 conversion points and the order of
// rescale, update and normalise.  Section 3.2 adds that KV-tile boundaries determine
// rescaling, P rounding and PV order.  This header fixes each of those once; all
// kernels call these functions and nothing else for that arithmetic.
//
//   * KV tile: 128 keys at absolute positions [128 j, 128 j + 128), ascending j.
//   * Chunk: 2048 keys (16 tiles), absolute-aligned.  The running state (m, l, O) is
//     reset at every chunk start in every regime; chunks are folded in ascending order.
//   * Scores: fp32 accumulators of a K=16 tcgen05 MMA chain (ascending over head_dim).
//   * c = softmax_scale * log2(e), one fp32 multiply on the host.
//   * Mask: select -inf where key position > query position (no arithmetic on masked
//     scores, so masked K contents never matter).
//   * Per tile and row: the reference m moves to the tile maximum only when that exceeds it
//     by more than 8 in the exponent, (tile max - m) * c > 8 (so always on the first tile of
//     a chunk), else m' = m; p = ex2.approx.ftz(fma(s, c, -(m' * c)));
//     row sums in the fixed two-halves-of-four-chains shape below; alpha = ex2.approx.ftz((m - m') * c);
//     l_half = fma(l_half, alpha, rowsum of that 64-column half); O = O * alpha with a non-flushing IEEE multiply (so
//     skipping it when alpha == 1.0f is bit-neutral); P rounded to bf16 (RNE) for the PV
//     MMA while l sums the unrounded fp32 p.
//   * Finalise: l = l_lo + l_hi; o = O * rcp.rn(l), rounded to bf16 (RNE).
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>
#include <stdint.h>

namespace tik {

constexpr int BN = 128;               // keys per KV tile
constexpr int BM = 128;               // query rows per MMA tile
constexpr int CHUNK = 2048;           // keys per split chunk
constexpr int TILES_PER_CHUNK = CHUNK / BN;
constexpr float LOG2E_F = 1.44269504088896340736f;
constexpr float LN2_F = 0.69314718055994530942f;
constexpr int LP_TILE = 128;          // vocabulary columns per log-sum-exp tile
constexpr int LP_SUPER = 1024;        // vocabulary columns per super-chunk (8 tiles)
constexpr int LP_UNIT_MODE_ROWS = 2048; // log-prob calls of at most this many rows keep one partial per tile (schedule only)

#define TIK_CONTRACT_ID "tik3-BN128-CH2048-M128N128K16-ex2ftz-lazy8-sum2x4-LP128x1024"

__device__ __forceinline__ float ex2_ftz(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Row sums have a fixed shape.  The 128 columns of a tile are two halves of 64; within a
// half, chain k adds the columns with (col / 2) % 4 == k in ascending order and the four
// chains are combined as (a0+a1)+(a2+a3).  Attention keeps the two halves apart for the
// whole computation: every row carries (l_lo, l_hi), each updated as l = fma(l, alpha, half
// sum), folded across chunks separately, and added only once, right before the final
// reciprocal.  So a row can be summed by one thread, by two threads owning 64 columns each,
// or by four threads owning interleaved column pairs, with identical bits.
struct RowSum4 {
    float a[4];
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = 0.0f;
    }
    __device__ __forceinline__ float total() const {
        return __fadd_rn(__fadd_rn(a[0], a[1]), __fadd_rn(a[2], a[3]));
    }
};
// `col` (0..63 within the half) must be a compile-time constant after unrolling.
__device__ __forceinline__ void rowsum_add(RowSum4& s, int col, float p) {
    const int chain = (col >> 1) & 3;
    s.a[chain] = __fadd_rn(s.a[chain], p);
}
// The log-probability kernels sum a 128-column tile as half(0..63) + half(64..127).
struct RowSum8 {
    RowSum4 h[2];
    __device__ __forceinline__ void reset() {
        h[0].reset();
        h[1].reset();
    }
    __device__ __forceinline__ float total() const { return __fadd_rn(h[0].total(), h[1].total()); }
};
__device__ __forceinline__ void rowsum_add(RowSum8& s, int col, float p) {
    rowsum_add(s.h[col >> 6], col & 63, p);
}

// max of three (the maximum is exact, so its evaluation order is free)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// Reference maximum after a tile whose (masked) maximum is mt.  The reference only moves when
// the tile maximum exceeds it by more than 2^RESCALE_LOG2 in the exponent (always on the first
// tile of a chunk, where it is -inf); otherwise it stays, weights may reach 2^RESCALE_LOG2
// instead of 1, alpha is exactly 1 and the accumulator is not rescaled.  The decision reads
// only the row's own scores and the fixed tile boundaries, so it is the same in every regime.
constexpr float RESCALE_LOG2 = 8.0f;
__device__ __forceinline__ float softmax_next_max(float m_ref, float mt, float c) {
    const float growth = __fmul_rn(__fsub_rn(mt, m_ref), c);
    return (growth > RESCALE_LOG2) ? mt : m_ref;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), RNE
    return *reinterpret_cast<uint32_t*>(&t);
}

// Two-wide forms of the same IEEE operations (fma.rn / add.rn on f32 pairs): identical bits to
// the scalar intrinsics, half the issue slots.
__device__ __forceinline__ void fma_rn_x2(float& d0, float& d1, float a0, float a1, float b, float c) {
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void add_rn_x2(float& a0, float& a1, float b0, float b1) {
    asm("{\n\t.reg .b64 ra, rb;\n\t"
        "mov.b64 ra, {%0, %1};\n\tmov.b64 rb, {%2, %3};\n\t"
        "add.rn.f32x2 ra, ra, rb;\n\tmov.b64 {%0, %1}, ra;\n\t}"
        : "+f"(a0), "+f"(a1)
        : "f"(b0), "f"(b1));
}
// Weights and half-row sum of 8 consecutive columns (chains 0,0,1,1,2,2,3,3): every chain still
// receives its columns in ascending order, two chains per packed add.  The two steps are also
// available separately: decode computes the weights of a row on four warps and sums on one.
__device__ __forceinline__ void softmax_x8(const uint32_t* s8, float c, float neg_mc, float* x) {
#pragma unroll
    for (int i = 0; i < 8; i += 2)
        fma_rn_x2(x[i], x[i + 1], __uint_as_float(s8[i]), __uint_as_float(s8[i + 1]), c, neg_mc);
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = ex2_ftz(x[i]);
}
__device__ __forceinline__ void softmax_sum_pack8(const float* x, RowSum4& rs, uint32_t* pk4) {
    add_rn_x2(rs.a[0], rs.a[1], x[0], x[2]);
    add_rn_x2(rs.a[2], rs.a[3], x[4], x[6]);
    add_rn_x2(rs.a[0], rs.a[1], x[1], x[3]);
    add_rn_x2(rs.a[2], rs.a[3], x[5], x[7]);
#pragma unroll
    for (int i = 0; i < 4; ++i) pk4[i] = pack_bf16x2(x[2 * i], x[2 * i + 1]);
}
__device__ __forceinline__ void softmax_p8(const uint32_t* s8, float c, float neg_mc, RowSum4& rs, uint32_t* pk4) {
    float x[8];
    softmax_x8(s8, c, neg_mc, x);
    softmax_sum_pack8(x, rs, pk4);
}

// exponent argument of one score: s * c - mc, one fused multiply-add.
__device__ __forceinline__ float softmax_p(float s, float c, float neg_mc) {
    return ex2_ftz(__fmaf_rn(s, c, neg_mc));
}
// rescale factor when the row maximum moves from m_old to m_new (m_new >= m_old).
// Subtract first: m_new == m_old gives ex2(0) = 1.0f exactly; m_old = -inf gives 0.
__device__ __forceinline__ float softmax_alpha(float m_old, float m_new, float c) {
    return ex2_ftz(__fmul_rn(__fsub_rn(m_old, m_new), c));
}
__device__ __forceinline__ float rescale_o(float o, float alpha) { return __fmul_rn(o, alpha); }


// Fold chunk state (m_c, l_c, O_c) into the global state (M, L, O).  The global state is
// initialised by copying chunk 0; chunks 1, 2, ... are folded in ascending order.
struct FoldCoef {
    float A, B, M_new;
};
__device__ __forceinline__ FoldCoef fold_coef(float M, float m_c, float c) {
    FoldCoef f;
    f.M_new = fmaxf(M, m_c);
    f.A = ex2_ftz(__fmul_rn(__fsub_rn(M, f.M_new), c));
    f.B = ex2_ftz(__fmul_rn(__fsub_rn(m_c, f.M_new), c));
    return f;
}
__device__ __forceinline__ float fold_value(float X, float x_c, const FoldCoef& f) {
    return __fmaf_rn(X, f.A, __fmul_rn(x_c, f.B));
}

__device__ __forceinline__ float finalize_l(float l_lo, float l_hi) { return __fadd_rn(l_lo, l_hi); }
__device__ __forceinline__ float finalize_inv(float L) { return __frcp_rn(L); }
__device__ __forceinline__ float finalize_o(float O, float inv) { return __fmul_rn(O, inv); }
// natural-log log-sum-exp of the scaled scores: (M * c + log2 L) * ln 2
__device__ __forceinline__ float finalize_lse(float M, float L, float c) {
    return __fmul_rn(__fadd_rn(__fmul_rn(M, c), log2f(L)), LN2_F);
}

// ---- log-probability: tile (m, l) with natural-exponent semantics via exp2 ----------
// l_j = sum ex2(fma(z, log2e, -(m_j * log2e))) in the RowSum8 shape; tiles and super-chunks
// are folded sequentially in ascending column order with fold_coef(c = log2e).
__device__ __forceinline__ float lp_lse(float M, float L) {
    return __fadd_rn(M, __fmul_rn(log2f(L), LN2_F));
}

// ---- pre-attention step: per-head RMSNorm and NeoX rotation of one (token, head) vector ------
// Sixteen lanes hold the vector: lane l has EP = d/32 consecutive elements of the first half and
// their partners i + d/2.  Sum of squares: per lane a fused chain over lo[0..EP), then hi[0..EP),
// then a butterfly over lane distances 8, 4, 2, 1 (both partners of an exchange add the same two
// numbers, so all sixteen lanes end with the same total).
template <int EP>
__device__ __forceinline__ float prep_sum_squares(const float* lo, const float* hi) {
    float part = __fmul_rn(lo[0], lo[0]);
#pragma unroll
    for (int e = 1; e < EP; ++e) part = __fmaf_rn(lo[e], lo[e], part);
#pragma unroll
    for (int e = 0; e < EP; ++e) part = __fmaf_rn(hi[e], hi[e], part);
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) part = __fadd_rn(part, __shfl_xor_sync(0xffffffffu, part, off));
    return part;
}
// 1 / sqrt(ss / d + eps), correctly rounded reciprocal square root of one fused multiply-add
__device__ __forceinline__ float prep_inv_rms(float ss, float inv_d, float eps) {
    return __frsqrt_rn(__fmaf_rn(ss, inv_d, eps));
}
__device__ __forceinline__ float prep_norm(float x, float inv, float w) { return __fmul_rn(__fmul_rn(x, inv), w); }
// (lo, hi) <- (lo cos - hi sin, hi cos + lo sin): four products and two sums, none fused
__device__ __forceinline__ void prep_rotate(float& lo, float& hi, float cs, float sn) {
    const float a = __fsub_rn(__fmul_rn(lo, cs), __fmul_rn(hi, sn));
    const float b = __fadd_rn(__fmul_rn(hi, cs), __fmul_rn(lo, sn));
    lo = a;
    hi = b;
}

// ---- hidden RMSNorm (optionally fused with the residual add) and SwiGLU ----------------------
// Row of H elements on 128 threads: thread t holds the 8-element vectors t, t + 128, ... in
// ascending order.  Residual form: s = bf16(fp32(x) + fp32(res)) is what is stored and what is
// normalised.  Sum of squares: per thread one fused chain over its elements in that order, a
// butterfly over lane distances 16..1, then the four warp totals as (w0 + w1) + (w2 + w3).
__device__ __forceinline__ float hn_residual_sum(float x, float res) {
    return __bfloat162float(__float2bfloat16_rn(__fadd_rn(x, res)));
}
__device__ __forceinline__ float hn_warp_total(float part) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) part = __fadd_rn(part, __shfl_xor_sync(0xffffffffu, part, off));
    return part;
}
__device__ __forceinline__ float hn_block_total(const float* w4) {
    return __fadd_rn(__fadd_rn(w4[0], w4[1]), __fadd_rn(w4[2], w4[3]));
}
// silu(g) * u with silu(g) = g * 1 / (1 + 2^(-g log2 e)): ex2.approx, correctly rounded reciprocal
__device__ __forceinline__ float swiglu_value(float g, float u) {
    const float e = ex2_ftz(__fmul_rn(g, -LOG2E_F));
    const float sig = __frcp_rn(__fadd_rn(1.0f, e));
    return __fmul_rn(__fmul_rn(g, sig), u);
}

// ---- attention backward: weight and score gradient of one (query, key) pair ------------------
// p = 2^(s c - lse log2 e) with the forward's log-sum-exp; ds = p (dp - delta): the softmax scale
// is applied once per output element when dQ / dK leave their fp32 accumulators.
__device__ __forceinline__ float bwd_p(float s, float c, float lse_log2) { return ex2_ftz(__fmaf_rn(s, c, -lse_log2)); }
__device__ __forceinline__ float bwd_ds(float p, float dp, float delta) { return __fmul_rn(p, __fsub_rn(dp, delta)); }
// the same for two neighbouring columns with two-wide instructions (identical roundings)
__device__ __forceinline__ void bwd_pds_x2(float s0, float s1, float dp0, float dp1, float c, float nl2_0, float nl2_1,
                                           float ndl0, float ndl1, float& p0, float& p1, float& ds0, float& ds1) {
    float x0, x1, t0, t1;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %6};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(x0), "=f"(x1)
        : "f"(s0), "f"(s1), "f"(c), "f"(nl2_0), "f"(nl2_1));
    p0 = ex2_ftz(x0);
    p1 = ex2_ftz(x1);
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(t0), "=f"(t1)
        : "f"(dp0), "f"(dp1), "f"(ndl0), "f"(ndl1));
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(ds0), "=f"(ds1)
        : "f"(p0), "f"(p1), "f"(t0), "f"(t1));
}

}  // namespace tik
