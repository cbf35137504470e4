/* CPU oracle for causal grouped-query attention, token log-probability and the pre-attention
 * step (RMSNorm -> NeoX RoPE; the indexed cache write is a numpy index copy in __init__.py).
 *
 * TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load this library.  It shares no code,
 * header, table or helper with the CUDA kernels and neither side includes the
 * other.
 *
 * Two instantiations of the same plain definitions (see oracle_impl.inc):
 *   oracle_*      all arithmetic in fp64 (the oracle proper)
 *   oracle_*_f32  all arithmetic in fp32 (a cross-check that bounds how much
 *                 of the GPU-vs-oracle tolerance plain fp32 rounding uses up)
 *
 * Pins (tests/test_oracle_*.py): softmax rows sum to one; identical keys give
 * the running mean of V; position 0 returns V[0]; a dominant key returns its
 * value; causality; GQA equals MHA with repeated KV; key-shift invariance;
 * brute-force loops on tiny inputs; library attention / log_softmax on a
 * textbook case; zero weights give -ln V; one-hot logits in closed form;
 * paged storage equals packed storage.  Pre-attention step (tests/test_oracle_prep.py): RoPE as
 * numpy's complex product on the pairs (i, i + d/2); position 0 is the identity; norms kept and
 * scores a function of relative position; RMSNorm against closed forms and torch's rms_norm in
 * fp64; norm before rotation; the cos/sin table against hand values and the angle-addition
 * identity; the cache write against its index definition.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REAL double
#define R_EXP exp
#define R_LOG log
#define FN(name) name
#include "oracle_impl.inc"
#undef REAL
#undef R_EXP
#undef R_LOG
#undef FN

#define REAL float
#define R_EXP expf
#define R_LOG logf
#define FN(name) name##_f32
#include "oracle_impl.inc"
#undef REAL
#undef R_EXP
#undef R_LOG
#undef FN

/* Threads the parallel regions will use (for the benchmark's report). */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
