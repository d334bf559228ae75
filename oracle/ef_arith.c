/*
 * TEST INFRASTRUCTURE ONLY — CPU oracle arithmetic for DD-EF-SGD (Algorithm 1 of the paper).
 *
 * This file holds the two element-wise fp32 steps of the method that numpy cannot express
 * with a single rounding.  Everything else of the oracle (selection, ring, policy) is plain
 * numpy / Python in the sibling modules.  Nothing here is shared with, imported by or linked
 * into the CUDA library; only tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it.
 *
 * Precision: the paper does not fix one.  State (error term, parameters) is fp32 and every
 * update is ONE fused multiply-add rounded to nearest-even, no flush-to-zero, so that the
 * integer decision that follows (which k entries are largest) is taken in the same
 * precision as the device path.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static float widen_bf16(uint16_t h)
{
    /* bfloat16 is the upper half of an IEEE-754 binary32: widening is exact. */
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/*
 * Algorithm 1, worker side, the argument of C_delta:  a_j = e_j + alpha * g_j
 * (alpha = gamma in the paper's form).  g is fp32 (g_is_bf16 == 0) or raw bfloat16 bits.
 */
void orc_accumulate(float alpha, const void *g, int g_is_bf16, const float *e,
                    float *a, uint64_t d)
{
    if (g_is_bf16) {
        const uint16_t *gh = (const uint16_t *)g;
        for (uint64_t j = 0; j < d; ++j)
            a[j] = fmaf(alpha, widen_bf16(gh[j]), e[j]);
    } else {
        const float *gf = (const float *)g;
        for (uint64_t j = 0; j < d; ++j)
            a[j] = fmaf(alpha, gf[j], e[j]);
    }
}

/*
 * Algorithm 1, server side:  x_j <- x_j - scale * S_j, written as one fused multiply-add
 * with the negated scale.
 */
void orc_apply(float neg_scale, const float *S, float *x, uint64_t d)
{
    for (uint64_t j = 0; j < d; ++j)
        x[j] = fmaf(neg_scale, S[j], x[j]);
}
