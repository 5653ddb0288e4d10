/*
 * Host-side check of the division sequence the CUDA kernels use for bfloat16 operands:
 *     r = RN(1/m);  q0 = RN(w r);  e = fma(-q0, m, w);  q = fma(e, r, q0).
 * Every operation is IEEE binary32 (fmaf is exact-then-rounded on the host as on the GPU), so
 * the comparison with w / m carries over.  Returns the number of operand pairs for which the
 * sequence differs from the IEEE quotient; *checked receives the number of pairs tried.
 *
 * Pairs: every bf16 m with 2^-60 <= |m| <= 2^60 (the kernels' div_safe range), every bf16 w
 * with |w| <= |m| whose exponent lies within `span` binades below m's, both signs of both.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static float bf16(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static int differs(float w, float m)
{
    float r = 1.0f / m;
    float q0 = w * r;
    float e = fmaf(-q0, m, w);
    float q = fmaf(e, r, q0);
    float t = w / m;
    return memcmp(&q, &t, 4) != 0;
}

long fast_division_mismatches(int span, long *checked)
{
    long bad = 0, tot = 0;
    for (uint32_t hm = 0; hm < 0x8000; ++hm) {
        int em = (hm >> 7) & 0xff;
        if (em < 67 || em > 187) /* 2^-60 .. 2^60 */
            continue;
        float m = bf16((uint16_t)hm);
        for (int ew = em - span; ew <= em; ++ew) {
            if (ew < 1)
                continue;
            for (uint32_t mw = 0; mw < 128; ++mw) {
                float w = bf16((uint16_t)((ew << 7) | mw));
                if (w > m)
                    continue;
                bad += differs(w, m) + differs(-w, m) + differs(w, -m) + differs(-w, -m);
                tot += 4;
            }
        }
    }
    *checked = tot;
    return bad;
}

/* A deliberately wrong variant (one Newton step missing) must be caught by the same sweep. */
long truncated_sequence_mismatches(long *checked)
{
    long bad = 0, tot = 0;
    for (uint32_t hm = 0x3f80; hm < 0x4000; ++hm)
        for (uint32_t hw = 0x3f00; hw < 0x3f80; ++hw) {
            float m = bf16((uint16_t)hm), w = bf16((uint16_t)hw);
            float q0 = w * (1.0f / m), t = w / m;
            bad += memcmp(&q0, &t, 4) != 0;
            ++tot;
        }
    *checked = tot;
    return bad;
}
