/*
 * Exhaustive check of the residual-corrected division the weight kernels use under one scale per row or group:
 *     s  = fl32(m / qmax)            (Eq. 2: the scale of a row whose absolute maximum is m)
 *     rs = fl32(1 / s)
 *     q0 = fl32(x * rs),  r = fma(-q0, s, x),  u = fma(r, rs, q0)
 * must equal the IEEE quotient fl32(x / s) for every 16-bit element x and every 16-bit maximum m.  Scaling x or m
 * by a power of two scales every intermediate value by a power of two as well (all of them normal numbers in the
 * range the kernels accept), so it is enough to enumerate the significands: integers 1..2047 cover every fp16
 * significand (11 bits, subnormals included) and every bf16 one (8 bits).  Prints the number of mismatches.
 */
#include <math.h>
#include <stdio.h>

int main(void) {
    const int qmaxs[2] = {7, 127};
    long total = 0, bad = 0;
    for (int qi = 0; qi < 2; ++qi) {
        for (int mm = 1; mm <= 2047; ++mm) {
            const float m = (float)mm;
            const float s = m / (float)qmaxs[qi];
            const float rs = 1.0f / s;
            for (int mx = 1; mx <= 2047; ++mx) {
                const float x = (float)mx;
                const float q0 = x * rs;
                const float r = fmaf(-q0, s, x);
                const float u = fmaf(r, rs, q0);
                const float want = x / s;
                ++total;
                if (!(u == want)) {
                    if (bad < 5) printf("mismatch qmax %d m %d x %d: %.9g vs %.9g\n", qmaxs[qi], mm, mx, (double)u, (double)want);
                    ++bad;
                }
            }
        }
    }
    printf("pairs %ld mismatches %ld\n", total, bad);
    return bad != 0;
}
