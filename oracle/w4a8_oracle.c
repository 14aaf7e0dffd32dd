/*
 * Plain-C statement of the W4A8 linear (Sec. 3.4 "Quantization"): TEST INFRASTRUCTURE ONLY.
 *
 * The same definition as oracle/w4a8_oracle.py, written as straightforward loops so
 * that full-size shapes finish in seconds and so that it can serve as the timed CPU
 * baseline.  Exact int32 per-group partials, fp64 scaling, group index ascending.
 * No tiling, no intrinsics, no code shared with the CUDA library; it reads the
 * UNPACKED codes qw[N,K] and knows nothing of the device layout.
 *
 *   s_a[m]   = fp16_rne(max_k |x[m,k]| / 127)  (saturating at 65504)
 *   q_a[m,k] = clamp(rne(x[m,k] / s_a[m]), -127, 127), all zero when s_a[m] == 0
 *   D[m,g,n] = sum_{k in g} q_w[n,k] q_a[m,k] - z[g,n] sum_{k in g} q_a[m,k]
 *   ref[m,n] = s_a[m] * sum_g s_w[g,n] * D[m,g,n]
 *
 * Build: gcc -O3 -march=native -fopenmp -shared -fPIC (see oracle/cfast.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double fp16_to_double(uint16_t h) {
    int sign = h >> 15, e = (h >> 10) & 31, mant = h & 1023;
    double v;
    if (e == 0)       v = ldexp((double)mant, -24);
    else if (e == 31) v = mant ? NAN : INFINITY;
    else              v = ldexp(1.0 + mant / 1024.0, e - 15);
    return sign ? -v : v;
}

/* non-negative double -> binary16 bits, round to nearest even, saturate at 65504 */
static uint16_t double_to_fp16_sat(double q) {
    if (!(q > 0.0)) return 0;
    if (q > 65504.0) q = 65504.0;
    int ex;
    frexp(q, &ex);                 /* q = f * 2^ex, f in [0.5,1)  =>  2^(ex-1) <= q */
    int e = ex - 1;
    if (e < -14) e = -14;
    double ulp = ldexp(1.0, e - 10);
    double r = nearbyint(q / ulp) * ulp;   /* default rounding mode: ties to even */
    if (r == 0.0) return 0;
    if (r < ldexp(1.0, -14)) return (uint16_t)(r / ldexp(1.0, -24));
    frexp(r, &ex);
    e = ex - 1;
    int mant = (int)((r / ldexp(1.0, e) - 1.0) * 1024.0);
    return (uint16_t)(((e + 15) << 10) | mant);
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* O1.  x: bf16 bits [M,K]; qa int8 [M,K]; sa fp16 bits [M]; asum int32 [M,K/group]. */
void oracle_quantize_act(const uint16_t* x, int M, int K, int group,
                         int8_t* qa, uint16_t* sa, int32_t* asum) {
    int G = K / group;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t* xr = x + (size_t)m * K;
        double amax = 0.0;
        for (int k = 0; k < K; ++k) {
            double a = fabs(bf16_to_double(xr[k]));
            if (a > amax) amax = a;
        }
        uint16_t sb = double_to_fp16_sat(amax / 127.0);
        sa[m] = sb;
        double s = fp16_to_double(sb);
        for (int g = 0; g < G; ++g) {
            int32_t sum = 0;
            for (int k = g * group; k < (g + 1) * group; ++k) {
                int q = 0;
                if (s != 0.0) {
                    double r = nearbyint(bf16_to_double(xr[k]) / s);
                    if (r > 127.0) r = 127.0;
                    if (r < -127.0) r = -127.0;
                    q = (int)r;
                }
                qa[(size_t)m * K + k] = (int8_t)q;
                sum += q;
            }
            asum[(size_t)m * G + g] = sum;
        }
    }
}

/*
 * O2 + O3.  qa int8 [M,K]; sa fp16 bits [M]; qw codes [N,K] one per byte; sw fp16 bits
 * [G,N]; z [G,N] one per byte.  ref: fp64 [M,N].  D: NULL or int32 [M,G,N].
 */
void oracle_linear(const int8_t* qa, const uint16_t* sa,
                   const uint8_t* qw, const uint16_t* sw, const uint8_t* z,
                   int M, int N, int K, int group, double* ref, int32_t* D) {
    int G = K / group;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        const uint8_t* wr = qw + (size_t)n * K;
        for (int m = 0; m < M; ++m) ref[(size_t)m * N + n] = 0.0;
        for (int g = 0; g < G; ++g) {
            double s = fp16_to_double(sw[(size_t)g * N + n]);
            int32_t zp = z[(size_t)g * N + n];
            for (int m = 0; m < M; ++m) {
                const int8_t* ar = qa + (size_t)m * K;
                int32_t p = 0, a = 0;
                for (int k = g * group; k < (g + 1) * group; ++k) {
                    p += (int32_t)wr[k] * (int32_t)ar[k];
                    a += (int32_t)ar[k];
                }
                int32_t d = p - zp * a;
                if (D) D[((size_t)m * G + g) * N + n] = d;
                ref[(size_t)m * N + n] += s * (double)d;
            }
        }
        for (int m = 0; m < M; ++m) ref[(size_t)m * N + n] *= fp16_to_double(sa[m]);
    }
}
