/*
 * CPU oracle for the DEER-GRU hot path: TEST INFRASTRUCTURE ONLY.
 * Only the test-suite, the smoke check and the benchmark's cpu_baseline /
 * reference arm may load this library; the CUDA product never does.
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fPIC -shared deer_oracle.c -lm
 * (no fast-math, no FMA contraction, so the fp32 trajectory is reproducible).
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REAL double
#define SFX f64
#define R_EXP exp
#define R_TANH tanh
#define R_ABS fabs
#define R_LOG log
#include "deer_oracle_impl.h"
#undef REAL
#undef SFX
#undef R_EXP
#undef R_TANH
#undef R_ABS
#undef R_LOG

#define REAL float
#define SFX f32
#define R_EXP expf
#define R_TANH tanhf
#define R_ABS fabsf
#define R_LOG logf
#include "deer_oracle_impl.h"
#undef REAL
#undef SFX
#undef R_EXP
#undef R_TANH
#undef R_ABS
#undef R_LOG

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
