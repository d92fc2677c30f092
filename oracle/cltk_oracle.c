/*
 * CLT-k oracle -- TEST INFRASTRUCTURE.
 *
 * A plain, slow, single-threaded CPU statement of one ScaleCom iteration
 * (Algorithm 1 with the CLT-k compressor of Eq. 2-3 and the low-pass-filtered
 * memory of Eq. 4), in fp32 and in fp64.  It exists so that tests, the smoke
 * check and the benchmark's CPU-baseline leg have something independent to
 * compare the CUDA library against.  It shares no code with that library and
 * nothing in the product path may call it.
 *
 * Build:  gcc -std=c99 -O2 -ffp-contract=off -fPIC -shared cltk_oracle.c -o libcltk_oracle.so -lm
 * (-ffp-contract=off: no fused multiply-add, so every operation rounds once.)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define REAL float
#define UKEY uint32_t
#define ABS_MASK 0x7FFFFFFFu
#define FN(name) name##_f32
#include "cltk_oracle_body.inc"
#undef REAL
#undef UKEY
#undef ABS_MASK
#undef FN

#define REAL double
#define UKEY uint64_t
#define ABS_MASK 0x7FFFFFFFFFFFFFFFull
#define FN(name) name##_f64
#include "cltk_oracle_body.inc"
#undef REAL
#undef UKEY
#undef ABS_MASK
#undef FN
