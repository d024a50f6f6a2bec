// Host-side bridge to the CUDA toolkit's own FP4 / FP8 conversion routines (cuda_fp4.h,
// cuda_fp8.h), used by the CPU tests as an independent library pin for the oracle's
// hand-written E2M1 and E4M3 rounding.  Nothing here runs on a GPU.
#include <cuda_fp4.h>
#include <cuda_fp8.h>

extern "C" unsigned char pin_e2m1(float x) {
    return (unsigned char)__nv_cvt_float_to_fp4(x, __NV_E2M1, cudaRoundNearest);
}
extern "C" unsigned char pin_e4m3(float x) {
    return (unsigned char)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
}
