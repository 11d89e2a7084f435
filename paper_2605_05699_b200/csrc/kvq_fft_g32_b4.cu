// Register-FFT kernels of libkvq, variant: groups of 32, 4-bit codes: the fused layout of Sec. 7.1.
#include "kvq_fft_kernels.cuh"

KVQ_FFT_DEFINE_VARIANT(fft_encode_g32_b4, fft_decode_g32_b4, 32, 4)
