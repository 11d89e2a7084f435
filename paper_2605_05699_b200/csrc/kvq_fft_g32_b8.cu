// Register-FFT kernels of libkvq, variant: groups of 32, 8-bit codes.
#include "kvq_fft_kernels.cuh"

KVQ_FFT_DEFINE_VARIANT(fft_encode_g32_b8, fft_decode_g32_b8, 32, 8)
