// Register-FFT kernels of libkvq, variant: one scale per vector, 8-bit codes (Sec. 3.2 steps 3-4).
#include "kvq_fft_kernels.cuh"

KVQ_FFT_DEFINE_VARIANT(fft_encode_gd_b8, fft_decode_gd_b8, 0, 8)
