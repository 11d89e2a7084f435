// Picks the register-FFT kernel variant for a plan's group size and bit width.
#include "kvq_internal.h"

namespace kvq {

#define KVQ_FFT_VARIANT_DECL(NAME) cudaError_t NAME(int D, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream);
KVQ_FFT_VARIANT_DECL(fft_encode_g32_b4)
KVQ_FFT_VARIANT_DECL(fft_decode_g32_b4)
KVQ_FFT_VARIANT_DECL(fft_encode_gd_b4)
KVQ_FFT_VARIANT_DECL(fft_decode_gd_b4)
KVQ_FFT_VARIANT_DECL(fft_encode_g32_b8)
KVQ_FFT_VARIANT_DECL(fft_decode_g32_b8)
KVQ_FFT_VARIANT_DECL(fft_encode_gd_b8)
KVQ_FFT_VARIANT_DECL(fft_decode_gd_b8)

// group is 32 or D (one scale per vector); bits is 4 or 8.
cudaError_t fft_encode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream)
{
    const bool per_vector = group == D;
    if (!per_vector && group != 32) return cudaErrorInvalidValue;
    if (bits == 4) return per_vector ? fft_encode_gd_b4(D, bf16, N, prm, stream) : fft_encode_g32_b4(D, bf16, N, prm, stream);
    if (bits == 8) return per_vector ? fft_encode_gd_b8(D, bf16, N, prm, stream) : fft_encode_g32_b8(D, bf16, N, prm, stream);
    return cudaErrorInvalidValue;
}

cudaError_t fft_decode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream)
{
    const bool per_vector = group == D;
    if (!per_vector && group != 32) return cudaErrorInvalidValue;
    if (bits == 4) return per_vector ? fft_decode_gd_b4(D, bf16, N, prm, stream) : fft_decode_g32_b4(D, bf16, N, prm, stream);
    if (bits == 8) return per_vector ? fft_decode_gd_b8(D, bf16, N, prm, stream) : fft_decode_g32_b8(D, bf16, N, prm, stream);
    return cudaErrorInvalidValue;
}

}  // namespace kvq
