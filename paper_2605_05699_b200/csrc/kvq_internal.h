// Declarations shared by the translation units of libkvq (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/kvq.h"

namespace kvq {

// Where row r of a contiguous block of rows lives in a cache laid out [stream][T][...]: every `rps` consecutive rows of
// the block belong to one stream and go to rows base .. base + rps - 1 of it; `stride` = rows per stream of the cache.
// The identity is {1, 1, 0}; kvq_append is {1, T_max, pos}.
struct RowMap {
    int64_t rps, stride, base;
    __host__ __device__ __forceinline__ int64_t operator()(int64_t r) const
    {
        return rps == 1 ? r * stride + base : (r / rps) * stride + base + (r % rps);
    }
};

// Arguments of the register-FFT kernels.  Passed by value as a __grid_constant__
// parameter, so the sign words are read straight from the constant bank.
struct FftParams {
    const void *in;        // encode: x [N, D] half precision
    const float *lambda;   // [n_lambda, D] fp32
    void *packed;          // [*, D bits / 8] bytes (encode: out, decode: in)
    void *scales;          // [*, D/group] fp16 (encode: out, decode: in)
    void *out;             // decode: x^ [N, D] half precision
    int64_t N;
    int64_t n_lambda, rows_per_lambda;
    int per_vector;        // one scale per vector (group = D) instead of one per 32 channels
    RowMap out_map;             // row of packed / scales (encode) or of out (decode) that row r goes to
    RowMap in_map;              // decode: row of packed / scales that row r comes from
    uint32_t *status;           // per-plan device status word
    float table_max;            // tensor-core encode: largest |entry| of the plan's forward table (sqrt(2/D) without a rotation)
    uint32_t first_wait_polls;  // tensor-core encode, D <= 160: polls the mma role gives its first operand build (0: the default)
    int bits;                   // tensor-core encode: 4 or 8 (the register-FFT launchers take it as an argument)
    uint32_t sign_xor[128];     // word m: bit 15 set if s_{2m} = -1, bit 31 set if s_{2m+1} = -1
};

// A decode whose rows live in a cache laid out [stream][T][...]: the call's N = S * rows logical rows are rows
// [base, base + rows) of each of S streams, `stride` cache rows apart, in packed, scales and out alike; the lambda row of
// stream s is s / streams_per_lambda.  rows == 0: the flat layout, row r at row r.
struct CacheView {
    int64_t rows, stride, base, streams_per_lambda;
};

// Arguments of the tcgen05 DFT-as-GEMM decode kernel (kvq_umma_decode.cu).
struct GemmParams {
    const void *packed;    // [N, D/2] bytes
    const void *scales;    // [N, D/32] fp16, or [N, 1] when per_vector
    const float *lambda;   // [n_lambda, D] fp32
    void *out;             // [N, D] fp16
    const float *b0;       // plan table [D, D] fp32: b0[n][c] = s_n M[c][n], M the real orthogonal DFT matrix of Eq. 1-2
    int64_t N;
    int64_t n_lambda, rows_per_lambda;
    int per_vector;        // one scale per vector (group = D) instead of one per 32 channels
    uint32_t *status;
    CacheView view = {0, 0, 0, 1};   // where the rows live (the block flush decodes a window of every stream's cache)
    // row of packed / scales / out that holds row `off` of segment `seg` (flat: segments of rows_per_segment rows back to back)
    __host__ __device__ __forceinline__ int64_t phys_row(int64_t seg, int64_t off, int64_t rows_per_segment) const
    {
        return view.rows ? seg * view.stride + view.base + off : seg * rows_per_segment + off;
    }
    __host__ __device__ __forceinline__ int64_t lambda_index(int64_t seg) const
    {
        return n_lambda == 1 ? 0 : view.rows ? seg / view.streams_per_lambda : seg;
    }
};

// tcgen05 DFT-as-GEMM kernels (kvq_umma_decode.cu, kvq_umma_encode.cu): which (D, 16-bit type) pairs are built, and the
// launchers.  Encode takes the register-FFT argument block (its sign words are unused) and the plan table e0 [D, D]
// fp32, e0[c][n] = M[c][n] s_n; decode takes the table b0 = e0 transposed through GemmParams.
bool umma_decode_supported(int D, bool bf16);
bool umma_encode_supported(int D, bool bf16);
bool umma_calibrate_supported(int D, bool bf16);
bool umma_decode_bits8_supported(int D, bool bf16);
cudaError_t umma_decode(int D, bool bf16, int bits, int64_t N, const GemmParams &prm, const uint32_t *sign_xor /* host, 128 words */,
                        cudaStream_t stream, bool radix2 = false /* the plan has no rotation: the D = 128 fp16 kernel may split by parity */);
cudaError_t umma_calibrate(int D, bool bf16, int64_t N, const FftParams &prm, const float *e0, uint32_t *amax_bits, cudaStream_t stream);
cudaError_t umma_calibrate_d256(bool bf16, int64_t N, const FftParams &prm, const float *e0, uint32_t *amax_bits, cudaStream_t stream);
cudaError_t umma_encode_d256(bool bf16, bool per_vector, int64_t N, const FftParams &prm, const float *e0, cudaStream_t stream);   // kvq_umma_encode256.cu
cudaError_t umma_decode_d256(bool bf16, int bits, int64_t N, const GemmParams &prm, const uint32_t *sign_xor, cudaStream_t stream);   // kvq_umma_decode256.cu
cudaError_t umma_decode_d256_dense(bool bf16, int64_t N, const GemmParams &prm, cudaStream_t stream);   // kvq_umma_decode256_dense.cu: any table
bool umma_encode_per_vector_supported(int D, bool bf16);
bool umma_encode_bits8_supported(int D, bool bf16);
cudaError_t umma_encode(int D, bool bf16, bool per_vector, int64_t N, const FftParams &prm, const float *e0, cudaStream_t stream);

// fp32 matrix-vector kernels for small calls (kvq_matvec.cu): every layout, dtype and D; b0 / e0 are the plan's tables
// A cache position that lives in device memory (read when the kernel runs): the base row of the output row map; it must
// lie in [0, limit], else the launch writes nothing and raises KVQ_DEV_POSITION in the plan's status word.
struct DevicePos {
    const int64_t *ptr;
    int64_t limit;
};
cudaError_t matvec_encode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, const float *b0, cudaStream_t stream,
                          const DevicePos *pos = nullptr);
cudaError_t matvec_decode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, const float *e0, cudaStream_t stream);
cudaError_t matvec_flush(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, const float *b0, const float *e0,
                         cudaStream_t stream, const DevicePos *pos = nullptr);   // encode + decode of the same rows in one launch
// group: 32 or D (one scale per vector); bits: 4 or 8
cudaError_t fft_encode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream);
cudaError_t fft_decode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream);


// A kernel's opt-in shared-memory size is a per-device function attribute, and SM counts differ between devices: the
// launchers keep what they looked up in one slot per device ordinal.  Racing first calls write the same values.
constexpr int kMaxDevices = 64;
struct DeviceSlots {
    int sms[kMaxDevices] = {};
    int blocks_per_sm[kMaxDevices] = {};
};
inline cudaError_t current_device_slot(int *dev)
{
    cudaError_t e = cudaGetDevice(dev);
    if (e != cudaSuccess) return e;
    return (*dev < 0 || *dev >= kMaxDevices) ? cudaErrorInvalidDevice : cudaSuccess;
}

void count_launch();

}  // namespace kvq

// The plan behind the opaque kvq_plan_t handle.
struct kvq_plan {
    int D, group;
    int bits;              // 4 (nibble pairs) or 8 (one byte per code)
    uint64_t seed;
    int8_t signs[256];
    uint32_t sign_xor[128];
    kvq_impl_t enc_impl, dec_impl;
    // device state, created on first use
    std::mutex mu;
    int device;            // -1 until initialised
    uint32_t *d_status;    // device status word
    float *d_b0;           // [D, D] fp32 inverse-transform matrix with the signs folded in (GEMM decode), or null
    float *d_e0;           // [D, D] fp32 forward-transform matrix with the signs folded in (GEMM encode), or null
    size_t table_bytes;
    double *rot;           // host, [D, D] row-major: the rotation between the transform and lambda, or null
    float table_max;       // largest |entry| of the forward table
    uint32_t first_wait_polls;   // see kvq_plan_set_wait_limit; 0 = default
};
