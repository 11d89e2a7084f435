// Whole-CTA fp32 decode of a run of rows on the CUDA cores: what the tensor-core decode kernels fall back to for a
// lambda row whose reciprocals span more than 2^8.  Their B operand carries M / max(lambda, 1e-6) in fp16, all
// channels side by side, and loses the small channels' bits on such a row; the inverse of Sec. 5.1 item 1 is defined
// for every lambda > 0 (with its 1e-6 clamp), so those rows are redone here from the codes: u_c = q_c sigma / max(lambda_c,
// 1e-6) in fp32, x_n = sum_c b0[n][c] u_c in fp32 (Sec. 3.2: dequantise, undo Eq. 2, inverse transform, sign), rounded once
// to the output type.  About a hundred times slower per row than the tensor-core path: a safety net for degenerate lambda
// rows, not a code path a calibrated lambda meets.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdint>

#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

// Is the lambda row too wide for the fp16 B operand?  The B builders' own test (RecipLambda), by one warp.
template <int D>
__device__ __forceinline__ bool lambda_row_is_wide(const float *__restrict__ lam, int lane, float *rho_out = nullptr)
{
    const RecipLambda<D> rl(lam, lane);
    if (rho_out) *rho_out = rl.rho;   // what the B builders divide the reciprocals by
    return rl.wide;
}

// Output channels [n0, n0 + NCOLS) of rows [row0, row0 + rows) of the call, all of one lambda row `lam`.  Every thread of
// the CTA calls it with the same arguments; `su` is shared-memory scratch of 32 * D floats.  A thread owns one output
// channel n and eight rows at a time; the table row b0[n][.] streams from L2.
template <int D, bool BF16OUT, int BITS, int NCOLS>
__device__ __noinline__ void decode_rows_fp32(const GemmParams &g, const float *__restrict__ lam, int64_t row0 /* in memory */, int rows, int n0, float *su)
{
    constexpr int G = D / 32, kPerThread = 8;
    const int T = (int)blockDim.x, tid = (int)threadIdx.x;
    const int groups = T / NCOLS < 4 ? T / NCOLS : 4;
    const int R = groups * kPerThread;   // rows per pass (<= 32)
    const unsigned char *packed = static_cast<const unsigned char *>(g.packed);
    const uint16_t *scales = static_cast<const uint16_t *>(g.scales);
    for (int base = 0; base < rows; base += R) {
        const int nr = rows - base < R ? rows - base : R;
        __syncthreads();   // the previous pass has read su
        for (int i = tid; i < R * D; i += T) {
            const int r = i / D, c = i - r * D;
            float u = 0.0f;
            if (r < nr) {
                const int64_t row = row0 + base + r;
                int q;
                if constexpr (BITS == 4) {
                    const uint32_t byte = packed[row * (D / 2) + (c >> 1)];
                    const uint32_t nib = (c & 1) ? byte >> 4 : byte & 15u;
                    q = (int)(nib ^ 8u) - 8;   // two's-complement nibble
                } else {
                    q = (int)static_cast<signed char>(packed[row * D + c]);
                }
                const float sig = __half2float(__ushort_as_half(scales[g.per_vector ? row : row * G + (c >> 5)]));
                u = __fdiv_rn((float)q * sig, fmaxf(__ldg(lam + c), 1e-6f));
            }
            su[i] = u;
        }
        __syncthreads();
        if (tid < groups * NCOLS) {
            const int gr = tid / NCOLS, n = n0 + tid - gr * NCOLS;
            float acc[kPerThread];
#pragma unroll
            for (int k = 0; k < kPerThread; ++k) acc[k] = 0.0f;
            const float4 *brow = reinterpret_cast<const float4 *>(g.b0 + (size_t)n * D);
            const float *ur = su + gr * kPerThread * D;
            for (int c4 = 0; c4 < D / 4; ++c4) {
                const float4 b = __ldg(brow + c4);
#pragma unroll
                for (int k = 0; k < kPerThread; ++k) {
                    const float4 u = *reinterpret_cast<const float4 *>(ur + k * D + 4 * c4);
                    acc[k] = fmaf(u.w, b.w, fmaf(u.z, b.z, fmaf(u.y, b.y, fmaf(u.x, b.x, acc[k]))));
                }
            }
#pragma unroll
            for (int k = 0; k < kPerThread; ++k) {
                const int r = gr * kPerThread + k;
                if (r < nr) {
                    const int64_t at = (row0 + base + r) * D + n;
                    if constexpr (BF16OUT) static_cast<__nv_bfloat16 *>(g.out)[at] = __float2bfloat16_rn(acc[k]);
                    else static_cast<__half *>(g.out)[at] = __float2half_rn(acc[k]);
                }
            }
        }
    }
    __syncthreads();
}

// The tail of a tensor-core decode kernel: the CTA's tiles [tile_begin, tile_begin + n_my) once more, and those the fp16
// operands could not carry decoded again in fp32 over what the pipeline stored for them: tiles of a wide lambda row and,
// for a kernel without a per-row rescue of its A operand (CHECK_SCALES), tiles with a stored scale that leaves q sigma rho's
// fp16 range (the kernel's own test, applied to the tile's scales again).  Called by every thread, after the pipeline's
// stores are complete (each storing thread has waited for its bulk groups) and a CTA-wide barrier.  A CTA that computes
// NCOLS < D output channels (from n0 on) redoes those only: its partner's stores may still be on their way.
template <int D, bool BF16OUT, int BITS, int TILE, int NCOLS = D, bool CHECK_SCALES = false>
__device__ __forceinline__ void redo_tiles_fp32(const GemmParams &g, int64_t tile_begin, int n_my, int64_t tps, int64_t rpl, float *su, int n0 = 0)
{
    const int lane = (int)threadIdx.x & 31;
    int64_t seen = -1;
    bool wide = false;
    float rho = 1.0f;
    for (int j = 0; j < n_my; ++j) {
        const int64_t t = tile_begin + j, seg = t / tps, off = (t - seg * tps) * TILE;
        const float *lam = g.lambda + g.lambda_index(seg) * D;
        if (seg != seen) {
            seen = seg;
            wide = lambda_row_is_wide<D>(lam, lane, &rho);
        }
        const int64_t row0 = g.phys_row(seg, off, rpl);   // where the tile's first row lives
        int64_t rows = rpl - off < TILE ? rpl - off : TILE;
        if (seg * rpl + off + rows > g.N) rows = g.N - (seg * rpl + off);   // the call's last segment may be short
        if (rows <= 0) continue;
        bool redo = wide;
        if (CHECK_SCALES && !wide) {
            const uint16_t *sc = static_cast<const uint16_t *>(g.scales) + row0 * (g.per_vector ? 1 : D / 32);
            const int count = (int)rows * (g.per_vector ? 1 : D / 32);
            int bad = 0;
            for (int i = (int)threadIdx.x; i < count; i += (int)blockDim.x) {
                const float sr = __half2float(__ushort_as_half(sc[i])) * rho;
                bad |= sr != 0.0f && (sr > 9357.0f || sr < 6.1035156e-5f);
            }
            redo = __syncthreads_or(bad) != 0;
        }
        if (redo) decode_rows_fp32<D, BF16OUT, BITS, NCOLS>(g, lam, row0, (int)rows, n0, su);
    }
}

}  // namespace kvq
