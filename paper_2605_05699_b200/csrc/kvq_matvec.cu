// Small-call kernels of libkvq: kvq_append, the window flush and other calls of a few thousand vectors at most.
//
// On such calls nothing is bandwidth-bound: what counts is the latency of one launch.  The register-FFT kernels
// give a whole vector to one thread (thousands of dependent instructions), the tensor-core kernels pay a fixed
// set-up per launch (operand build, pipeline fill); both take 10 us and more for 64 vectors.  Here the transform
// is a plain fp32 matrix-vector product with the plan's D x D table (Sec. 3.1 Eq. 1-2 written as a matrix, signs
// and, if the plan has one, the rotation of Sec. 5.1 item 2 folded in), spread over a whole CTA:
//
//   * a CTA takes 8 vectors; its 8 warps split the contraction index (K) into 8 slices;
//   * a lane owns four consecutive output coordinates (eight for D > 128): table rows are read as coalesced
//     float4 (all rows of a slice in flight at once: about one L2 round trip per CTA), the vectors' entries come
//     from shared memory as broadcasts;
//   * partial sums meet in shared memory; warp w then finishes vector w: lambda, group maxima by shuffles, scale,
//     rounding and packing (encode) or the conversion to half precision (decode).
//
// Every (group, bits) layout, both dtypes, rotated plans and row maps are served; group and bits are run-time
// (warp-uniform) values.  Arithmetic of the quantizer follows the register-FFT kernels (same operations in the
// same order), so the two families agree wherever fp32 rounding of the transform does not decide a code.
#include "kvq_internal.h"
#include "kvq_device.cuh"

namespace kvq {

namespace {

constexpr int kWarps = 8;   // warps per CTA = slices of the contraction index
constexpr int kV = 8;       // vectors per CTA = one per warp in the finishing phase

struct MatvecParams {
    const void *in;        // encode: x [N, D] half precision
    const float *lambda;   // [n_lambda, D]
    void *packed;          // [*, D bits / 8]
    void *scales;          // [*, D / group] fp16
    void *out;             // decode: [*, D] half precision
    const float *table;    // encode: b0[n][c] (column c of the forward transform along a row); decode: e0[c][n]
    const float *table2;   // fused window flush: e0[c][n], for the way back
    int64_t N, n_lambda, rows_per_lambda;
    RowMap out_map, in_map;
    int group, bits;
    // Position on the device: when pos_dev is set, the base row of out_map is *pos_dev, read when the kernel runs, and must
    // lie in [0, pos_limit]; otherwise the launch writes nothing and raises KVQ_DEV_POSITION in *status.
    const int64_t *pos_dev;
    int64_t pos_limit;
    uint32_t *status;
};

// The row map of this launch's output rows: as passed, or based at the position found in device memory.  False (for the
// whole grid alike) when that position is outside the cache.
__device__ __forceinline__ bool resolve_out_map(const MatvecParams &prm, RowMap &map)
{
    map = prm.out_map;
    if (prm.pos_dev) {
        const int64_t p = __ldg(prm.pos_dev);
        if (p < 0 || p > prm.pos_limit) {
            if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(prm.status, KVQ_DEV_POSITION);
            return false;
        }
        map.base = p;
    }
    return true;
}

template <int D>
struct Geo {
    static constexpr int P = (D / 4 + 31) / 32;   // coordinate quads per lane
    static constexpr int KW = D / kWarps;         // contraction indices per warp
    // table rows a lane holds in flight per pass: the whole slice where registers allow (one L2 round trip per CTA)
    static constexpr int CH = P == 1 ? KW : (D == 160 ? 10 : 16);
    static_assert(D % (4 * kWarps) == 0 && KW % CH == 0, "slices must be whole quads and whole passes");
    static constexpr bool kLoops = CH == KW;      // the slice stays in registers: a CTA may take several batches of vectors
    static constexpr int kSmemBytes = (kV * D + kWarps * kV * D) * (int)sizeof(float);
};

__device__ __forceinline__ int64_t lambda_row(int64_t r, int64_t n_lambda, int64_t rows_per_lambda)
{
    return n_lambda == 1 ? 0 : r / rows_per_lambda;
}

// Rows k0 .. k0 + CH - 1 of this warp's slice of the table into registers (coalesced float4 per row).
template <int D>
__device__ __forceinline__ void load_rows(const float *__restrict__ table, int warp, int lane, int k0, float4 (&t)[Geo<D>::CH][Geo<D>::P])
{
    using Gm = Geo<D>;
#pragma unroll
    for (int k = 0; k < Gm::CH; ++k)
#pragma unroll
        for (int p = 0; p < Gm::P; ++p) {
            const int i = lane + 32 * p;
            t[k][p] = i < D / 4 ? __ldg(reinterpret_cast<const float4 *>(table + (size_t)(warp * Gm::KW + k0 + k) * D) + i)
                                : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
}

// y_v[c] = sum_k table[k][c] xs[v][k] for the CTA's kV vectors: this warp's K slice into registers (its first pass
// of table rows, t, was fetched by the caller while the vectors were being staged), partial sums through shared
// memory, and the sums of vector `warp` back into y[P][4] (coordinates 4 i .. 4 i + 3, i = lane + 32 p).
template <int D>
__device__ __forceinline__ void matvec(const float *__restrict__ table, float4 (&t)[Geo<D>::CH][Geo<D>::P], const float *xs, float *red,
                                       int warp, int lane, float (&y)[Geo<D>::P][4])
{
    using Gm = Geo<D>;
    constexpr int P = Gm::P, KW = Gm::KW, CH = Gm::CH;
    float acc[kV][P][4];
#pragma unroll
    for (int v = 0; v < kV; ++v)
#pragma unroll
        for (int p = 0; p < P; ++p)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[v][p][e] = 0.0f;

#pragma unroll 1
    for (int k0 = 0; k0 < KW; k0 += CH) {
        if (k0 > 0) load_rows<D>(table, warp, lane, k0, t);
#pragma unroll
        for (int v = 0; v < kV; ++v) {
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                const float xk = xs[v * D + warp * KW + k0 + k];   // broadcast
#pragma unroll
                for (int p = 0; p < P; ++p) {
                    acc[v][p][0] = fmaf(t[k][p].x, xk, acc[v][p][0]);
                    acc[v][p][1] = fmaf(t[k][p].y, xk, acc[v][p][1]);
                    acc[v][p][2] = fmaf(t[k][p].z, xk, acc[v][p][2]);
                    acc[v][p][3] = fmaf(t[k][p].w, xk, acc[v][p][3]);
                }
            }
        }
    }
#pragma unroll
    for (int v = 0; v < kV; ++v)
#pragma unroll
        for (int p = 0; p < P; ++p) {
            const int i = lane + 32 * p;
            if (i < D / 4)
                *reinterpret_cast<float4 *>(red + (size_t)(warp * kV + v) * D + 4 * i) =
                    make_float4(acc[v][p][0], acc[v][p][1], acc[v][p][2], acc[v][p][3]);
        }
    __syncthreads();
#pragma unroll
    for (int p = 0; p < P; ++p) {
        const int i = lane + 32 * p;
        float4 s = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (i < D / 4) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float4 a = *reinterpret_cast<const float4 *>(red + (size_t)(w * kV + warp) * D + 4 * i);
                s.x += a.x, s.y += a.y, s.z += a.z, s.w += a.w;
            }
        }
        y[p][0] = s.x, y[p][1] = s.y, y[p][2] = s.z, y[p][3] = s.w;
    }
}

// ------------------------------------------------------------------------------------------------
// encode: x -> codes and scales  (Sec. 3.2 steps 1-4, lambda and group scales of Sec. 7.1)
// ------------------------------------------------------------------------------------------------
// FLUSH: the window flush in one launch (Sec. 7.2).  After the codes of a vector are stored, the warp that finished it puts
// q sigma / max(lambda, 1e-6) -- what kvq_decode would rebuild from the stored bytes -- back into shared memory, and the
// CTA runs the matrix-vector product once more with the inverse table: rows out_map(r) of prm.out get the dequantized
// vectors.
// One batch of kV vectors.  t: the first pass of this warp's table rows, requested by the caller.
template <int D, bool BF16, bool FLUSH>
__device__ __forceinline__ void encode_batch(const MatvecParams &prm, const RowMap &out_map, float4 (&t)[Geo<D>::CH][Geo<D>::P], float *xs,
                                             float *red, int warp, int lane, int64_t batch)
{
    using Gm = Geo<D>;
    constexpr int P = Gm::P;
    const int64_t v0 = batch * kV;
    const int64_t r = v0 + warp;   // the vector this warp finishes
    float4 lam4[P];
#pragma unroll
    for (int p = 0; p < P; ++p) {
        const int i = lane + 32 * p;
        lam4[p] = (r < prm.N && i < D / 4)
                      ? __ldg(reinterpret_cast<const float4 *>(prm.lambda + lambda_row(r, prm.n_lambda, prm.rows_per_lambda) * D) + i)
                      : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }

    // ---- the CTA's vectors, widened to fp32 (rows past the end are zeros)
    const uint32_t *x = static_cast<const uint32_t *>(prm.in);
    for (int idx = threadIdx.x; idx < kV * (D / 2); idx += kWarps * 32) {
        const int v = idx / (D / 2), j = idx % (D / 2);
        const int64_t r = v0 + v;
        const float2 f = widen2<BF16>(r < prm.N ? __ldg(x + r * (D / 2) + j) : 0u);
        xs[v * D + 2 * j] = f.x, xs[v * D + 2 * j + 1] = f.y;
    }
    __syncthreads();

    float z[P][4];
    matvec<D>(prm.table, t, xs, red, warp, lane, z);

    // ---- warp w finishes vector w
    const bool live = r < prm.N;
    if (!FLUSH && !live) return;   // only in a CTA's last batch, and no barrier follows
    const int64_t orow = live ? out_map(r) : 0;
    const bool per_vector = prm.group == D;
    const float Q = prm.bits == 4 ? 7.0f : 127.0f;
    float amax[P];
#pragma unroll
    for (int p = 0; p < P; ++p) {
        const int i = lane + 32 * p;
        amax[p] = 0.0f;
        if (i < D / 4) {
            const float4 l = lam4[p];
            z[p][0] *= l.x, z[p][1] *= l.y, z[p][2] *= l.z, z[p][3] *= l.w;
            amax[p] = fmaxf(fmaxf(fabsf(z[p][0]), fabsf(z[p][1])), fmaxf(fabsf(z[p][2]), fabsf(z[p][3])));
        }
    }
    // group maxima: a group of 32 coordinates is 8 neighbouring lanes of one p; one group over the vector is everything
    if (per_vector) {
        float m = amax[0];
#pragma unroll
        for (int p = 1; p < P; ++p) m = fmaxf(m, amax[p]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
#pragma unroll
        for (int p = 0; p < P; ++p) amax[p] = m;
    } else {
#pragma unroll
        for (int p = 0; p < P; ++p)
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) amax[p] = fmaxf(amax[p], __shfl_xor_sync(0xFFFFFFFFu, amax[p], o));
    }
    uint16_t *scl = static_cast<uint16_t *>(prm.scales);
    unsigned char *pk = static_cast<unsigned char *>(prm.packed);
#pragma unroll
    for (int p = 0; p < P; ++p) {
        const int i = lane + 32 * p;
        // sigma = fp16(absmax / Q); codes are taken against the stored value
        const float sig = fminf(__fdiv_rn(amax[p], Q), 65504.0f);
        const __half hs = __float2half_rn(sig);
        const float sg = __half2float(hs);
        const float rs = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
        const bool clamp = !(amax[p] * rs < Q + 0.25f);   // saturated or subnormal scale: codes could leave [-Q, Q]
        if (i >= D / 4) continue;
        if (live && (per_vector ? (lane == 0 && p == 0) : ((i & 7) == 0)))
            scl[orow * (D / prm.group) + (per_vector ? 0 : i >> 3)] = __half_as_ushort(hs);
        uint32_t code[4];
        float qf[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float t = clamp ? fminf(fmaxf(z[p][e] * rs, -Q), Q) + 12582912.0f : fmaf(z[p][e], rs, 12582912.0f);
            code[e] = __float_as_uint(t);   // low bits: q in two's complement (1.5 * 2^23 + q)
            qf[e] = t - 12582912.0f;        // q itself, exactly
        }
        if (live) {
            if (prm.bits == 4) {
                const uint32_t w = (code[0] & 0xFu) | ((code[1] & 0xFu) << 4) | ((code[2] & 0xFu) << 8) | ((code[3] & 0xFu) << 12);
                *reinterpret_cast<uint16_t *>(pk + orow * (D / 2) + 2 * i) = (uint16_t)w;
            } else {
                const uint32_t w = (code[0] & 0xFFu) | ((code[1] & 0xFFu) << 8) | ((code[2] & 0xFFu) << 16) | (code[3] << 24);
                *reinterpret_cast<uint32_t *>(pk + orow * D + 4 * i) = w;
            }
        }
        if constexpr (FLUSH) {   // the way back starts from the stored values: q times the STORED scale over the clamped lambda
            const float4 l = lam4[p];
            const float4 o = make_float4(qf[0] * (sg * __frcp_rn(fmaxf(l.x, 1e-6f))), qf[1] * (sg * __frcp_rn(fmaxf(l.y, 1e-6f))),
                                         qf[2] * (sg * __frcp_rn(fmaxf(l.z, 1e-6f))), qf[3] * (sg * __frcp_rn(fmaxf(l.w, 1e-6f))));
            *reinterpret_cast<float4 *>(xs + warp * D + 4 * i) = live ? o : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
    }
    if constexpr (FLUSH) {
        float4 t2[Gm::CH][P];
        load_rows<D>(prm.table2, warp, lane, 0, t2);   // in flight across the barrier
        __syncthreads();                               // every warp's vector is back in shared memory; red is free again
        float y[P][4];
        matvec<D>(prm.table2, t2, xs, red, warp, lane, y);
        if (!live) return;
        unsigned char *out = static_cast<unsigned char *>(prm.out) + orow * (2 * D);
#pragma unroll
        for (int p = 0; p < P; ++p) {
            const int i = lane + 32 * p;
            if (i < D / 4)
                *reinterpret_cast<uint2 *>(out + 8 * i) = make_uint2(narrow2<BF16>(y[p][0], y[p][1]), narrow2<BF16>(y[p][2], y[p][3]));
        }
    }
}

// Where a warp's whole table slice fits its registers (D <= 128), a CTA takes batches blockIdx.x, blockIdx.x + gridDim.x,
// ... and the launch is one resident wave: on calls of more batches than the device holds CTAs the table crosses L2 once
// per CTA, not once per batch.  The barriers inside one batch also order the next batch's writes to xs and red after this
// batch's reads.  For D > 128 a CTA takes one batch.
template <int D, bool BF16, bool FLUSH>
__global__ void __launch_bounds__(kWarps * 32) kvq_encode_matvec_kernel(const __grid_constant__ MatvecParams prm)
{
    using Gm = Geo<D>;
    extern __shared__ __align__(16) float sm[];
    float *xs = sm, *red = sm + kV * D;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- everything that does not depend on the vectors is requested first, so that one round trip covers it all
    float4 t[Gm::CH][Gm::P];
    load_rows<D>(prm.table, warp, lane, 0, t);
    RowMap out_map;
    if (!resolve_out_map(prm, out_map)) return;   // uniform over the grid: no barrier is left waiting
    if constexpr (Gm::kLoops) {
        const int64_t n_batches = (prm.N + kV - 1) / kV;
#pragma unroll 1
        for (int64_t batch = blockIdx.x; batch < n_batches; batch += gridDim.x)
            encode_batch<D, BF16, FLUSH>(prm, out_map, t, xs, red, warp, lane, batch);
    } else {
        encode_batch<D, BF16, FLUSH>(prm, out_map, t, xs, red, warp, lane, blockIdx.x);
    }
}

// ------------------------------------------------------------------------------------------------
// decode: codes and scales -> x^  (Sec. 3.1: Eq. 2 undone, inverse real DFT, signs last; 1 / max(lambda, 1e-6) of Sec. 5.1)
// ------------------------------------------------------------------------------------------------
template <int D, bool BF16>
__device__ __forceinline__ void decode_batch(const MatvecParams &prm, float4 (&t)[Geo<D>::CH][Geo<D>::P], float *zs, float *red, int warp,
                                             int lane, int64_t batch)
{
    using Gm = Geo<D>;
    constexpr int P = Gm::P;
    const int64_t v0 = batch * kV;

    // ---- the CTA's stored vectors, dequantised: q sigma / max(lambda, 1e-6), four coordinates per thread and pass
    const unsigned char *pk = static_cast<const unsigned char *>(prm.packed);
    const uint16_t *scl = static_cast<const uint16_t *>(prm.scales);
    const int G = D / prm.group;
    for (int idx = threadIdx.x; idx < kV * (D / 4); idx += kWarps * 32) {
        const int v = idx / (D / 4), i = idx % (D / 4);
        const int64_t r = v0 + v;
        float4 o = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (r < prm.N) {
            const int64_t irow = prm.in_map(r);
            int q[4];
            if (prm.bits == 4) {
                const uint32_t w = __ldg(reinterpret_cast<const uint16_t *>(pk + irow * (D / 2) + 2 * i));
#pragma unroll
                for (int e = 0; e < 4; ++e) q[e] = (int)(((w >> (4 * e)) & 0xFu) ^ 8u) - 8;
            } else {
                const uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(pk + irow * D + 4 * i));
#pragma unroll
                for (int e = 0; e < 4; ++e) q[e] = (int)(signed char)((w >> (8 * e)) & 0xFFu);
            }
            const float sig = __half2float(__ushort_as_half(__ldg(scl + irow * G + (4 * i) / prm.group)));
            const float4 l = __ldg(reinterpret_cast<const float4 *>(prm.lambda + lambda_row(r, prm.n_lambda, prm.rows_per_lambda) * D) + i);
            o.x = (float)q[0] * (sig * __frcp_rn(fmaxf(l.x, 1e-6f)));
            o.y = (float)q[1] * (sig * __frcp_rn(fmaxf(l.y, 1e-6f)));
            o.z = (float)q[2] * (sig * __frcp_rn(fmaxf(l.z, 1e-6f)));
            o.w = (float)q[3] * (sig * __frcp_rn(fmaxf(l.w, 1e-6f)));
        }
        *reinterpret_cast<float4 *>(zs + v * D + 4 * i) = o;
    }
    __syncthreads();

    float y[P][4];
    matvec<D>(prm.table, t, zs, red, warp, lane, y);

    const int64_t r = v0 + warp;
    if (r >= prm.N) return;
    unsigned char *out = static_cast<unsigned char *>(prm.out) + prm.out_map(r) * (2 * D);
#pragma unroll
    for (int p = 0; p < P; ++p) {
        const int i = lane + 32 * p;
        if (i < D / 4)
            *reinterpret_cast<uint2 *>(out + 8 * i) = make_uint2(narrow2<BF16>(y[p][0], y[p][1]), narrow2<BF16>(y[p][2], y[p][3]));
    }
}

template <int D, bool BF16>
__global__ void __launch_bounds__(kWarps * 32) kvq_decode_matvec_kernel(const __grid_constant__ MatvecParams prm)
{
    using Gm = Geo<D>;
    extern __shared__ __align__(16) float sm[];
    float *zs = sm, *red = sm + kV * D;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float4 t[Gm::CH][Gm::P];
    load_rows<D>(prm.table, warp, lane, 0, t);   // in flight while the codes are fetched and dequantised
    if constexpr (Gm::kLoops) {   // as in the encode kernel
        const int64_t n_batches = (prm.N + kV - 1) / kV;
#pragma unroll 1
        for (int64_t batch = blockIdx.x; batch < n_batches; batch += gridDim.x) decode_batch<D, BF16>(prm, t, zs, red, warp, lane, batch);
    } else {
        decode_batch<D, BF16>(prm, t, zs, red, warp, lane, blockIdx.x);
    }
}

// MODE: 0 decode, 1 encode, 2 encode + decode of the same rows (window flush)
template <int D, bool BF16, int MODE>
cudaError_t launch(const MatvecParams &prm, cudaStream_t stream)
{
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    auto kern = MODE == 0 ? kvq_decode_matvec_kernel<D, BF16> : MODE == 1 ? kvq_encode_matvec_kernel<D, BF16, false> : kvq_encode_matvec_kernel<D, BF16, true>;
    if (slots.sms[dev] == 0) {   // slots.sms: the CTAs of this kernel that the device holds at once
        int sms = 0, per_sm = 0;
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<D>::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kWarps * 32, Geo<D>::kSmemBytes)) != cudaSuccess) return e;
        slots.sms[dev] = sms * (per_sm > 0 ? per_sm : 1);
    }
    if (prm.N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    const int64_t batches = (prm.N + kV - 1) / kV;
    if (batches > 0x7FFFFFFF) return cudaErrorInvalidValue;
    // one resident wave of CTAs that loop over batches where the kernel does; else a CTA per batch
    const int ctas = (int)(Geo<D>::kLoops && batches > slots.sms[dev] ? slots.sms[dev] : batches);
    kern<<<ctas, kWarps * 32, Geo<D>::kSmemBytes, stream>>>(prm);
    count_launch();
    return cudaGetLastError();
}

template <int MODE>
cudaError_t dispatch(int D, bool bf16, const MatvecParams &prm, cudaStream_t stream)
{
    switch (D) {
        case 64: return bf16 ? launch<64, true, MODE>(prm, stream) : launch<64, false, MODE>(prm, stream);
        case 96: return bf16 ? launch<96, true, MODE>(prm, stream) : launch<96, false, MODE>(prm, stream);
        case 128: return bf16 ? launch<128, true, MODE>(prm, stream) : launch<128, false, MODE>(prm, stream);
        case 160: return bf16 ? launch<160, true, MODE>(prm, stream) : launch<160, false, MODE>(prm, stream);
        case 256: return bf16 ? launch<256, true, MODE>(prm, stream) : launch<256, false, MODE>(prm, stream);
    }
    return cudaErrorInvalidValue;
}

MatvecParams from_fft(const FftParams &f, const float *table, int group, int bits)
{
    MatvecParams p;
    p.in = f.in, p.lambda = f.lambda, p.packed = f.packed, p.scales = f.scales, p.out = f.out;
    p.table = table;
    p.table2 = nullptr;
    p.N = f.N, p.n_lambda = f.n_lambda, p.rows_per_lambda = f.rows_per_lambda;
    p.out_map = f.out_map, p.in_map = f.in_map;
    p.group = group, p.bits = bits;
    p.pos_dev = nullptr, p.pos_limit = 0, p.status = f.status;
    return p;
}

}  // namespace

// b0: the plan's [n][c] table; e0: its transpose
cudaError_t matvec_encode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &f, const float *b0, cudaStream_t stream,
                          const DevicePos *pos)
{
    (void)N;
    MatvecParams p = from_fft(f, b0, group, bits);
    if (pos) p.pos_dev = pos->ptr, p.pos_limit = pos->limit;
    return dispatch<1>(D, bf16, p, stream);
}

cudaError_t matvec_decode(int D, int group, int bits, bool bf16, int64_t N, const FftParams &f, const float *e0, cudaStream_t stream)
{
    (void)N;
    return dispatch<0>(D, bf16, from_fft(f, e0, group, bits), stream);
}

// The window flush in one launch: x rows -> codes and scales at rows out_map(r) of the caches, and the dequantized
// vectors at the same rows of f.out.
cudaError_t matvec_flush(int D, int group, int bits, bool bf16, int64_t N, const FftParams &f, const float *b0, const float *e0,
                         cudaStream_t stream, const DevicePos *pos)
{
    (void)N;
    MatvecParams p = from_fft(f, b0, group, bits);
    if (pos) p.pos_dev = pos->ptr, p.pos_limit = pos->limit;
    p.table2 = e0;
    return dispatch<2>(D, bf16, p, stream);
}

}  // namespace kvq
