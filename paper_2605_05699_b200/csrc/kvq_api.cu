// C ABI of libkvq (see include/kvq.h): plan object, host-side validation, dispatch.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/kvq.h"
#include "kvq_internal.h"

namespace kvq {

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

// SplitMix64 output function (Steele, Lea, Flood 2014); sign n uses the n-th output for `seed`.
static inline uint64_t splitmix64_at(uint64_t seed, uint64_t n)
{
    uint64_t z = seed + (n + 1) * 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

// AUTO sends kvq_encode / kvq_append calls of at least this many rows to the tensor-core kernel.
// calls up to this size are latency-bound: matrix-vector kernel (measured cross-over with the other two families)
static int64_t matvec_max_rows(int D) { return D <= 128 ? 2048 : 1024; }

static bool dim_supported(int D) { return D == 64 || D == 96 || D == 128 || D == 160 || D == 256; }

// Radices of the length-n complex FFT in the order the recursion splits them off (4 first,
// then 2, 3, 5), mirroring radix_of() on the device side.
static int radix_plan(int n, int *out)
{
    int k = 0;
    while (n > 1) {
        int r = n % 4 == 0 ? 4 : n % 2 == 0 ? 2 : n % 3 == 0 ? 3 : n % 5 == 0 ? 5 : n;
        out[k++] = r;
        n /= r;
    }
    return k;
}

}  // namespace kvq

// b0[n][c] = s_n M[c][n] with z = M (s (.) x) the transform of Eq. 1-2: row c of M is
//   D^-1/2                       (c = 0),        (-1)^n D^-1/2               (c = D/2),
//   sqrt(2/D) cos(2 pi c n / D)  (0 < c < D/2),  -sqrt(2/D) sin(2 pi k n / D) (c = D/2 + k, 0 < k < D/2).
// M is orthogonal, so the inverse transform is x^_n = s_n sum_c M[c][n] z^_c.
// With a rotation R (Sec. 5.1 item 2: v = lambda (.) R z, z^ = R^T (v^ / lambda)) the table becomes
// b0'[n][c'] = sum_c b0[n][c] R[c'][c]: the forward table is its transpose either way.  Sums in fp64.
// Returns the largest |entry|.
static double build_b0(const kvq_plan *p, float *b0)
{
    const int D = p->D, H = D / 2;
    const double pi = 3.14159265358979323846;
    std::vector<double> row((size_t)D);
    double tmax = 0.0;
    for (int n = 0; n < D; ++n) {
        for (int c = 0; c < D; ++c) {
            double m;
            if (c == 0) m = 1.0 / std::sqrt((double)D);
            else if (c == H) m = ((n & 1) ? -1.0 : 1.0) / std::sqrt((double)D);
            else if (c < H) m = std::sqrt(2.0 / D) * std::cos(2.0 * pi * (double)((long)c * n % D) / D);
            else m = -std::sqrt(2.0 / D) * std::sin(2.0 * pi * (double)((long)(c - H) * n % D) / D);
            row[(size_t)c] = p->signs[n] * m;
        }
        for (int c = 0; c < D; ++c) {
            double v = row[(size_t)c];
            if (p->rot) {
                v = 0.0;
                for (int k = 0; k < D; ++k) v += row[(size_t)k] * p->rot[(size_t)c * D + k];
            }
            b0[(size_t)n * D + c] = (float)v;
            tmax = std::fmax(tmax, std::fabs(v));
        }
    }
    return tmax;
}

// Host copies of both tables: b0 [n][c] for the decode kernels, its transpose e0 [c][n] for the encode kernels.
static bool make_tables(kvq_plan *p, std::vector<float> &b0, std::vector<float> &e0)
{
    const size_t D = (size_t)p->D;
    try {
        b0.resize(D * D);
        e0.resize(D * D);
    } catch (...) {
        return false;
    }
    p->table_max = (float)build_b0(p, b0.data());
    for (size_t n = 0; n < D; ++n)
        for (size_t c = 0; c < D; ++c) e0[c * D + n] = b0[n * D + c];
    return true;
}

using namespace kvq;

static kvq_status_t ensure_device(kvq_plan *p)
{
    std::lock_guard<std::mutex> lk(p->mu);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    if (p->device == dev) return KVQ_OK;
    if (p->device >= 0) return KVQ_ERR_INVALID_ARG;   // a plan stays on the device of its first use
    uint32_t *st = nullptr;
    if (cudaMalloc(&st, 256) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_NOMEM;
    }
    if (cudaMemset(st, 0, 256) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaFree(st);
        return KVQ_ERR_CUDA;
    }
    p->d_status = st;
    p->table_bytes = 256;
    if (umma_encode_supported(p->D, false) || umma_decode_supported(p->D, false)) {   // tables of the tensor-core kernels
        const size_t bytes = sizeof(float) * (size_t)p->D * p->D;
        std::vector<float> b0, e0;
        float *db = nullptr, *de = nullptr;
        bool ok = make_tables(p, b0, e0) && cudaMalloc(&db, bytes) == cudaSuccess && cudaMalloc(&de, bytes) == cudaSuccess;
        kvq_status_t why = KVQ_ERR_NOMEM;
        if (ok) {
            ok = cudaMemcpy(db, b0.data(), bytes, cudaMemcpyHostToDevice) == cudaSuccess &&
                 cudaMemcpy(de, e0.data(), bytes, cudaMemcpyHostToDevice) == cudaSuccess;
            why = KVQ_ERR_CUDA;
        }
        if (!ok) {
            (void)cudaGetLastError();
            if (db) cudaFree(db);
            if (de) cudaFree(de);
            cudaFree(st);
            p->d_status = nullptr;
            return why;
        }
        p->d_b0 = db;
        p->d_e0 = de;
        p->table_bytes += 2 * bytes;
    }
    p->device = dev;
    return KVQ_OK;
}

// the tensor-core kernels take groups of 32 (the fused layout) or one scale per vector; byte codes up to D = 160
static bool gemm_encode_ok(const kvq_plan *p, bool bf16)
{
    if (p->bits == 8) return umma_encode_bits8_supported(p->D, bf16);
    return p->group == p->D ? umma_encode_per_vector_supported(p->D, bf16) : umma_encode_supported(p->D, bf16);
}
static bool gemm_decode_ok(const kvq_plan *p, bool bf16)
{
    if (p->bits == 8 && p->D == 256 && p->rot) return false;   // the dense D = 256 kernel of rotated plans has no byte-code form
    return p->bits == 8 ? umma_decode_bits8_supported(p->D, bf16) : umma_decode_supported(p->D, bf16);
}

static bool misaligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

static kvq_status_t check_lambda(int64_t N, const float *lambda, int64_t n_lambda, int64_t rows_per_lambda)
{
    if (!lambda || n_lambda < 1) return KVQ_ERR_INVALID_ARG;
    if (n_lambda > 1) {
        if (rows_per_lambda < 1) return KVQ_ERR_INVALID_ARG;
        if ((N + rows_per_lambda - 1) / rows_per_lambda > n_lambda) return KVQ_ERR_INVALID_ARG;
    }
    if (misaligned16(lambda)) return KVQ_ERR_ALIGNMENT;
    return KVQ_OK;
}

static void fill_params(const kvq_plan *p, FftParams &prm, int64_t N, const float *lambda, int64_t n_lambda,
                        int64_t rows_per_lambda)
{
    std::memset(&prm, 0, sizeof(prm));
    prm.N = N;
    prm.lambda = lambda;
    prm.n_lambda = n_lambda;
    prm.rows_per_lambda = rows_per_lambda < 1 ? 1 : rows_per_lambda;
    prm.out_map = RowMap{1, 1, 0};
    prm.in_map = RowMap{1, 1, 0};
    prm.status = p->d_status;
    prm.table_max = p->table_max;
    prm.first_wait_polls = p->first_wait_polls;
    prm.bits = p->bits;
    std::memcpy(prm.sign_xor, p->sign_xor, sizeof(prm.sign_xor));
}

extern "C" {

kvq_status_t kvq_plan_create(int D, int group, uint64_t seed, kvq_plan_t **out)
{
    return kvq_plan_create_ex(D, group, 4, seed, out);
}

kvq_status_t kvq_plan_create_ex(int D, int group, int bits, uint64_t seed, kvq_plan_t **out)
{
    if (!out) return KVQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!dim_supported(D) || (group != 32 && group != D) || (bits != 4 && bits != 8)) return KVQ_ERR_UNSUPPORTED_DIM;
    kvq_plan *p = new (std::nothrow) kvq_plan();
    if (!p) return KVQ_ERR_NOMEM;
    p->D = D;
    p->group = group;
    p->bits = bits;
    p->seed = seed;
    p->enc_impl = p->dec_impl = KVQ_IMPL_AUTO;
    p->device = -1;
    p->d_status = nullptr;
    p->d_b0 = nullptr;
    p->d_e0 = nullptr;
    p->table_bytes = 0;
    p->rot = nullptr;
    p->table_max = (float)std::sqrt(2.0 / D);
    p->first_wait_polls = 0;
    std::memset(p->signs, 0, sizeof(p->signs));
    std::memset(p->sign_xor, 0, sizeof(p->sign_xor));
    for (int n = 0; n < D; ++n) {
        bool neg = (splitmix64_at(seed, (uint64_t)n) >> 63) != 0;
        p->signs[n] = neg ? -1 : 1;
        if (neg) p->sign_xor[n / 2] |= (n & 1) ? 0x80000000u : 0x00008000u;
    }
    *out = p;
    return KVQ_OK;
}

kvq_status_t kvq_plan_destroy(kvq_plan_t *plan)
{
    if (!plan) return KVQ_OK;
    if (plan->d_status) {
        if (cudaFree(plan->d_status) != cudaSuccess) (void)cudaGetLastError();
    }
    if (plan->d_b0) {
        if (cudaFree(plan->d_b0) != cudaSuccess) (void)cudaGetLastError();
    }
    if (plan->d_e0) {
        if (cudaFree(plan->d_e0) != cudaSuccess) (void)cudaGetLastError();
    }
    delete[] plan->rot;
    delete plan;
    return KVQ_OK;
}

kvq_status_t kvq_plan_set_rotation(kvq_plan_t *plan, const float *R_host)
{
    if (!plan) return KVQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(plan->mu);
    const size_t n = (size_t)plan->D * plan->D;
    double *rot = nullptr;
    if (R_host) {
        rot = new (std::nothrow) double[n];
        if (!rot) return KVQ_ERR_NOMEM;
        for (size_t i = 0; i < n; ++i) {
            if (!std::isfinite(R_host[i])) {
                delete[] rot;
                return KVQ_ERR_INVALID_ARG;
            }
            rot[i] = (double)R_host[i];
        }
    }
    delete[] plan->rot;
    plan->rot = rot;
    if (plan->device < 0 || !plan->d_b0) {   // tables are built on first use
        if (!rot) plan->table_max = (float)std::sqrt(2.0 / plan->D);
        return KVQ_OK;
    }
    // tables exist: rewrite them in place, on the plan's device, after everything queued there has finished
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess || cur != plan->device) {
        (void)cudaGetLastError();
        return KVQ_ERR_INVALID_ARG;
    }
    std::vector<float> b0, e0;
    if (!make_tables(plan, b0, e0)) return KVQ_ERR_NOMEM;
    const size_t bytes = sizeof(float) * n;
    if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(plan->d_b0, b0.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(plan->d_e0, e0.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}

kvq_status_t kvq_plan_get_signs(const kvq_plan_t *plan, int8_t *host_signs)
{
    if (!plan || !host_signs) return KVQ_ERR_INVALID_ARG;
    std::memcpy(host_signs, plan->signs, (size_t)plan->D);
    return KVQ_OK;
}

kvq_status_t kvq_plan_describe(const kvq_plan_t *plan, int *radices, int *n_radices, size_t *table_bytes)
{
    if (!plan) return KVQ_ERR_INVALID_ARG;
    int r[16];
    int n = radix_plan(plan->D / 2, r);
    if (radices)
        for (int i = 0; i < n && i < 8; ++i) radices[i] = r[i];
    if (n_radices) *n_radices = n;
    if (table_bytes) *table_bytes = plan->table_bytes;
    return KVQ_OK;
}

kvq_status_t kvq_plan_set_impl(kvq_plan_t *plan, kvq_impl_t encode_impl, kvq_impl_t decode_impl)
{
    if (!plan) return KVQ_ERR_INVALID_ARG;
    if ((int)encode_impl < 0 || (int)encode_impl > 3 || (int)decode_impl < 0 || (int)decode_impl > 3)
        return KVQ_ERR_INVALID_ARG;
    plan->enc_impl = encode_impl;
    plan->dec_impl = decode_impl;
    return KVQ_OK;
}

kvq_status_t kvq_plan_set_wait_limit(kvq_plan_t *plan, uint32_t polls)
{
    if (!plan) return KVQ_ERR_INVALID_ARG;
    plan->first_wait_polls = polls;
    return KVQ_OK;
}

// Device tables and launch attributes of every kernel a call with this plan and this 16-bit type can take: each
// launcher is entered with N = 0, sets its kernel's attributes for the current device and returns before its launch.
kvq_status_t kvq_plan_prepare(kvq_plan_t *plan, kvq_dtype_t dtype)
{
    if (!plan) return KVQ_ERR_INVALID_ARG;
    if (dtype != KVQ_F16 && dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
    kvq_status_t st = ensure_device(plan);
    if (st != KVQ_OK) return st;
    const bool bf16 = dtype == KVQ_BF16, per_vector = plan->group == plan->D;
    FftParams prm;
    fill_params(plan, prm, 0, nullptr, 1, 1);
    GemmParams g;
    std::memset(&g, 0, sizeof(g));
    g.n_lambda = g.rows_per_lambda = 1;
    g.per_vector = per_vector;
    g.status = plan->d_status;
    g.b0 = plan->d_b0;
    cudaError_t e = cudaSuccess;
    auto also = [&e](cudaError_t r) {
        if (e == cudaSuccess) e = r;
    };
    if (gemm_encode_ok(plan, bf16)) also(umma_encode(plan->D, bf16, per_vector, 0, prm, plan->d_e0, nullptr));
    if (gemm_decode_ok(plan, bf16))
        also(plan->rot && plan->D == 256 ? umma_decode_d256_dense(bf16, 0, g, nullptr)
                                         : umma_decode(plan->D, bf16, plan->bits, 0, g, plan->sign_xor, nullptr, !plan->rot));
    if (umma_calibrate_supported(plan->D, bf16)) also(umma_calibrate(plan->D, bf16, 0, prm, plan->d_e0, nullptr, nullptr));
    also(matvec_encode(plan->D, plan->group, plan->bits, bf16, 0, prm, plan->d_b0, nullptr));
    also(matvec_decode(plan->D, plan->group, plan->bits, bf16, 0, prm, plan->d_e0, nullptr));
    also(matvec_flush(plan->D, plan->group, plan->bits, bf16, 0, prm, plan->d_b0, plan->d_e0, nullptr));
    if (!plan->rot) {
        also(fft_encode(plan->D, plan->group, plan->bits, bf16, 0, prm, nullptr));
        also(fft_decode(plan->D, plan->group, plan->bits, bf16, 0, prm, nullptr));
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}

kvq_status_t kvq_plan_device_status(kvq_plan_t *plan, uint32_t *word)
{
    if (!plan || !word) return KVQ_ERR_INVALID_ARG;
    *word = 0;
    if (!plan->d_status) return KVQ_OK;   // never used on a device
    if (cudaDeviceSynchronize() != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    if (cudaMemcpy(word, plan->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    if (*word & 7u) return KVQ_ERR_TIMEOUT;
    if (*word & 16u) return KVQ_ERR_INVALID_ARG;   // a position read on the device was outside the cache
    return *word ? KVQ_ERR_RANGE : KVQ_OK;
}

kvq_status_t kvq_plan_clear_device_status(kvq_plan_t *plan)
{
    if (!plan) return KVQ_ERR_INVALID_ARG;
    if (!plan->d_status) return KVQ_OK;   // never used on a device
    if (cudaDeviceSynchronize() != cudaSuccess || cudaMemset(plan->d_status, 0, sizeof(uint32_t)) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}

// The decode half of a block flush: small blocks (the window flush) and rotated plans take the matrix-vector kernel,
// large plain blocks the register FFT.
static bool flush_decode_is_matvec(const kvq_plan_t *plan, int64_t N)
{
    return plan->rot || plan->dec_impl == KVQ_IMPL_MATVEC || (plan->dec_impl != KVQ_IMPL_FFT && N <= matvec_max_rows(plan->D));
}

// dq / fused: the window flush.  Where the call takes the matrix-vector kernel and the plan's decode side would take it
// too, the dequantized rows go to dq (rows out_map(r)) in the same launch and *fused is set.
static kvq_status_t encode_common(kvq_plan_t *plan, const void *x, kvq_dtype_t dtype, int64_t N, const float *lambda,
                                  int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed, void *scales,
                                  const RowMap &out_map, void *cuda_stream, void *dq = nullptr, bool *fused = nullptr,
                                  const DevicePos *pos = nullptr)
{
    if (!plan || N < 0) return KVQ_ERR_INVALID_ARG;
    if (dtype != KVQ_F16 && dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
    if (N == 0) return KVQ_OK;   // nothing to do; empty buffers may be null
    if (!x || !packed || !scales) return KVQ_ERR_INVALID_ARG;
    kvq_status_t st = check_lambda(N, lambda, n_lambda, rows_per_lambda);
    if (st != KVQ_OK) return st;
    if (misaligned16(x) || misaligned16(packed) || misaligned16(scales)) return KVQ_ERR_ALIGNMENT;
    const bool bf16 = dtype == KVQ_BF16;
    const bool per_vector = plan->group == plan->D;
    // tensor-map coordinates are 32-bit: the tensor-core kernels take up to 2^31 - 1 rows per call
    const bool gemm_ok = gemm_encode_ok(plan, bf16) && N < ((int64_t)1 << 31);
    if (!pos) {
        if (plan->enc_impl == KVQ_IMPL_GEMM && !gemm_ok) return KVQ_ERR_UNSUPPORTED_DIM;
        if (plan->rot && plan->enc_impl == KVQ_IMPL_FFT) return KVQ_ERR_UNSUPPORTED_DIM;   // the rotation lives in the D x D tables
    }
    if ((st = ensure_device(plan)) != KVQ_OK) return st;
    FftParams prm;
    fill_params(plan, prm, N, lambda, n_lambda, rows_per_lambda);
    prm.in = x;
    prm.packed = packed;
    prm.scales = scales;
    prm.out_map = out_map;
    // AUTO: the matrix-vector kernel for small calls (latency), beyond that the tensor-core kernel (measured faster than
    // the register FFT at every size above the matrix-vector limit), the register FFT where no tensor-core kernel is
    // built.  A rotated plan has no FFT path: matrix-vector wherever the tensor-core kernel does not apply.
    kvq_impl_t impl = pos ? KVQ_IMPL_MATVEC : plan->enc_impl;   // a position in device memory: the matrix-vector kernels read it
    if (impl == KVQ_IMPL_AUTO) {
        if (N <= matvec_max_rows(plan->D)) impl = KVQ_IMPL_MATVEC;
        else if (gemm_ok) impl = KVQ_IMPL_GEMM;
        else impl = plan->rot ? KVQ_IMPL_MATVEC : KVQ_IMPL_FFT;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (impl == KVQ_IMPL_GEMM) e = umma_encode(plan->D, bf16, per_vector, N, prm, plan->d_e0, stream);
    else if (impl == KVQ_IMPL_MATVEC && dq && fused && (pos || flush_decode_is_matvec(plan, N))) {
        prm.out = dq;
        e = matvec_flush(plan->D, plan->group, plan->bits, bf16, N, prm, plan->d_b0, plan->d_e0, stream, pos);
        *fused = e == cudaSuccess;
    } else if (impl == KVQ_IMPL_MATVEC) e = matvec_encode(plan->D, plan->group, plan->bits, bf16, N, prm, plan->d_b0, stream, pos);
    else e = fft_encode(plan->D, plan->group, plan->bits, bf16, N, prm, stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}

kvq_status_t kvq_encode(kvq_plan_t *plan, const void *x, kvq_dtype_t dtype, int64_t N, const float *lambda,
                        int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed, void *scales, void *cuda_stream)
{
    return encode_common(plan, x, dtype, N, lambda, n_lambda, rows_per_lambda, packed, scales, RowMap{1, 1, 0}, cuda_stream);
}

kvq_status_t kvq_append(kvq_plan_t *plan, const void *x_new, kvq_dtype_t dtype, int64_t S, const float *lambda,
                        int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache, void *scales_cache,
                        int64_t T_max, int64_t pos, void *cuda_stream)
{
    if (T_max < 1 || pos < 0 || pos >= T_max) return KVQ_ERR_INVALID_ARG;
    return encode_common(plan, x_new, dtype, S, lambda, n_lambda, streams_per_lambda, packed_cache, scales_cache,
                         RowMap{1, T_max, pos}, cuda_stream);
}

kvq_status_t kvq_decode(kvq_plan_t *plan, const uint8_t *packed, const void *scales, int64_t N, const float *lambda,
                        int64_t n_lambda, int64_t rows_per_lambda, void *out, kvq_dtype_t dtype, void *cuda_stream)
{
    if (!plan || N < 0) return KVQ_ERR_INVALID_ARG;
    if (dtype != KVQ_F16 && dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
    if (N == 0) return KVQ_OK;   // nothing to do; empty buffers may be null
    if (!packed || !scales || !out) return KVQ_ERR_INVALID_ARG;
    kvq_status_t st = check_lambda(N, lambda, n_lambda, rows_per_lambda);
    if (st != KVQ_OK) return st;
    if (misaligned16(packed) || misaligned16(scales) || misaligned16(out)) return KVQ_ERR_ALIGNMENT;
    const bool bf16 = dtype == KVQ_BF16;
    const bool gemm_ok = gemm_decode_ok(plan, bf16) && N < ((int64_t)1 << 31);
    if (plan->dec_impl == KVQ_IMPL_GEMM && !gemm_ok) return KVQ_ERR_UNSUPPORTED_DIM;
    if (plan->rot && plan->dec_impl == KVQ_IMPL_FFT) return KVQ_ERR_UNSUPPORTED_DIM;   // the rotation lives in the D x D tables
    if ((st = ensure_device(plan)) != KVQ_OK) return st;
    kvq_impl_t impl = plan->dec_impl;
    if (impl == KVQ_IMPL_AUTO) {
        if (N <= matvec_max_rows(plan->D)) impl = KVQ_IMPL_MATVEC;
        else if (gemm_ok) impl = KVQ_IMPL_GEMM;
        else impl = plan->rot ? KVQ_IMPL_MATVEC : KVQ_IMPL_FFT;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (impl == KVQ_IMPL_GEMM) {
        GemmParams g;
        g.packed = packed;
        g.scales = scales;
        g.lambda = lambda;
        g.out = out;
        g.b0 = plan->d_b0;
        g.N = N;
        g.n_lambda = n_lambda;
        g.rows_per_lambda = rows_per_lambda < 1 ? 1 : rows_per_lambda;
        g.per_vector = plan->group == plan->D;
        g.status = plan->d_status;
        // D = 256: the radix-2 kernel needs the transform's even / odd structure, which a rotation destroys
        const cudaError_t e = plan->rot && plan->D == 256 ? umma_decode_d256_dense(bf16, N, g, stream)
                                                          : umma_decode(plan->D, bf16, plan->bits, N, g, plan->sign_xor, stream, !plan->rot);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return KVQ_ERR_CUDA;
        }
        return KVQ_OK;
    }
    FftParams prm;
    fill_params(plan, prm, N, lambda, n_lambda, rows_per_lambda);
    prm.packed = const_cast<uint8_t *>(packed);
    prm.scales = const_cast<void *>(scales);
    prm.out = out;
    const cudaError_t e = impl == KVQ_IMPL_MATVEC ? matvec_decode(plan->D, plan->group, plan->bits, bf16, N, prm, plan->d_e0, stream)
                                                  : fft_decode(plan->D, plan->group, plan->bits, bf16, N, prm, stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}

kvq_status_t kvq_append_at(kvq_plan_t *plan, const void *x_new, kvq_dtype_t dtype, int64_t S, const float *lambda,
                           int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache, void *scales_cache,
                           int64_t T_max, const int64_t *pos_device, void *cuda_stream)
{
    if (T_max < 1) return KVQ_ERR_INVALID_ARG;
    if (S == 0) return plan ? KVQ_OK : KVQ_ERR_INVALID_ARG;
    if (!pos_device) return KVQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(pos_device) & 7u) return KVQ_ERR_ALIGNMENT;
    const DevicePos pos{pos_device, T_max - 1};
    return encode_common(plan, x_new, dtype, S, lambda, n_lambda, streams_per_lambda, packed_cache, scales_cache,
                         RowMap{1, T_max, 0}, cuda_stream, nullptr, nullptr, &pos);
}

static kvq_status_t flush_common(kvq_plan_t *plan, const void *x_block, kvq_dtype_t dtype, int64_t S, int64_t rows,
                                 const float *lambda, int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache,
                                 void *scales_cache, void *dq_cache, int64_t T_max, int64_t pos0, const int64_t *pos0_device,
                                 bool at, void *cuda_stream);

kvq_status_t kvq_flush_block(kvq_plan_t *plan, const void *x_block, kvq_dtype_t dtype, int64_t S, int64_t rows, const float *lambda,
                             int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache, void *scales_cache, void *dq_cache,
                             int64_t T_max, int64_t pos0, void *cuda_stream)
{
    return flush_common(plan, x_block, dtype, S, rows, lambda, n_lambda, streams_per_lambda, packed_cache, scales_cache, dq_cache,
                        T_max, pos0, nullptr, false, cuda_stream);
}

kvq_status_t kvq_flush_block_at(kvq_plan_t *plan, const void *x_block, kvq_dtype_t dtype, int64_t S, int64_t rows, const float *lambda,
                                int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache, void *scales_cache,
                                void *dq_cache, int64_t T_max, const int64_t *pos0_device, void *cuda_stream)
{
    return flush_common(plan, x_block, dtype, S, rows, lambda, n_lambda, streams_per_lambda, packed_cache, scales_cache, dq_cache,
                        T_max, 0, pos0_device, true, cuda_stream);
}

static kvq_status_t flush_common(kvq_plan_t *plan, const void *x_block, kvq_dtype_t dtype, int64_t S, int64_t rows,
                                 const float *lambda, int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache,
                                 void *scales_cache, void *dq_cache, int64_t T_max, int64_t pos0, const int64_t *pos0_device,
                                 bool at, void *cuda_stream)
{
    if (!plan || S < 0 || rows < 0) return KVQ_ERR_INVALID_ARG;
    if (T_max < 1 || pos0 < 0 || rows > T_max || pos0 > T_max - rows) return KVQ_ERR_INVALID_ARG;
    if (dtype != KVQ_F16 && dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
    if (S == 0 || rows == 0) return KVQ_OK;
    if (!dq_cache || (at && !pos0_device)) return KVQ_ERR_INVALID_ARG;
    if (misaligned16(dq_cache) || (reinterpret_cast<uintptr_t>(pos0_device) & 7u)) return KVQ_ERR_ALIGNMENT;
    if (S > INT64_MAX / rows) return KVQ_ERR_INVALID_ARG;
    const int64_t N = S * rows;
    // lambda row of block row r: stream (r / rows) / streams_per_lambda
    const int64_t rpl = (streams_per_lambda < 1 ? 1 : streams_per_lambda) * rows;
    const RowMap map{rows, T_max, pos0};
    if (!at && plan->rot && plan->dec_impl == KVQ_IMPL_FFT) return KVQ_ERR_UNSUPPORTED_DIM;
    bool fused = false;
    const DevicePos pos{pos0_device, T_max - rows};
    kvq_status_t st = encode_common(plan, x_block, dtype, N, lambda, n_lambda, rpl, packed_cache, scales_cache, map, cuda_stream,
                                    dq_cache, &fused, at ? &pos : nullptr);
    if (st != KVQ_OK || fused) return st;
    if (at) return KVQ_ERR_CUDA;   // the fused launch is the only form that reads the position on the device
    // the same rows back out of the int4 cache into the dequantized-prefix cache: what a later full-prefix decode would give
    FftParams prm;
    fill_params(plan, prm, N, lambda, n_lambda, rpl);
    prm.packed = packed_cache;
    prm.scales = scales_cache;
    prm.out = dq_cache;
    prm.in_map = map;
    prm.out_map = map;
    const bool mv = flush_decode_is_matvec(plan, N);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool bf16 = dtype == KVQ_BF16;
    // A large block of a plan without a rotation: the tensor-core decode, reading and writing the window [pos0, pos0 + rows)
    // of every stream's cache in place through a cache view (tiles of 128 rows per stream, so blocks of 64 rows and more;
    // the whole cache must fit 32-bit tensor-map coordinates).
    if (!mv && plan->dec_impl != KVQ_IMPL_FFT && gemm_decode_ok(plan, bf16) && (rows >= 64 || plan->dec_impl == KVQ_IMPL_GEMM) &&
        S <= (((int64_t)1 << 31) - 1) / T_max) {
        GemmParams g;
        g.packed = packed_cache;
        g.scales = scales_cache;
        g.lambda = lambda;
        g.out = dq_cache;
        g.b0 = plan->d_b0;
        g.N = N;
        g.n_lambda = n_lambda;
        g.rows_per_lambda = rpl;
        g.per_vector = plan->group == plan->D;
        g.status = plan->d_status;
        g.view = CacheView{rows, T_max, pos0, streams_per_lambda < 1 ? 1 : streams_per_lambda};
        if (umma_decode(plan->D, bf16, plan->bits, N, g, plan->sign_xor, stream, true) != cudaSuccess) {
            (void)cudaGetLastError();
            return KVQ_ERR_CUDA;
        }
        return KVQ_OK;
    }
    const cudaError_t e = mv ? matvec_decode(plan->D, plan->group, plan->bits, bf16, N, prm, plan->d_e0, stream)
                             : fft_decode(plan->D, plan->group, plan->bits, bf16, N, prm, stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    return KVQ_OK;
}

// lambda_c = 1 / amax_c (1 where the channel carried nothing), in place over the bit patterns the reducing epilogue left
static __global__ void kvq_calibrate_finish_kernel(float *lambda, int D)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < D) {
        const float a = lambda[c];
        lambda[c] = a > 0.0f ? 1.0f / a : 1.0f;
    }
}

kvq_status_t kvq_calibrate_lambda(kvq_plan_t *plan, const void *x, kvq_dtype_t dtype, int64_t N, float *lambda_out, void *cuda_stream)
{
    if (!plan || N < 0 || !lambda_out) return KVQ_ERR_INVALID_ARG;
    if (dtype != KVQ_F16 && dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
    if (N > 0 && !x) return KVQ_ERR_INVALID_ARG;
    if (misaligned16(x) || misaligned16(lambda_out)) return KVQ_ERR_ALIGNMENT;
    if (!umma_calibrate_supported(plan->D, dtype == KVQ_BF16)) return KVQ_ERR_UNSUPPORTED_DIM;
    kvq_status_t st = ensure_device(plan);
    if (st != KVQ_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(lambda_out, 0, sizeof(float) * (size_t)plan->D, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVQ_ERR_CUDA;
    }
    if (N > 0) {
        FftParams prm;
        fill_params(plan, prm, N, nullptr, 1, 1);
        prm.in = x;
        if (umma_calibrate(plan->D, dtype == KVQ_BF16, N, prm, plan->d_e0, reinterpret_cast<uint32_t *>(lambda_out), stream) !=
            cudaSuccess) {
            (void)cudaGetLastError();
            return KVQ_ERR_CUDA;
        }
    }
    kvq_calibrate_finish_kernel<<<(plan->D + 127) / 128, 128, 0, stream>>>(lambda_out, plan->D);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return KVQ_ERR_CUDA;
    return KVQ_OK;
}

const char *kvq_status_string(kvq_status_t status)
{
    switch (status) {
        case KVQ_OK: return "KVQ_OK";
        case KVQ_ERR_INVALID_ARG: return "KVQ_ERR_INVALID_ARG";
        case KVQ_ERR_UNSUPPORTED_DIM: return "KVQ_ERR_UNSUPPORTED_DIM";
        case KVQ_ERR_ALIGNMENT: return "KVQ_ERR_ALIGNMENT";
        case KVQ_ERR_CUDA: return "KVQ_ERR_CUDA";
        case KVQ_ERR_TIMEOUT: return "KVQ_ERR_TIMEOUT";
        case KVQ_ERR_NOMEM: return "KVQ_ERR_NOMEM";
        case KVQ_ERR_SCRATCH_LIMIT: return "KVQ_ERR_SCRATCH_LIMIT";
        case KVQ_ERR_RANGE: return "KVQ_ERR_RANGE";
    }
    return "KVQ_ERR_UNKNOWN";
}

uint64_t kvq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
