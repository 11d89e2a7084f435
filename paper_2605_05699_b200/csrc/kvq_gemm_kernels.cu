// tcgen05 DFT-as-GEMM decode kernel of libkvq (sm_100a), D = 128, fp16 output.
//
// The inverse path x^ = diag(s) M^T diag(1 / max(lambda, 1e-6)) (q (.) sigma) (Sec. 3.1 "unpack,
// irfft, apply s"; Sec. 5.1 item 1) is a dense D x D contraction per vector.  Over a tile of 128
// vectors it is one 128 x 128 x 128 GEMM, which the 5th-generation tensor core runs in a quarter
// of the time the tile's bytes need to cross HBM, while the fp32 register FFT needs ~3000
// instructions per vector and is issue-bound at about a third of the HBM roofline.
//
//   A [128 vectors, K = 128]  fp16, built in shared memory by the CTA's 128 threads: thread t
//                             unpacks the nibbles of vector t and multiplies by the group scale
//                             (two codes per half2 instruction);
//   B [N = 128 outputs, K]    fp16, W'[n, c] = s_n M[c, n] / max(lambda_c, 1e-6) / rho, built by the
//                             CTA from the plan's fp32 table each time the lambda row changes
//                             (rho = power of two that normalises the largest 1 / lambda to [1, 2));
//   D [128, 128]              fp32 accumulator in tensor memory; thread t reads back row t
//                             (tcgen05.ld 32x32b), rounds to fp16 and stages it for a bulk store.
//
// Both operands are K-major with the 128-byte swizzle: two K blocks of [128 rows x 128 B].  The
// K order inside a word of 8 codes is (0,4,1,5,2,6,3,7): that is how the half2 nibble trick
// delivers them, and B is built in the same order, so no instruction is spent on reordering.
//
// Precision: A and B are each rounded once to fp16 (q sigma rho and W'), accumulation is fp32:
// about 3e-4 relative L2 per vector before the output rounding, inside the 1e-3 tolerance for
// fp16 output.  bf16 output, whose rounding step is 8x coarser, stays on the fp32 FFT kernels.
// Domain: group scales times rho and the entries of W' must stay in fp16's normal range
// (6.1e-5 .. 65504); lambda rows whose entries spread over more than ~2^9 lose precision on the
// small-1/lambda channels.  Outside that domain use KVQ_IMPL_FFT.
//
// Every wait on an mbarrier is bounded; on a time-out the CTA records the reason in the plan's
// status word, frees its tensor memory and returns.
#include "kvq_device.cuh"
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kD = 128;
constexpr int kTile = 128;                 // vectors per tile = MMA M
constexpr int kThreads = 128;
constexpr int kBBytes = 2 * kTile * 128;   // 32 KB: two K blocks of [128 rows x 128 B]
constexpr int kABytes = 2 * kTile * 128;
constexpr int kOutStride = 2 * kD + 16;    // padded fp16 row in the staging area (aliases A)
constexpr int kAOutBytes = kTile * kOutStride;
constexpr int kInStride = kD / 2 + 16;
constexpr int kInBytes = 2 * kTile * kInStride;
constexpr int kRlBytes = kD * 4;
constexpr int kCtrlBytes = 64;
constexpr int kSmemBytes = kBBytes + kAOutBytes + kInBytes + kRlBytes + kCtrlBytes + 1024;   // + alignment slack
constexpr uint32_t kTmemCols = 128;

// instruction descriptor: D = f32, A = B = f16, both K-major, N = 128, M = 128
constexpr uint32_t kIdesc = (1u << 4) | ((uint32_t)(kD >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);

__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    // start address >> 4 | LBO 0 | SBO 1024 B (8 rows x 128 B) | version 1 | 128-byte swizzle
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));   // (a & b) | c
    return d;
}

// byte offset of 16-byte chunk j (0..15 along K) of row r in a [2 K blocks][128 rows][128 B] swizzled operand
__device__ __forceinline__ uint32_t sw128_chunk(int r, int j) { return (uint32_t)((j >> 3) * (kTile * 128) + r * 128 + (((j & 7) ^ (r & 7)) << 4)); }

}  // namespace

__global__ void __launch_bounds__(kThreads) kvq_decode_gemm_d128_kernel(const __grid_constant__ GemmParams prm)
{
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the swizzled operands
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;
    unsigned char *sA = smem + kBBytes;              // also the output staging area
    unsigned char *sIn = sA + kAOutBytes;
    float *sRl = reinterpret_cast<float *>(sIn + kInBytes);
    unsigned char *sCtrl = reinterpret_cast<unsigned char *>(sRl) + kRlBytes;
    const uint32_t in_bar0 = smem_u32(sCtrl), in_bar1 = in_bar0 + 8, mma_bar = in_bar0 + 16;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sCtrl + 32);
    float *rho_slot = reinterpret_cast<float *>(sCtrl + 40);

    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;

    if (t == 0) {
        mbar_init(in_bar0, kThreads);
        mbar_init(in_bar1, kThreads);
        mbar_init(mma_bar, 1);
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // ---- tiles: lambda segments of rows_per_lambda rows, cut into tiles of 128 rows; a contiguous
    // ---- range of tiles per CTA so that the B operand is rebuilt as rarely as possible
    const int64_t N = prm.N;
    const int64_t rpl = prm.n_lambda == 1 ? N : prm.rows_per_lambda;
    const int64_t tps = (rpl + kTile - 1) / kTile;                 // tiles per segment
    const int64_t n_seg = (N + rpl - 1) / rpl;
    const int64_t n_tiles = n_seg * tps;
    const int64_t per_cta = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per_cta;
    const int64_t tile_end = tile_begin + per_cta < n_tiles ? tile_begin + per_cta : n_tiles;

    const unsigned char *packed = static_cast<const unsigned char *>(prm.packed);
    const uint2 *scales = static_cast<const uint2 *>(prm.scales);   // 4 fp16 scales per row
    unsigned char *out = static_cast<unsigned char *>(prm.out);

    auto tile_rows = [&](int64_t tile, int64_t &row0, int &nrows, int64_t &seg) {
        seg = tile / tps;
        const int64_t off = (tile - seg * tps) * kTile;
        int64_t seg_rows = N - seg * rpl;
        if (seg_rows > rpl) seg_rows = rpl;
        row0 = seg * rpl + off;
        const int64_t left = seg_rows - off;
        nrows = left >= kTile ? kTile : (left > 0 ? (int)left : 0);
    };
    auto issue = [&](int64_t tile, int stage) {
        int64_t row0, seg;
        int nrows;
        tile_rows(tile, row0, nrows, seg);
        const uint32_t bar = stage ? in_bar1 : in_bar0;
        if (t < nrows) {
            mbar_arrive_expect_tx(bar, kD / 2);
            bulk_load(smem_u32(sIn + (stage * kTile + t) * kInStride), packed + (row0 + t) * (kD / 2), kD / 2, bar);
        } else {
            mbar_arrive(bar);
        }
    };
    auto load_scales = [&](int64_t tile) -> uint2 {
        int64_t row0, seg;
        int nrows;
        tile_rows(tile, row0, nrows, seg);
        return t < nrows ? __ldg(scales + row0 + t) : make_uint2(0u, 0u);
    };

    uint2 sc_next = make_uint2(0u, 0u);
    if (tile_begin < tile_end) {
        issue(tile_begin, 0);
        sc_next = load_scales(tile_begin);
    }
    int64_t cached_seg = -1;
    float rho = 1.0f;
    uint32_t in_phases = 0, mma_phase = 0;
    int stage = 0;
    bool failed = false;

    for (int64_t tile = tile_begin; tile < tile_end; ++tile, stage ^= 1) {
        const uint2 sc = sc_next;
        if (tile + 1 < tile_end) {
            issue(tile + 1, stage ^ 1);
            sc_next = load_scales(tile + 1);
        }
        int64_t row0, seg;
        int nrows;
        tile_rows(tile, row0, nrows, seg);

        // ---- B operand for this lambda row (rare)
        if (seg != cached_seg) {
            const int64_t lr = prm.n_lambda == 1 ? 0 : seg;
            __syncthreads();   // nobody still reads sRl / the tensor core no longer reads sB (previous MMA was waited for)
            float rl = __frcp_rn(fmaxf(__ldg(prm.lambda + lr * kD + t), 1e-6f));
            float mx = rl;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            if (lane == 0) sRl[warp] = mx;   // temporarily: per-warp maxima in the first four slots
            __syncthreads();
            mx = fmaxf(fmaxf(sRl[0], sRl[1]), fmaxf(sRl[2], sRl[3]));
            rho = __uint_as_float(__float_as_uint(mx) & 0x7F800000u);   // 2^floor(log2 max): exact to divide by
            __syncthreads();
            sRl[t] = rl / rho;
            __syncthreads();
            const float4 *b0 = reinterpret_cast<const float4 *>(prm.b0 + (size_t)t * kD);   // row n = t, canonical c order
#pragma unroll 4
            for (int w = 0; w < 16; ++w) {
                float4 m0 = __ldg(b0 + 2 * w), m1 = __ldg(b0 + 2 * w + 1);
                float4 l0 = reinterpret_cast<const float4 *>(sRl)[2 * w], l1 = reinterpret_cast<const float4 *>(sRl)[2 * w + 1];
                auto sat = [](float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); };
                uint4 ch;
                ch.x = narrow2<false>(sat(m0.x * l0.x), sat(m1.x * l1.x));   // K order (0,4,1,5,2,6,3,7) of the word
                ch.y = narrow2<false>(sat(m0.y * l0.y), sat(m1.y * l1.y));
                ch.z = narrow2<false>(sat(m0.z * l0.z), sat(m1.z * l1.z));
                ch.w = narrow2<false>(sat(m0.w * l0.w), sat(m1.w * l1.w));
                *reinterpret_cast<uint4 *>(sB + sw128_chunk(t, w)) = ch;
            }
            cached_seg = seg;
            // visibility to the tensor core is established by the fence + barrier before the MMA below
        }

        // ---- packed codes of this tile have landed?
        bool ok = mbar_wait_bounded(stage ? in_bar1 : in_bar0, (in_phases >> stage) & 1u);
        in_phases ^= 1u << stage;
        // ---- all bulk stores of the previous tile have drained the staging area that A aliases
        bulk_wait_read_all();
        if (__syncthreads_or(!ok)) {
            if (t == 0) atomicOr(prm.status, KVQ_DEV_LOAD_TIMEOUT);
            failed = true;
            break;
        }

        // ---- A row: nibbles -> fp16 codes -> times sigma * rho, two codes per instruction
        if (t < nrows) {
            const uint4 *row = reinterpret_cast<const uint4 *>(sIn + (stage * kTile + t) * kInStride);
            const __half2 h1032 = __float2half2_rn(1032.0f);
            __half2 s2[4];
            {
                __half2 a = *reinterpret_cast<const __half2 *>(&sc.x), b = *reinterpret_cast<const __half2 *>(&sc.y);
                float2 fa = __half22float2(a), fb = __half22float2(b);
                s2[0] = __float2half2_rn(fa.x * rho), s2[1] = __float2half2_rn(fa.y * rho);
                s2[2] = __float2half2_rn(fb.x * rho), s2[3] = __float2half2_rn(fb.y * rho);
            }
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                uint4 pk = row[q4];
                uint32_t words[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int w = 4 * q4 + i;                       // word w: codes 8w .. 8w+7, group w / 4
                    const uint32_t u = words[i] ^ 0x88888888u;      // nibbles now hold q + 8
                    uint32_t r[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint32_t m = lop3_and_or(u >> (4 * e), 0x000F000Fu, 0x64006400u);   // {1024 + n_e, 1024 + n_{e+4}}
                        __half2 h = __hmul2(__hsub2(*reinterpret_cast<__half2 *>(&m), h1032), s2[w >> 2]);
                        r[e] = *reinterpret_cast<uint32_t *>(&h);
                    }
                    *reinterpret_cast<uint4 *>(sA + sw128_chunk(t, w)) = make_uint4(r[0], r[1], r[2], r[3]);
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();

        // ---- one thread issues the 128 x 128 x 128 MMA as 8 K steps of 16
        if (t == 0) {
            tc_fence_after();
            const uint32_t a0 = smem_u32(sA), b0s = smem_u32(sB);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t koff = (uint32_t)((ks >> 2) * (kTile * 128) + (ks & 3) * 32);
                umma_f16(tmem_base, smem_desc_sw128(a0 + koff), smem_desc_sw128(b0s + koff), kIdesc, ks > 0 ? 1u : 0u);
            }
            umma_commit(mma_bar);
        }
        ok = mbar_wait_bounded(mma_bar, mma_phase);
        mma_phase ^= 1u;
        if (__syncthreads_or(!ok)) {
            if (t == 0) atomicOr(prm.status, KVQ_DEV_MMA_TIMEOUT);
            failed = true;
            break;
        }
        tc_fence_after();

        // ---- epilogue: row t of the accumulator -> fp16 -> staging row -> bulk store
        {
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
            unsigned char *orow = sA + t * kOutStride;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t r[32];
                tmem_ld32(taddr + cc * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 o;
                    o.x = narrow2<false>(__uint_as_float(r[8 * j]), __uint_as_float(r[8 * j + 1]));
                    o.y = narrow2<false>(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3]));
                    o.z = narrow2<false>(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5]));
                    o.w = narrow2<false>(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7]));
                    *reinterpret_cast<uint4 *>(orow + cc * 64 + j * 16) = o;
                }
            }
        }
        tc_fence_before();
        // the staging rows overlap other threads' A rows: everyone must be done reading tensor memory and
        // writing staging before any bulk store is issued or the next tile's A is written
        fence_proxy_async();
        __syncthreads();
        if (t < nrows) {
            bulk_store(out + (row0 + t) * (2 * kD), smem_u32(sA + t * kOutStride), 2 * kD);
            bulk_commit();
        }
    }

    if (failed) {
        // let this thread's own copies in flight land (bounded) before the CTA goes away
        (void)mbar_wait_bounded(in_bar0, in_phases & 1u, 1u << 16);
        (void)mbar_wait_bounded(in_bar1, (in_phases >> 1) & 1u, 1u << 16);
    }
    bulk_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

cudaError_t gemm_decode_d128(int64_t N, const GemmParams &prm, cudaStream_t stream)
{
    static int blocks_per_sm = 0, sms = 0;
    if (blocks_per_sm == 0) {
        cudaError_t e = cudaFuncSetAttribute(kvq_decode_gemm_d128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        int dev = 0, nb = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kvq_decode_gemm_d128_kernel, kThreads, kSmemBytes)) != cudaSuccess)
            return e;
        if (nb < 1) return cudaErrorLaunchOutOfResources;
        if (nb > 2) nb = 2;   // 2 x 128 tensor-memory columns per SM; more CTAs would only wait in tcgen05.alloc
        blocks_per_sm = nb;
    }
    const int64_t rpl = prm.n_lambda == 1 ? N : prm.rows_per_lambda;
    const int64_t tiles = ((N + rpl - 1) / rpl) * ((rpl + kTile - 1) / kTile);
    const int64_t cap = (int64_t)blocks_per_sm * sms;
    const int grid = (int)(tiles < cap ? tiles : cap);
    kvq_decode_gemm_d128_kernel<<<grid, kThreads, kSmemBytes, stream>>>(prm);
    count_launch();
    return cudaGetLastError();
}

}  // namespace kvq
