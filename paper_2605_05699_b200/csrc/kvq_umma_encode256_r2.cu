// tcgen05 encode kernel of libkvq for D = 256 with one radix-2 step of the transform taken out of the GEMM (sm_100a):
// groups of 32, 4-bit codes, fp16 or bf16 input, plans without a rotation.
//
// Rows of the forward transform M (Sec. 3.1 Eq. 1-2) are cos / sin(2 pi k n / D).  With D / 2 = 128,
//     cos(2 pi (128 - k) n / D) = (-1)^n cos(2 pi k n / D),      sin(2 pi (128 - k) n / D) = -(-1)^n sin(2 pi k n / D),
// so with E_k / O_k the sums over the even / odd inputs n,
//     z_k = E_k + O_k,      z_{128 - k} = +-(E_k - O_k)      (+ for the cosine channels, - for the sine channels):
// channels k and 128 - k come out of the same two half-size sums.  The inputs are ROUTED by the parity of n, not added, so
// x stays exact in its 16-bit format and the table keeps its two 16-bit terms (the codes must agree with an fp64
// evaluation on all but 1e-4 of the entries): per tile of 128 vectors, two 128 x 128 x 128 contractions per term instead
// of one 128 x 256 x 256.  Half the tensor work of the dense kernel -- which at D = 256 is what bounds it: the dense
// form needs more tensor-core time per vector than the vector's bytes need to cross HBM -- and the whole tile fits one
// CTA, so no pair of CTAs reads the same x twice.
//
// Columns of E and O (128 each): j < 64: cos k = j (channel j; E - O is channel 128 - j, the Nyquist channel for j = 0);
// 64 <= j < 127: sin k = j - 63 (channel 128 + k; O - E is channel 256 - k); j = 127: cos 64 in E and sin 64 in O (each is
// zero on the other parity).  A column serves two channels, so lambda (Sec. 5.1 item 1) cannot live in the B operand: it
// is applied in the epilogue, in fp32, and B does not depend on the lambda row.  B is therefore one fixed 128 KB image
// per plan and input type, built on the host when the plan's tables are made and fetched by one bulk copy per CTA.
//
//   warp 0       producer   the B image (bulk copy), then TMA tensor loads of the x tile: a ring of K blocks (64 inputs x
//                           128 rows, 128-byte swizzle)
//   warps 2-5    router     thread = row: LDS.128 of the landed block, even / odd inputs pulled apart (PRMT), A operands
//                           into tensor memory (two stages)
//   warp 1       mma        per tile: 2 parities x 2 terms x 8 K-steps (A from tensor memory, B from shared memory) into
//                           the one accumulator stage (E: columns 0-127, O: 128-255)
//   warps 6-21   epilogue   thread = (row, two groups of 32 channels): E and O columns -> sums and differences in
//                           channel order -> lambda -> group abs-max, fp16 scale, codes, nibble pack (Sec. 3.2 steps 3-4,
//                           Sec. 7.1) -> global memory.  The accumulator is read in two passes of 64 columns per thread and
//                           handed back when the second pass is in registers.
// Every wait on an mbarrier is bounded (status word, abort flag): on a time-out the CTA lets what it issued land, frees its
// tensor memory and returns.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cmath>

#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

namespace {

constexpr int kD = 256, kG = kD / 32, kTile = 128;
constexpr int kRouterWarps = 4, kEpiWarps = 16;
constexpr int kEpi0 = 2 + kRouterWarps;                  // first epilogue warp
constexpr int kThreads = (kEpi0 + kEpiWarps) * 32;       // producer, mma, 4 router and 16 epilogue warps
constexpr int kBlockBytes = kTile * 128;                 // one K block of x: 128 rows x 128 B
constexpr int kKBlocks = kD / 64;                        // 4 K blocks per tile
constexpr int kRing = 6;                                 // K blocks of x in flight
constexpr int kBBlock = 128 * 128;                       // one K block of one B part: 128 columns x 128 B
constexpr int kBPart = 2 * kBBlock;                      // [128 columns][128 inputs of one parity], 16-bit: 32 KB
constexpr int kBBytes = 4 * kBPart;                      // [term][parity]: 128 KB
constexpr int kCtrlBytes = 1024;
constexpr int kSmemBytes = kBBytes + kRing * kBlockBytes + kCtrlBytes + 1024;
static_assert(kSmemBytes <= 232448, "shared memory over the per-CTA limit");
static_assert(kBBytes == kR2ImageBytes, "image size");
constexpr uint32_t kTmemCols = 512, kACol0 = 256, kAStride = 128;   // accumulator E | O at 0, two A stages (even | odd) behind it
constexpr int kAStages = 2;

struct Ctrl {
    uint64_t in_full[kRing], in_empty[kRing];
    uint64_t a_full[kAStages], a_empty[kAStages];
    uint64_t acc_full, acc_empty;
    uint64_t b_full;
    uint32_t tmem_base;
    volatile uint32_t abort;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// channel whose even-input (p = 0) or odd-input (p = 1) sum column j holds
__host__ __device__ constexpr int column_channel(int j, int p) { return j < 64 ? j : j < 127 ? j + 65 : (p ? 192 : 64); }

__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t &r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
}

}  // namespace

struct UmmaEncode256R2Params {
    const float *lambda;    // [n_lambda, D] fp32
    const void *b_image;    // the plan's B image for this input type (kR2ImageBytes, the shared-memory layout)
    unsigned char *packed;  // [*, D/2] bytes out
    uint16_t *scales;       // [*, D/32] fp16 out
    int64_t N, n_lambda, rpl, n_seg;
    RowMap out_map;
    float unlift;           // 1 / 2^k, 2^k the lift the image was built with
    uint32_t *status;
};

template <bool BF16>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_encode_umma_d256_r2_kernel(const __grid_constant__ UmmaEncode256R2Params prm, const __grid_constant__ CUtensorMap tm_x)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;                    // [term][parity][2 K blocks][128 columns][128 B]
    unsigned char *sIn = sB + kBBytes;           // ring of K blocks of x
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sIn + kRing * kBlockBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range per CTA
    const int64_t N = prm.N, rpl = prm.rpl;
    const int64_t tps = (rpl + kTile - 1) / kTile;
    const int64_t n_tiles = prm.n_seg * tps;
    const int64_t per_cta = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per_cta;
    const int64_t tile_end = tile_begin + per_cta < n_tiles ? tile_begin + per_cta : n_tiles;
    const int n_my = tile_end > tile_begin ? (int)(tile_end - tile_begin) : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
            mbar_init(smem_u32(&ctrl->in_empty[s]), kRouterWarps);
        }
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(smem_u32(&ctrl->a_full[s]), kRouterWarps);
            mbar_init(smem_u32(&ctrl->a_empty[s]), 1);
        }
        mbar_init(smem_u32(&ctrl->acc_full), 1);
        mbar_init(smem_u32(&ctrl->acc_empty), kEpiWarps);
        mbar_init(smem_u32(&ctrl->b_full), 1);
        ctrl->abort = 0u;
        mbar_init_fence();
        if (n_my > 0) {   // the B image: eight bulk copies of 16 KB onto one barrier
            const uint32_t bar = smem_u32(&ctrl->b_full);
            mbar_arrive_expect_tx(bar, kBBytes);
            for (int i = 0; i < kBBytes / 16384; ++i)
                bulk_load(smem_u32(sB + i * 16384), static_cast<const unsigned char *>(prm.b_image) + i * 16384, 16384, bar);
        }
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile uint32_t *abort_flag = &ctrl->abort;
    uint32_t *status = prm.status;
    int issued = 0;   // producer thread: K blocks of x whose loads have been issued

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my && ok; ++j, cur.advance(1)) {
                const int64_t row0 = cur.seg * rpl + cur.row_in_segment();
#pragma unroll
                for (int kb = 0; kb < kKBlocks; ++kb) {
                    const int u = kKBlocks * j + kb, s = u % kRing;
                    ok = wait_or_abort(smem_u32(&ctrl->in_empty[s]), ((uint32_t)(u / kRing) & 1u) ^ 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                    mbar_arrive_expect_tx(bar, kBlockBytes);
                    tma_load_2d(smem_u32(sIn + s * kBlockBytes), &tm_x, 64 * kb, (int)row0, bar);   // rows past N arrive as zeros
                    issued = u + 1;
                }
            }
        }
    } else if (warp == 1) {
        // =========================== mma issuer ===========================
        if (lane == 0) {
            const uint64_t b_desc = smem_desc_sw128(smem_u32(sB));
            const uint32_t b_lo = (uint32_t)b_desc, b_hi = (uint32_t)(b_desc >> 32);
            constexpr uint32_t kIdesc = umma_idesc_m128(128, BF16);
            int n_mma = n_my;
            if (n_my > 0 && !wait_or_abort(smem_u32(&ctrl->b_full), 0u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) n_mma = 0;
            for (int j = 0; j < n_mma; ++j) {
                const int sa = j % kAStages;
                if (!wait_or_abort(smem_u32(&ctrl->a_full[sa]), (uint32_t)(j / kAStages) & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                // the epilogue has taken the previous tile's E and O out of tensor memory
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty), ((uint32_t)j & 1u) ^ 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                tc_fence_after();
#pragma unroll
                for (int p = 0; p < 2; ++p) {   // E = (even inputs) x B_even, O = (odd inputs) x B_odd
                    const uint32_t d_tmem = tmem_base + (uint32_t)p * 128u;
                    const uint32_t a_tmem = tmem_base + kACol0 + (uint32_t)sa * kAStride + (uint32_t)p * 64u;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t koff = (uint32_t)(ks >> 2) * (kBBlock >> 4) + (uint32_t)(ks & 3) * 2u;   // (bytes >> 4) of K-step ks
                            const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + (uint32_t)((t * 2 + p) * (kBPart >> 4)) + koff);
                            if (t > 0 || ks > 0) umma_f16_ts<true>(d_tmem, a_tmem + (uint32_t)ks * 8u, bd, kIdesc);
                            else umma_f16_ts<false>(d_tmem, a_tmem, bd, kIdesc);
                        }
                    }
                }
                umma_commit(smem_u32(&ctrl->acc_full));
                umma_commit(smem_u32(&ctrl->a_empty[sa]));
            }
        }
    } else if (warp < kEpi0) {
        // =========================== router: x tile -> even / odd A operands in tensor memory ===========================
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int r = q * 32 + lane;            // tile row and tensor-memory lane of this thread
        const uint32_t a_row = tmem_base + ((uint32_t)(q * 32) << 16) + kACol0;
        for (int j = 0; j < n_my; ++j) {
            const int sa = j % kAStages;
            if (j >= kAStages) {   // the MMAs that read this A stage last
                const int jp = j - kAStages;
                if (!wait_or_abort(smem_u32(&ctrl->a_empty[sa]), (uint32_t)(jp / kAStages) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            }
            tc_fence_after();
            const uint32_t a_dst = a_row + (uint32_t)sa * kAStride;
            bool ok = true;
#pragma unroll
            for (int kb = 0; kb < kKBlocks; ++kb) {   // 64 inputs: 16 words of each parity
                const int u = kKBlocks * j + kb, s = u % kRing;
                if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(u / kRing) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) {
                    ok = false;
                    break;
                }
                const unsigned char *row = sIn + s * kBlockBytes + r * 128;
                uint32_t ev[16], od[16];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 w = *reinterpret_cast<const uint4 *>(row + ((c ^ (r & 7)) << 4));
                    ev[2 * c] = __byte_perm(w.x, w.y, 0x5410), ev[2 * c + 1] = __byte_perm(w.z, w.w, 0x5410);
                    od[2 * c] = __byte_perm(w.x, w.y, 0x7632), od[2 * c + 1] = __byte_perm(w.z, w.w, 0x7632);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));   // the block is in registers
                tmem_st16(a_dst + 16u * (uint32_t)kb, ev);
                tmem_st16(a_dst + 64u + 16u * (uint32_t)kb, od);
            }
            if (!ok) break;
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->a_full[sa]));
        }
    } else {
        // =========================== epilogue ===========================
        // role 0: groups 0 and 3 from columns  0 .. 31 (+ column 32)      role 2: groups 4 and 7 from columns 64 .. 95 (+ column 0)
        // role 1: groups 1 and 2 from columns 32 .. 63 (+ E column 127)   role 3: groups 5 and 6 from columns 96 .. 127 (+ column 95)
        const int q = warp & 3;
        const int role = (warp - kEpi0) >> 2;   // warp-uniform
        const int r = q * 32 + lane;
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t e_main = t_addr + 32u * (uint32_t)role, o_main = e_main + 128u;
        const int gx = role == 0 ? 0 : role == 1 ? 1 : role == 2 ? 4 : 5;   // the group made of sums
        const int gy = role == 0 ? 3 : role == 1 ? 2 : role == 2 ? 7 : 6;   // the group made of differences
        const float unlift = prm.unlift;
        TileCursor cur(tile_begin, tps);
        for (int j = 0; j < n_my; ++j, cur.advance(1)) {
            __syncwarp();
            const int64_t seg = cur.seg, off = cur.row_in_segment();
            if (!wait_or_abort(smem_u32(&ctrl->acc_full), (uint32_t)j & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();
            int64_t seg_rows = N - seg * rpl;
            if (seg_rows > rpl) seg_rows = rpl;
            const bool live = off + r < seg_rows;
            const int64_t orow = prm.out_map(seg * rpl + off + r);
            const float *lam = prm.lambda + (prm.n_lambda == 1 ? 0 : seg) * kD;

            // Two passes of 32 channels each: the group made of sums, then the group made of differences (read in the mirrored
            // order).  A pass takes its 32 E and 32 O columns out of tensor memory 16 at a time; one copy of the group code
            // serves both passes.
#pragma unroll 1
            for (int pass = 0; pass < 2; ++pass) {
                float v[32];
                uint32_t x0 = 0u, x1 = 0u;
                if (pass == 0) {
                    if (role == 2) {          // channel 128 = E_0 - O_0
                        tmem_ld1(t_addr, x0);
                        tmem_ld1(t_addr + 128u, x1);
                    } else if (role == 3) {   // channel 160 = sin 32 = column 95
                        tmem_ld1(t_addr + 95u, x0);
                        tmem_ld1(t_addr + 128u + 95u, x1);
                    }
                } else {
                    if (role == 0) {          // channel 96 = E_32 - O_32
                        tmem_ld1(t_addr + 32u, x0);
                        tmem_ld1(t_addr + 128u + 32u, x1);
                    } else if (role == 1) {   // channel 64 = cos 64 = E column 127
                        tmem_ld1(t_addr + 127u, x0);
                    }
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t e[16], o[16];
                    tmem_ld16(e_main + 16u * (uint32_t)h, e);
                    tmem_ld16(o_main + 16u * (uint32_t)h, o);
                    tmem_ld_wait();
                    if (pass == 1 && h == 1) {   // the last accumulator values are in registers: hand it back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty));
                    }
                    if (pass == 0) {
                        if (role < 2) {       // channel base + m = E + O of main column m
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[16 * h + i] = __uint_as_float(e[i]) + __uint_as_float(o[i]);
                        } else {              // channel base + m + 1 = E + O of main column m = 0 .. 30
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                if (16 * h + i < 31) v[16 * h + i + 1] = __uint_as_float(e[i]) + __uint_as_float(o[i]);
                        }
                    } else {
                        if (role < 2) {       // channel base + 32 - m = E - O of main column m = 1 .. 31
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                if (16 * h + i > 0) v[32 - 16 * h - i] = __uint_as_float(e[i]) - __uint_as_float(o[i]);
                        } else {              // channel base + 31 - m = O - E of main column m = 0 .. 30; m = 31: sin 96 | sin 64
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                if (16 * h + i < 31) v[31 - 16 * h - i] = __uint_as_float(o[i]) - __uint_as_float(e[i]);
                                else v[0] = role == 2 ? __uint_as_float(o[i]) - __uint_as_float(e[i]) : __uint_as_float(o[i]);
                            }
                        }
                    }
                }
                if (pass == 0) {
                    if (role == 2) v[0] = __uint_as_float(x0) - __uint_as_float(x1);
                    else if (role == 3) v[0] = __uint_as_float(x0) + __uint_as_float(x1);
                } else {
                    if (role == 0) v[0] = __uint_as_float(x0) - __uint_as_float(x1);
                    else if (role == 1) v[0] = __uint_as_float(x0);
                }

                // ---- lambda, group abs-max, fp16 scale, codes against the stored scale, nibble pack, store
                const int g = pass == 0 ? gx : gy;
                const float4 *l4 = reinterpret_cast<const float4 *>(lam + 32 * g);
                float am[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int k4 = 0; k4 < 8; ++k4) {
                    const float4 l = __ldg(l4 + k4);
                    v[4 * k4] *= l.x, v[4 * k4 + 1] *= l.y, v[4 * k4 + 2] *= l.z, v[4 * k4 + 3] *= l.w;   // still times the lift 2^k
                    am[k4 & 3] = fmaxf(fmaxf(am[k4 & 3], fabsf(v[4 * k4])), fabsf(v[4 * k4 + 1]));
                    am[k4 & 3] = fmaxf(fmaxf(am[k4 & 3], fabsf(v[4 * k4 + 2])), fabsf(v[4 * k4 + 3]));
                }
                const float amax = fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])) * unlift;   // the product is exact: a power of two
                // sigma = fp16(absmax / 7), the division taken as a product with fp32(1 / 7): the stored scale differs from
                // the exactly rounded one by an fp16 ulp on about 2e-4 of the groups, and the codes follow the stored scale
                const float sig = fminf(amax * 0.142857149f, 65504.0f);
                const __half hs = __float2half_rn(sig);
                const float sg = __half2float(hs);
                const float rs1 = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
                const bool clamp = !(amax * rs1 < 7.25f);   // saturated or subnormal scale: codes could leave [-7, 7]
                const float rs = rs1 * unlift;              // applies to the lifted values
                uint32_t words[4];
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    uint32_t a = 0;
                    if (!clamp) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) a += __float_as_uint(fmaf(v[8 * w + c], rs, kMagicRound)) << (4 * c);
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c) a += __float_as_uint(fminf(fmaxf(v[8 * w + c] * rs, -7.0f), 7.0f) + kMagicRound) << (4 * c);
                    }
                    words[w] = (a - kMagicSum) ^ 0x88888888u;
                }
                if (live) {
                    *reinterpret_cast<uint4 *>(prm.packed + orow * (kD / 2) + g * 16) = make_uint4(words[0], words[1], words[2], words[3]);
                    prm.scales[orow * kG + g] = __half_as_ushort(hs);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (*abort_flag) {
            // Every role has left its loop.  What may still be in flight was this thread's to issue: give the B image and the
            // last K blocks a bounded chance to land, then let tensor-core work that was already issued drain.
            if (lane == 0) {
                if (n_my > 0) (void)mbar_wait_bounded(smem_u32(&ctrl->b_full), 0u, 1u << 16);
                for (int u = issued > kRing ? issued - kRing : 0; u < issued; ++u)
                    (void)mbar_wait_bounded(smem_u32(&ctrl->in_full[u % kRing]), (uint32_t)(u / kRing) & 1u, 1u << 16);
            }
            __nanosleep(20000);
            __syncwarp();
        }
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------

// 2^k that brings the table's largest entry into [2^13, 2^14): the first 16-bit term of every entry times 2^k stays below
// fp16's maximum, the second above its subnormals
float r2_encode_lift(float table_max)
{
    int ex = 0;
    (void)std::frexp(table_max > 0.0f ? table_max : 1.0f, &ex);   // table_max = m 2^ex, m in [0.5, 1)
    return std::ldexp(1.0f, 14 - ex);
}

// The kernel's B operand as it sits in shared memory: [term][parity][K block][column][128 B, 128-byte swizzle].
// Entry (column j, input m of parity p) = term t of e0[column_channel(j, p)][2 m + p] 2^k, the terms being the value
// rounded to the 16-bit type and what that rounding left behind (exact in fp32), rounded again.
void r2_encode_b_image(const float *e0, float lift, bool bf16, void *image)
{
    unsigned char *img = static_cast<unsigned char *>(image);
    for (int p = 0; p < 2; ++p)
        for (int j = 0; j < 128; ++j) {
            const float *row = e0 + (size_t)column_channel(j, p) * kD;
            for (int m = 0; m < 128; ++m) {
                float w = row[2 * m + p] * lift;
                const size_t off = (size_t)(m >> 6) * kBBlock + (size_t)j * 128 + (size_t)(((((m & 63) >> 3)) ^ (j & 7)) << 4) + (size_t)(m & 7) * 2;
                for (int t = 0; t < 2; ++t) {
                    uint16_t bits;
                    float back;
                    if (bf16) {
                        const __nv_bfloat16 h = __float2bfloat16_rn(w);
                        bits = *reinterpret_cast<const uint16_t *>(&h);
                        back = __bfloat162float(h);
                    } else {
                        const __half h = __float2half_rn(w);
                        bits = *reinterpret_cast<const uint16_t *>(&h);
                        back = __half2float(h);
                    }
                    *reinterpret_cast<uint16_t *>(img + (size_t)(t * 2 + p) * kBPart + off) = bits;
                    w -= back;
                }
            }
        }
}

namespace {

template <bool BF16>
cudaError_t launch(int64_t N, const FftParams &f, cudaStream_t stream)
{
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int &sms = slots.sms[dev];
    if (sms == 0) {
        int n = 0;
        if ((e = cudaFuncSetAttribute(kvq_encode_umma_d256_r2_kernel<BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms = n;
    }
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaEncode256R2Params prm;
    prm.lambda = f.lambda;
    prm.b_image = f.r2_image;
    prm.packed = static_cast<unsigned char *>(f.packed);
    prm.scales = static_cast<uint16_t *>(f.scales);
    prm.N = N;
    prm.n_lambda = f.n_lambda;
    prm.rpl = f.n_lambda == 1 ? N : f.rows_per_lambda;
    prm.n_seg = (N + prm.rpl - 1) / prm.rpl;
    prm.out_map = f.out_map;
    prm.unlift = 1.0f / r2_encode_lift(f.table_max);
    prm.status = f.status;

    CUtensorMap tm_x;
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)(2 * kD)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    if (!make_tensor_map(&tm_x, BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, f.in, dims, strides, box,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    const int grid = (int)(tiles < sms ? tiles : sms);
    kvq_encode_umma_d256_r2_kernel<BF16><<<grid, kThreads, kSmemBytes, stream>>>(prm, tm_x);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t umma_encode_d256_r2(bool bf16, int64_t N, const FftParams &f, cudaStream_t stream)
{
    return bf16 ? launch<true>(N, f, stream) : launch<false>(N, f, stream);
}

}  // namespace kvq
