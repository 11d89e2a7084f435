// fp32 register-FFT kernels of libkvq: kvq_encode / kvq_append / kvq_decode for every
// supported head dimension, both half-precision types, groups of 32 or of the whole vector,
// and 4- or 8-bit codes.  Kernel templates; each (group, bits) variant is instantiated in a
// translation unit of its own (kvq_fft_*.cu) through KVQ_FFT_DEFINE_VARIANT.
//
// Mapping.  One thread owns one vector for its whole life: the length-D/2 complex
// FFT, the Hermitian glue, the lambda rescale, the per-group abs-max, the rounding
// and the nibble pack all happen in that thread's registers, so the path needs no
// shuffle, no shared-memory exchange and no barrier between lanes.  (The paper's
// Metal kernel spreads a vector over a SIMD group and meets in shuffles; on this
// machine the shuffle pipe is the scarce one, registers are not.)
//
// Memory.  A warp is an independent pipeline over tiles of 32 consecutive rows.
// Each lane fetches its own row with one bulk asynchronous copy (TMA, untiled)
// into a padded shared-memory row, two tiles in flight per warp, completion
// signalled on a per-warp mbarrier.  Results are staged in a padded row and leave
// with one bulk store per lane; the few bytes of group scales go out with plain
// coalesced stores.  Rows are padded by 16 bytes so that the 128-bit shared
// accesses of a quarter warp fall in distinct banks.
//
// Larger D (P = 2).  The complex FFT is split by output parity into two
// sequential passes of half length (decimation in frequency on the forward path,
// the mirrored decimation in time on the inverse).  The first pass parks D/2
// floats in a per-warp shared-memory stash while the second runs, which halves
// the live registers of a thread.
#pragma once
#include "kvq_fft.cuh"
#include "kvq_internal.h"

namespace kvq {


// ------------------------------------------------------------------------------------------
// shared-memory geometry (per warp)
// ------------------------------------------------------------------------------------------
template <int D, int P, int BITS>
struct EncSmem {
    static constexpr int IN_STRIDE = 2 * D + 16;
    static constexpr int OUT_STRIDE = D * BITS / 8 + 16;
    static constexpr int IN_BYTES = 2 * 32 * IN_STRIDE;
    static constexpr int OUT_BYTES = 32 * OUT_STRIDE;
    static constexpr int STASH_BYTES = (P == 2) ? D * 64 : 0;
    static constexpr int LAM_BYTES = D * 4;
    static constexpr int WARP_BYTES = IN_BYTES + OUT_BYTES + STASH_BYTES + LAM_BYTES;
};

template <int D, int P, int BITS>
struct DecSmem {
    static constexpr int IN_STRIDE = D * BITS / 8 + 16;
    static constexpr int OUT_STRIDE = 2 * D + 16;
    static constexpr int IN_BYTES = 2 * 32 * IN_STRIDE;
    static constexpr int OUT_BYTES = 32 * OUT_STRIDE;
    static constexpr int STASH_BYTES = (P == 2) ? D * 64 : 0;
    static constexpr int LAM_BYTES = D * 4;
    static constexpr int WARP_BYTES = IN_BYTES + OUT_BYTES + STASH_BYTES + LAM_BYTES;
};

constexpr int kBarBytes = 128;   // room for 2 mbarriers per warp, up to 8 warps

// ------------------------------------------------------------------------------------------
// forward path of one row (Sec. 3.2 steps 1-4, fused lambda and group scales of Sec. 7.1)
//   row      this lane's D half-precision inputs in shared memory
//   lam      lambda row in shared memory (warp-shared)
//   out      this lane's D BITS / 8 output bytes in shared memory
//   stash    warp stash, float4 [D/8][32] (P == 2 only)
//   scl      this row's D/GRP fp16 scales in global memory
// BITS = 8 (Sec. 3.2 step 4): codes in [-127, 127], one two's-complement byte per value.
// ------------------------------------------------------------------------------------------
template <int D, int GRP, int BITS, int P, bool BF16>
__device__ __forceinline__ void encode_row(const uint4 *__restrict__ row, const uint32_t *__restrict__ sign_xor,
                                           const float4 *__restrict__ lam, uint4 *__restrict__ out,
                                           float4 *__restrict__ stash, uint16_t *__restrict__ scl, int lane)
{
    constexpr int H = D / 2, L = H / P, G = D / GRP, SLOTS = D / P;
    constexpr float Q = (float)((1 << (BITS - 1)) - 1);   // largest code: 7 or 127
    float amax[G];
#pragma unroll
    for (int j = 0; j < G; ++j) amax[j] = 0.0f;
    float v[SLOTS];

    static_for<P>([&](auto pp) {
        constexpr int p = decltype(pp)::value;
        cf w[L];
        // ---- load: w_m = s_{2m} x_{2m} + i s_{2m+1} x_{2m+1}; P == 2 folds the first radix-2 stage in
        static_for<L / 4>([&](auto ii) {
            constexpr int I = decltype(ii)::value;
            uint4 a = row[I];
            uint32_t aw[4] = {a.x, a.y, a.z, a.w};
            if constexpr (P == 1) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float2 f = widen2<BF16>(aw[t] ^ sign_xor[4 * I + t]);
                    w[4 * I + t] = {f.x, f.y};
                }
            } else {
                uint4 b = row[I + L / 4];
                uint32_t bw[4] = {b.x, b.y, b.z, b.w};
                static_for<4>([&](auto tt) {
                    constexpr int t = decltype(tt)::value, m = 4 * I + t;
                    float2 fa = widen2<BF16>(aw[t] ^ sign_xor[m]);
                    float2 fb = widen2<BF16>(bw[t] ^ sign_xor[m + L]);
                    if constexpr (p == 0) {
                        w[m] = {fa.x + fb.x, fa.y + fb.y};
                    } else {
                        w[m] = twiddle_mul<H, -1, m>(cf{fa.x - fb.x, fa.y - fb.y});
                    }
                });
            }
        });
        // ---- length-L complex FFT: bins P k + p
        cf W[L];
        Fft<L, -1, 1>::run(w, W);
        // ---- Eq. 2 packing, then lambda, then the running group maxima
        float z[SLOTS];
        hermitian_unpack<D, P, p>(W, z);
        static_for<D / 4>([&](auto ii) {
            constexpr int I = decltype(ii)::value;
            float4 l4 = lam[I];
            float l[4] = {l4.x, l4.y, l4.z, l4.w};
            static_for<4>([&](auto tt) {
                constexpr int c = 4 * I + decltype(tt)::value;
                if constexpr (c % P == p) {
                    float t = z[c / P] * l[c % 4];
                    z[c / P] = t;
                    amax[c / GRP] = fmaxf(amax[c / GRP], fabsf(t));
                }
            });
        });
        if constexpr (P == 2 && p == 0) {
            static_for<SLOTS / 4>([&](auto ii) {
                constexpr int I = decltype(ii)::value;
                stash[I * 32 + lane] = make_float4(z[4 * I], z[4 * I + 1], z[4 * I + 2], z[4 * I + 3]);
            });
        } else {
#pragma unroll
            for (int s = 0; s < SLOTS; ++s) v[s] = z[s];
        }
    });

    // ---- scales: sigma = fp16(absmax / Q); codes are taken against the stored value
    float rs[G];
    bool clamp[G];
    uint32_t sbits[G];
#pragma unroll
    for (int j = 0; j < G; ++j) {
        float sig = fminf(__fdiv_rn(amax[j], Q), 65504.0f);
        __half hs = __float2half_rn(sig);
        sbits[j] = (uint32_t)__half_as_ushort(hs);
        float sg = __half2float(hs);
        rs[j] = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
        clamp[j] = !(amax[j] * rs[j] < Q + 0.25f);   // saturated or subnormal scale: codes could leave [-Q, Q]
    }
    // ---- scales out (coalesced across the warp: consecutive rows are consecutive in memory)
    if constexpr ((G * 2) % 16 == 0) {
        static_for<G / 8>([&](auto ii) {
            constexpr int I = decltype(ii)::value;
            reinterpret_cast<uint4 *>(scl)[I] =
                make_uint4(sbits[8 * I] | (sbits[8 * I + 1] << 16), sbits[8 * I + 2] | (sbits[8 * I + 3] << 16),
                           sbits[8 * I + 4] | (sbits[8 * I + 5] << 16), sbits[8 * I + 6] | (sbits[8 * I + 7] << 16));
        });
    } else if constexpr ((G * 2) % 8 == 0) {
        static_for<G / 4>([&](auto ii) {
            constexpr int I = decltype(ii)::value;
            reinterpret_cast<uint2 *>(scl)[I] =
                make_uint2(sbits[4 * I] | (sbits[4 * I + 1] << 16), sbits[4 * I + 2] | (sbits[4 * I + 3] << 16));
        });
    } else if constexpr ((G * 2) % 4 == 0) {
        static_for<G / 2>([&](auto ii) {
            constexpr int I = decltype(ii)::value;
            reinterpret_cast<uint32_t *>(scl)[I] = sbits[2 * I] | (sbits[2 * I + 1] << 16);
        });
    } else {
#pragma unroll
        for (int j = 0; j < G; ++j) scl[j] = (uint16_t)sbits[j];
    }

    // ---- round, bias to unsigned codes, pack: 32 codes per step are one 16-byte store of nibbles or two of bytes
    static_for<D / 32>([&](auto ii) {
        constexpr int I = decltype(ii)::value;
        uint32_t words[BITS];
        static_for<4>([&](auto ww) {
            constexpr int wi = 4 * I + decltype(ww)::value;   // octet index: codes 8 wi .. 8 wi + 7
            constexpr int j = (8 * wi) / GRP;
            float t[8];
            if constexpr (P == 1) {
#pragma unroll
                for (int e = 0; e < 8; ++e) t[e] = v[8 * wi + e];
            } else {
                float4 s4 = stash[wi * 32 + lane];   // even coordinates 8wi, 8wi+2, .. (first pass)
                t[0] = s4.x, t[2] = s4.y, t[4] = s4.z, t[6] = s4.w;
                t[1] = v[4 * wi], t[3] = v[4 * wi + 1], t[5] = v[4 * wi + 2], t[7] = v[4 * wi + 3];
            }
            if constexpr (BITS == 4) {
                uint32_t acc = 0;
                if (!clamp[j]) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc += __float_as_uint(fmaf(t[e], rs[j], kMagicRound)) << (4 * e);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        acc += __float_as_uint(fminf(fmaxf(t[e] * rs[j], -Q), Q) + kMagicRound) << (4 * e);
                }
                words[decltype(ww)::value] = (acc - kMagicSum) ^ 0x88888888u;
            } else {
                uint32_t acc[2] = {0u, 0u};
                if (!clamp[j]) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e >> 2] += __float_as_uint(fmaf(t[e], rs[j], kMagicRound8)) << (8 * (e & 3));
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        acc[e >> 2] += __float_as_uint(fminf(fmaxf(t[e] * rs[j], -Q), Q) + kMagicRound8) << (8 * (e & 3));
                }
                words[2 * decltype(ww)::value] = (acc[0] - kMagicSum8) ^ 0x80808080u;
                words[2 * decltype(ww)::value + 1] = (acc[1] - kMagicSum8) ^ 0x80808080u;
            }
        });
        if constexpr (BITS == 4) {
            out[I] = make_uint4(words[0], words[1], words[2], words[3]);
        } else {
            out[2 * I] = make_uint4(words[0], words[1], words[2], words[3]);
            out[2 * I + 1] = make_uint4(words[4], words[5], words[6], words[7]);
        }
    });
}

// ------------------------------------------------------------------------------------------
// inverse path of one row (Sec. 3.1: Eq. 2 undone, inverse real DFT, signs last; 1 / max(lambda, 1e-6) of Sec. 5.1)
//   row      this lane's D BITS / 8 code bytes in shared memory
//   sig      this row's D/GRP scales, already widened
//   rl       1 / max(lambda, 1e-6) in shared memory (warp-shared)
//   out      this lane's D half-precision outputs in shared memory
//   stash    warp stash, float4 [D/8][32] (P == 2 only)
// ------------------------------------------------------------------------------------------
template <int D, int GRP, int BITS, int P, bool BF16>
__device__ __forceinline__ void decode_row(const uint4 *__restrict__ row, const float *__restrict__ sig,
                                           const uint32_t *__restrict__ sign_xor, const float4 *__restrict__ rl,
                                           uint4 *__restrict__ out, float4 *__restrict__ stash, int lane)
{
    constexpr int H = D / 2, L = H / P, SLOTS = D / P;
    constexpr int CPW = 32 / BITS;                                       // codes per 32-bit word
    constexpr uint32_t kBias = BITS == 4 ? 0x88888888u : 0x80808080u;    // two's complement -> q + 8 / q + 128
    constexpr float kUnbias = BITS == 4 ? 8388616.0f : 8388736.0f;       // 2^23 + 8 / 2^23 + 128
    uint32_t pk[D / CPW];
    static_for<D / CPW / 4>([&](auto ii) {
        constexpr int I = decltype(ii)::value;
        uint4 a = row[I];
        pk[4 * I] = a.x ^ kBias, pk[4 * I + 1] = a.y ^ kBias;
        pk[4 * I + 2] = a.z ^ kBias, pk[4 * I + 3] = a.w ^ kBias;
    });

    static_for<P>([&](auto pp) {
        constexpr int p = decltype(pp)::value;
        // ---- nibble -> float -> times sigma / lambda
        float z[SLOTS];
        static_for<D / 4>([&](auto ii) {
            constexpr int I = decltype(ii)::value;
            float4 r4 = rl[I];
            float r[4] = {r4.x, r4.y, r4.z, r4.w};
            static_for<4>([&](auto tt) {
                constexpr int c = 4 * I + decltype(tt)::value;
                if constexpr (c % P == p) {
                    uint32_t n = (pk[c / CPW] >> (BITS * (c % CPW))) & ((1u << BITS) - 1u);   // q + 8 or q + 128
                    float f = __uint_as_float(0x4B000000u | n) - kUnbias;                     // q, exactly
                    z[c / P] = f * (sig[c / GRP] * r[c % 4]);
                }
            });
        });
        // ---- undo Eq. 2, inverse complex FFT
        cf W[L], w[L];
        hermitian_repack<D, P, p>(z, W);
        Fft<L, +1, 1>::run(W, w);
        // ---- to half precision, sign diagonal, staged store
        if constexpr (P == 1) {
            static_for<L / 4>([&](auto ii) {
                constexpr int I = decltype(ii)::value;
                uint32_t o[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) o[t] = narrow2<BF16>(w[4 * I + t].r, w[4 * I + t].i) ^ sign_xor[4 * I + t];
                out[I] = make_uint4(o[0], o[1], o[2], o[3]);
            });
        } else if constexpr (p == 0) {
            static_for<L / 2>([&](auto ii) {
                constexpr int I = decltype(ii)::value;
                stash[I * 32 + lane] = make_float4(w[2 * I].r, w[2 * I].i, w[2 * I + 1].r, w[2 * I + 1].i);
            });
        } else {
            static_for<L / 4>([&](auto ii) {
                constexpr int I = decltype(ii)::value;
                uint32_t lo[4], hi[4];
                static_for<2>([&](auto hh) {
                    constexpr int h = decltype(hh)::value;
                    float4 a4 = stash[(2 * I + h) * 32 + lane];
                    cf a[2] = {{a4.x, a4.y}, {a4.z, a4.w}};
                    static_for<2>([&](auto tt) {
                        constexpr int t = decltype(tt)::value, m = 4 * I + 2 * h + t;
                        cf b = twiddle_mul<H, +1, m>(w[m]);
                        lo[2 * h + t] = narrow2<BF16>(a[t].r + b.r, a[t].i + b.i) ^ sign_xor[m];
                        hi[2 * h + t] = narrow2<BF16>(a[t].r - b.r, a[t].i - b.i) ^ sign_xor[m + L];
                    });
                });
                out[I] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                out[I + L / 4] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            });
        }
    });
}

// ------------------------------------------------------------------------------------------
// kernels
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t lambda_row_of(int64_t r, int64_t n_lambda, int64_t rows_per_lambda)
{
    return n_lambda == 1 ? 0 : r / rows_per_lambda;
}

// Fills the warp's lambda cache with row `lr` of the table: the values themselves (RECIP ==
// false) or 1 / max(value, 1e-6) (RECIP == true).
template <int D, bool RECIP>
__device__ __forceinline__ void fill_lambda(float *cache, const float *__restrict__ lam, int64_t lr, int lane)
{
#pragma unroll
    for (int c = lane; c < D; c += 32) {
        float l = __ldg(lam + lr * D + c);
        cache[c] = RECIP ? __frcp_rn(fmaxf(l, 1e-6f)) : l;
    }
}

template <int D, int GRP, int BITS, int P, bool BF16, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) kvq_encode_fft_kernel(const __grid_constant__ FftParams prm)
{
    using S = EncSmem<D, P, BITS>;
    constexpr int kRowBytes = D * BITS / 8;
    extern __shared__ __align__(128) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char *wb = smem + kBarBytes + (size_t)warp * S::WARP_BYTES;
    unsigned char *in_base = wb;
    unsigned char *out_row = wb + S::IN_BYTES + lane * S::OUT_STRIDE;
    float4 *stash = reinterpret_cast<float4 *>(wb + S::IN_BYTES + S::OUT_BYTES);
    float *lam_cache = reinterpret_cast<float *>(wb + S::IN_BYTES + S::OUT_BYTES + S::STASH_BYTES);
    const uint32_t bar0 = smem_u32(smem + warp * 16), bar1 = bar0 + 8;

    if (lane == 0) {
        mbar_init(bar0, 32);
        mbar_init(bar1, 32);
        mbar_init_fence();
    }
    fence_proxy_async();
    __syncwarp();

    const int64_t N = prm.N;
    const int64_t n_tiles = (N + 31) >> 5;
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    int64_t tile = (int64_t)blockIdx.x * WARPS + warp;
    const unsigned char *x = static_cast<const unsigned char *>(prm.in);

    auto issue = [&](int64_t t, int stage) {
        const int64_t r = t * 32 + lane;
        const uint32_t bar = stage ? bar1 : bar0;
        if (r < N) {
            mbar_arrive_expect_tx(bar, 2 * D);
            bulk_load(smem_u32(in_base + (stage * 32 + lane) * S::IN_STRIDE), x + r * (2 * D), 2 * D, bar);
        } else {
            mbar_arrive(bar);
        }
    };

    if (tile < n_tiles) issue(tile, 0);
    uint32_t phases = 0;
    int64_t cached_lr = -1;
    int stage = 0;
    for (; tile < n_tiles; tile += stride, stage ^= 1) {
        if (tile + stride < n_tiles) issue(tile + stride, stage ^ 1);
        const bool ok = mbar_wait_bounded(stage ? bar1 : bar0, (phases >> stage) & 1u);
        if (!__all_sync(0xFFFFFFFFu, ok)) {
            if (lane == 0) atomicOr(prm.status, KVQ_DEV_LOAD_TIMEOUT);
            // give this warp's own copies in flight a last bounded chance to land before leaving
            (void)mbar_wait_bounded(stage ? bar1 : bar0, (phases >> stage) & 1u, 1u << 16);
            if (tile + stride < n_tiles) (void)mbar_wait_bounded(stage ? bar0 : bar1, (phases >> (stage ^ 1)) & 1u, 1u << 16);
            break;
        }
        phases ^= 1u << stage;

        const int64_t r = tile * 32 + lane;
        const bool active = r < N;
        const int64_t lr = active ? lambda_row_of(r, prm.n_lambda, prm.rows_per_lambda) : -1;
        bulk_wait_read_all();   // the previous tile's bulk store has drained this lane's staging row
        unsigned todo = __ballot_sync(0xFFFFFFFFu, active);
        while (todo) {
            const int leader = __ffs(todo) - 1;
            const int64_t cur = __shfl_sync(0xFFFFFFFFu, lr, leader);
            const unsigned mine = __ballot_sync(0xFFFFFFFFu, active && lr == cur);
            if (cur != cached_lr) {
                __syncwarp();
                fill_lambda<D, false>(lam_cache, prm.lambda, cur, lane);
                cached_lr = cur;
                __syncwarp();
            }
            if (active && lr == cur) {
                const int64_t orow = prm.out_map(r);
                encode_row<D, GRP, BITS, P, BF16>(
                    reinterpret_cast<const uint4 *>(in_base + (stage * 32 + lane) * S::IN_STRIDE), prm.sign_xor,
                    reinterpret_cast<const float4 *>(lam_cache), reinterpret_cast<uint4 *>(out_row), stash,
                    static_cast<uint16_t *>(prm.scales) + orow * (D / GRP), lane);
                fence_proxy_async();
                bulk_store(static_cast<unsigned char *>(prm.packed) + orow * kRowBytes, smem_u32(out_row), kRowBytes);
                bulk_commit();
            }
            todo &= ~mine;
        }
    }
    bulk_wait_all();
}

template <int D, int GRP, int BITS, int P, bool BF16, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) kvq_decode_fft_kernel(const __grid_constant__ FftParams prm)
{
    using S = DecSmem<D, P, BITS>;
    constexpr int G = D / GRP;
    constexpr int kRowBytes = D * BITS / 8;
    extern __shared__ __align__(128) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char *wb = smem + kBarBytes + (size_t)warp * S::WARP_BYTES;
    unsigned char *in_base = wb;
    unsigned char *out_row = wb + S::IN_BYTES + lane * S::OUT_STRIDE;
    float4 *stash = reinterpret_cast<float4 *>(wb + S::IN_BYTES + S::OUT_BYTES);
    float *lam_cache = reinterpret_cast<float *>(wb + S::IN_BYTES + S::OUT_BYTES + S::STASH_BYTES);
    const uint32_t bar0 = smem_u32(smem + warp * 16), bar1 = bar0 + 8;

    if (lane == 0) {
        mbar_init(bar0, 32);
        mbar_init(bar1, 32);
        mbar_init_fence();
    }
    fence_proxy_async();
    __syncwarp();

    const int64_t N = prm.N;
    const int64_t n_tiles = (N + 31) >> 5;
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    int64_t tile = (int64_t)blockIdx.x * WARPS + warp;
    const unsigned char *packed = static_cast<const unsigned char *>(prm.packed);
    const uint16_t *scales = static_cast<const uint16_t *>(prm.scales);

    auto issue = [&](int64_t t, int stage) {
        const int64_t r = t * 32 + lane;
        const uint32_t bar = stage ? bar1 : bar0;
        if (r < N) {
            mbar_arrive_expect_tx(bar, kRowBytes);
            bulk_load(smem_u32(in_base + (stage * 32 + lane) * S::IN_STRIDE), packed + prm.in_map(r) * kRowBytes, kRowBytes, bar);
        } else {
            mbar_arrive(bar);
        }
    };
    // the row's group scales travel in registers, fetched one tile ahead
    auto load_scales = [&](int64_t t, uint32_t (&sb)[(G + 1) / 2]) {
        const int64_t r = t * 32 + lane;
#pragma unroll
        for (int j = 0; j < (G + 1) / 2; ++j) sb[j] = 0;
        if (r < N) {
            const uint16_t *sp = scales + prm.in_map(r) * G;
            if constexpr ((G * 2) % 16 == 0) {
#pragma unroll
                for (int j = 0; j < G / 8; ++j) {
                    uint4 q = __ldg(reinterpret_cast<const uint4 *>(sp) + j);
                    sb[4 * j] = q.x, sb[4 * j + 1] = q.y, sb[4 * j + 2] = q.z, sb[4 * j + 3] = q.w;
                }
            } else if constexpr ((G * 2) % 8 == 0) {
#pragma unroll
                for (int j = 0; j < G / 4; ++j) {
                    uint2 q = __ldg(reinterpret_cast<const uint2 *>(sp) + j);
                    sb[2 * j] = q.x, sb[2 * j + 1] = q.y;
                }
            } else if constexpr ((G * 2) % 4 == 0) {
#pragma unroll
                for (int j = 0; j < G / 2; ++j) sb[j] = __ldg(reinterpret_cast<const uint32_t *>(sp) + j);
            } else {
#pragma unroll
                for (int j = 0; j < G; ++j) sb[j / 2] |= (uint32_t)__ldg(sp + j) << (16 * (j & 1));
            }
        }
    };

    uint32_t sb_next[(G + 1) / 2];
    if (tile < n_tiles) {
        issue(tile, 0);
        load_scales(tile, sb_next);
    }
    uint32_t phases = 0;
    int64_t cached_lr = -1;
    int stage = 0;
    for (; tile < n_tiles; tile += stride, stage ^= 1) {
        uint32_t sb[(G + 1) / 2];
#pragma unroll
        for (int j = 0; j < (G + 1) / 2; ++j) sb[j] = sb_next[j];
        if (tile + stride < n_tiles) {
            issue(tile + stride, stage ^ 1);
            load_scales(tile + stride, sb_next);
        }
        const bool ok = mbar_wait_bounded(stage ? bar1 : bar0, (phases >> stage) & 1u);
        if (!__all_sync(0xFFFFFFFFu, ok)) {
            if (lane == 0) atomicOr(prm.status, KVQ_DEV_LOAD_TIMEOUT);
            (void)mbar_wait_bounded(stage ? bar1 : bar0, (phases >> stage) & 1u, 1u << 16);
            if (tile + stride < n_tiles) (void)mbar_wait_bounded(stage ? bar0 : bar1, (phases >> (stage ^ 1)) & 1u, 1u << 16);
            break;
        }
        phases ^= 1u << stage;

        const int64_t r = tile * 32 + lane;
        const bool active = r < N;
        const int64_t lr = active ? lambda_row_of(r, prm.n_lambda, prm.rows_per_lambda) : -1;
        float sig[G];
#pragma unroll
        for (int j = 0; j < G; ++j)
            sig[j] = __half2float(__ushort_as_half((unsigned short)((sb[j / 2] >> (16 * (j & 1))) & 0xFFFFu)));
        bulk_wait_read_all();
        unsigned todo = __ballot_sync(0xFFFFFFFFu, active);
        while (todo) {
            const int leader = __ffs(todo) - 1;
            const int64_t cur = __shfl_sync(0xFFFFFFFFu, lr, leader);
            const unsigned mine = __ballot_sync(0xFFFFFFFFu, active && lr == cur);
            if (cur != cached_lr) {
                __syncwarp();
                fill_lambda<D, true>(lam_cache, prm.lambda, cur, lane);
                cached_lr = cur;
                __syncwarp();
            }
            if (active && lr == cur) {
                decode_row<D, GRP, BITS, P, BF16>(
                    reinterpret_cast<const uint4 *>(in_base + (stage * 32 + lane) * S::IN_STRIDE), sig, prm.sign_xor,
                    reinterpret_cast<const float4 *>(lam_cache), reinterpret_cast<uint4 *>(out_row), stash, lane);
                fence_proxy_async();
                bulk_store(static_cast<unsigned char *>(prm.out) + prm.out_map(r) * (2 * D), smem_u32(out_row), 2 * D);
                bulk_commit();
            }
            todo &= ~mine;
        }
    }
    bulk_wait_all();
}

// ------------------------------------------------------------------------------------------
// host side: per-instantiation launch with cached occupancy
// ------------------------------------------------------------------------------------------
template <typename Kern>
static cudaError_t launch_persistent(Kern kern, int warps, size_t smem, int64_t N, const FftParams &prm,
                                     cudaStream_t stream, DeviceSlots *slots)
{
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int *cached_blocks_per_sm = &slots->blocks_per_sm[dev], *cached_sms = &slots->sms[dev];
    if (*cached_blocks_per_sm == 0) {
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        int nb = 0, sms = 0;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, warps * 32, smem)) != cudaSuccess) return e;
        if (nb < 1) return cudaErrorLaunchOutOfResources;
        *cached_blocks_per_sm = nb;
        *cached_sms = sms;
    }
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    const int64_t tiles = (N + 31) / 32;
    const int64_t want = (tiles + warps - 1) / warps;
    const int64_t cap = (int64_t)(*cached_blocks_per_sm) * (*cached_sms);
    const int grid = (int)(want < cap ? want : cap);
    kern<<<grid, warps * 32, smem, stream>>>(prm);
    count_launch();
    return cudaGetLastError();
}

// GRP == 0 stands for one group over the whole vector (GRP = D).
template <int D, int GRP, int BITS, int P, bool BF16, int WARPS>
static cudaError_t launch_encode(int64_t N, const FftParams &prm, cudaStream_t stream)
{
    static DeviceSlots slots;
    constexpr int kGrp = GRP ? GRP : D;
    constexpr size_t smem = kBarBytes + (size_t)WARPS * EncSmem<D, P, BITS>::WARP_BYTES;
    static_assert(smem <= 232448, "encode kernel: shared memory over the per-CTA limit");
    return launch_persistent(kvq_encode_fft_kernel<D, kGrp, BITS, P, BF16, WARPS>, WARPS, smem, N, prm, stream, &slots);
}

template <int D, int GRP, int BITS, int P, bool BF16, int WARPS>
static cudaError_t launch_decode(int64_t N, const FftParams &prm, cudaStream_t stream)
{
    static DeviceSlots slots;
    constexpr int kGrp = GRP ? GRP : D;
    constexpr size_t smem = kBarBytes + (size_t)WARPS * DecSmem<D, P, BITS>::WARP_BYTES;
    static_assert(smem <= 232448, "decode kernel: shared memory over the per-CTA limit");
    return launch_persistent(kvq_decode_fft_kernel<D, kGrp, BITS, P, BF16, WARPS>, WARPS, smem, N, prm, stream, &slots);
}

// Defines kvq::ENC and kvq::DEC, the per-D dispatchers of one (GRP, BITS) variant.  Four warps per CTA, three for
// the D = 256 encode with byte codes (its staging rows would not fit otherwise).
#define KVQ_FFT_CASE(FN, GRP, BITS, DD, PP, WW)                                                               \
    case DD:                                                                                                  \
        return bf16 ? FN<DD, GRP, BITS, PP, true, WW>(N, prm, stream) : FN<DD, GRP, BITS, PP, false, WW>(N, prm, stream);

#define KVQ_FFT_DEFINE_VARIANT(ENC, DEC, GRP, BITS)                                                           \
    namespace kvq {                                                                                           \
    cudaError_t ENC(int D, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream)                   \
    {                                                                                                         \
        switch (D) {                                                                                          \
            KVQ_FFT_CASE(launch_encode, GRP, BITS, 64, 1, 4)                                                  \
            KVQ_FFT_CASE(launch_encode, GRP, BITS, 96, 1, 4)                                                  \
            KVQ_FFT_CASE(launch_encode, GRP, BITS, 128, 1, 4)                                                 \
            KVQ_FFT_CASE(launch_encode, GRP, BITS, 160, 2, 4)                                                 \
            KVQ_FFT_CASE(launch_encode, GRP, BITS, 256, 2, (BITS == 8 ? 3 : 4))                               \
        }                                                                                                     \
        return cudaErrorInvalidValue;                                                                         \
    }                                                                                                         \
    cudaError_t DEC(int D, bool bf16, int64_t N, const FftParams &prm, cudaStream_t stream)                   \
    {                                                                                                         \
        switch (D) {                                                                                          \
            KVQ_FFT_CASE(launch_decode, GRP, BITS, 64, 1, 4)                                                  \
            KVQ_FFT_CASE(launch_decode, GRP, BITS, 96, 1, 4)                                                  \
            KVQ_FFT_CASE(launch_decode, GRP, BITS, 128, 1, 4)                                                 \
            KVQ_FFT_CASE(launch_decode, GRP, BITS, 160, 2, 4)                                                 \
            KVQ_FFT_CASE(launch_decode, GRP, BITS, 256, 2, 4)                                                 \
        }                                                                                                     \
        return cudaErrorInvalidValue;                                                                         \
    }                                                                                                         \
    }

}  // namespace kvq
