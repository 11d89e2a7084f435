// Register-resident mixed-radix complex FFT and the real-transform glue around it.
//
// One thread owns one whole vector.  All indices are compile-time constants, so
// the local arrays below live in registers, the index permutations of the
// Cooley-Tukey recursion cost nothing, and every twiddle factor is an immediate
// (Sec. 3.2 step 2 runs radix-2 passes from a table; at these lengths radix 4
// with immediates needs fewer instructions and no table at all).
//
//   real length-D transform  =  complex length-H FFT (H = D/2) on w_m = u_{2m} + i u_{2m+1}
//                               + Hermitian unpack (forward) / repack (inverse).
//
// For the larger D the complex FFT is split once more by output parity into
// P = 2 sequential passes of length L = H/2 (decimation in frequency), which
// halves the number of live registers; see kvq_fft_kernels.cuh.
#pragma once

#include "kvq_device.cuh"

namespace kvq {

struct cf {
    float r, i;
};

__device__ __forceinline__ cf operator+(cf a, cf b) { return {a.r + b.r, a.i + b.i}; }
__device__ __forceinline__ cf operator-(cf a, cf b) { return {a.r - b.r, a.i - b.i}; }

// multiply by i^SIGN, i.e. by e^{SIGN i pi/2}
template <int SIGN>
__device__ __forceinline__ cf mul_i(cf a)
{
    if constexpr (SIGN > 0) return {-a.i, a.r};
    else return {a.i, -a.r};
}

// a * e^{SIGN 2 pi i M / N}, the angle known at compile time
template <int N, int SIGN, int M>
__device__ __forceinline__ cf twiddle_mul(cf a)
{
    constexpr int m = ((M % N) + N) % N;
    if constexpr (m == 0) {
        return a;
    } else if constexpr (4 * m == N) {
        return mul_i<SIGN>(a);
    } else if constexpr (2 * m == N) {
        return {-a.r, -a.i};
    } else if constexpr (4 * m == 3 * N) {
        return mul_i<-SIGN>(a);
    } else {
        constexpr float c = (float)ct_cos2pi(m, N);
        constexpr float s = (float)((double)SIGN * ct_sin2pi(m, N));
        return {fmaf(-s, a.i, c * a.r), fmaf(s, a.r, c * a.i)};
    }
}

constexpr int radix_of(int n) { return n % 4 == 0 ? 4 : n % 2 == 0 ? 2 : n % 3 == 0 ? 3 : n % 5 == 0 ? 5 : n; }

// In-place DFT of R points: t[q] <- sum_j t[j] e^{SIGN 2 pi i j q / R}
template <int R, int SIGN>
__device__ __forceinline__ void butterfly(cf *t)
{
    static_assert(R == 2 || R == 3 || R == 4 || R == 5, "radix not implemented");
    if constexpr (R == 2) {
        cf a = t[0], b = t[1];
        t[0] = a + b;
        t[1] = a - b;
    } else if constexpr (R == 4) {
        cf s02 = t[0] + t[2], d02 = t[0] - t[2];
        cf s13 = t[1] + t[3], d13 = mul_i<SIGN>(t[1] - t[3]);
        t[0] = s02 + s13;
        t[2] = s02 - s13;
        t[1] = d02 + d13;
        t[3] = d02 - d13;
    } else if constexpr (R == 3) {
        constexpr float hs3 = (float)(0.5 * ct_sqrt(3.0));
        cf s = t[1] + t[2], d = t[1] - t[2];
        cf m = {fmaf(-0.5f, s.r, t[0].r), fmaf(-0.5f, s.i, t[0].i)};
        cf e = mul_i<SIGN>(cf{hs3 * d.r, hs3 * d.i});
        t[0] = t[0] + s;
        t[1] = m + e;
        t[2] = m - e;
    } else {
        constexpr float c1 = (float)ct_cos2pi(1, 5), c2 = (float)ct_cos2pi(2, 5);
        constexpr float n1 = (float)ct_sin2pi(1, 5), n2 = (float)ct_sin2pi(2, 5);
        cf s1 = t[1] + t[4], s2 = t[2] + t[3], d1 = t[1] - t[4], d2 = t[2] - t[3];
        cf a1 = {fmaf(c2, s2.r, fmaf(c1, s1.r, t[0].r)), fmaf(c2, s2.i, fmaf(c1, s1.i, t[0].i))};
        cf a2 = {fmaf(c1, s2.r, fmaf(c2, s1.r, t[0].r)), fmaf(c1, s2.i, fmaf(c2, s1.i, t[0].i))};
        cf b1 = mul_i<SIGN>(cf{fmaf(n2, d2.r, n1 * d1.r), fmaf(n2, d2.i, n1 * d1.i)});
        cf b2 = mul_i<SIGN>(cf{fmaf(-n1, d2.r, n2 * d1.r), fmaf(-n1, d2.i, n2 * d1.i)});
        t[0] = t[0] + s1 + s2;
        t[1] = a1 + b1;
        t[4] = a1 - b1;
        t[2] = a2 + b2;
        t[3] = a2 - b2;
    }
}

// out[k] = sum_n in[n * IS] e^{SIGN 2 pi i k n / N}, k = 0..N-1 (unnormalised), by
// decimation in time: N = R * M, R sub-transforms of length M on the residues mod R,
// twiddle, then M radix-R butterflies.
template <int N, int SIGN, int IS>
struct Fft {
    static constexpr int R = radix_of(N), M = N / R;
    __device__ __forceinline__ static void run(const cf *in, cf *out)
    {
        cf sub[R][M];
        static_for<R>([&](auto j) { Fft<M, SIGN, IS * R>::run(in + decltype(j)::value * IS, sub[decltype(j)::value]); });
        static_for<M>([&](auto k) {
            constexpr int K = decltype(k)::value;
            cf t[R];
            static_for<R>([&](auto j) {
                constexpr int J = decltype(j)::value;
                t[J] = twiddle_mul<N, SIGN, J * K>(sub[J][K]);
            });
            butterfly<R, SIGN>(t);
            static_for<R>([&](auto q) { out[K + decltype(q)::value * M] = t[decltype(q)::value]; });
        });
    }
};

template <int SIGN, int IS>
struct Fft<1, SIGN, IS> {
    __device__ __forceinline__ static void run(const cf *in, cf *out) { out[0] = in[0]; }
};

// ---------------------------------------------------------------------------
// Forward glue (Eq. 1-2).  W[k], k < L, holds bin kk = P k + p of the unnormalised
// length-H FFT of w.  Writes the packed real coefficients z_c of parity p to
// z[c / P]: z_0 = Re Y_0, z_H = Re Y_H, z_k = sqrt2 Re Y_k, z_{H+k} = sqrt2 Im Y_k,
// with Y the unitary length-D DFT.
// ---------------------------------------------------------------------------
template <int D, int P, int p>
__device__ __forceinline__ void hermitian_unpack(const cf *W, float *z)
{
    constexpr int H = D / 2, L = H / P;
    constexpr float rsD = (float)(1.0 / ct_sqrt((double)D));
    constexpr float f = (float)(ct_sqrt(2.0) / (2.0 * ct_sqrt((double)D)));
    static_for<L>([&](auto k) {
        constexpr int K = decltype(k)::value, kk = P * K + p;
        if constexpr (kk == 0) {
            z[0] = (W[K].r + W[K].i) * rsD;
            z[H / P] = (W[K].r - W[K].i) * rsD;
        } else if constexpr (2 * kk == H) {
            z[kk / P] = (2.0f * f) * W[K].r;
            z[(H + kk) / P] = (-2.0f * f) * W[K].i;
        } else if constexpr (2 * kk < H) {
            constexpr int KP = (H - kk - p) / P;  // local index of bin H - kk
            constexpr float c = (float)((double)f * ct_cos2pi(kk, D)), s = (float)((double)f * ct_sin2pi(kk, D));
            float Sr = W[K].r + W[KP].r, Di = W[K].i - W[KP].i;
            float Si = W[K].i + W[KP].i, Dr = W[K].r - W[KP].r;
            float Pr = fmaf(-s, Dr, c * Si);
            float Pi = -fmaf(s, Si, c * Dr);
            z[kk / P] = fmaf(f, Sr, Pr);
            z[(H + kk) / P] = fmaf(f, Di, Pi);
            z[(H - kk) / P] = fmaf(f, Sr, -Pr);
            z[(2 * H - kk) / P] = fmaf(-f, Di, Pi);
        }
    });
}

// Inverse glue: from the packed coefficients of parity p (z[c / P]) build the bins
// W[k] = bin P k + p that the unnormalised inverse length-H FFT turns into
// w_m = u_{2m} + i u_{2m+1}, u the unitary inverse real DFT.
template <int D, int P, int p>
__device__ __forceinline__ void hermitian_repack(const float *z, cf *W)
{
    constexpr int H = D / 2, L = H / P;
    constexpr float rsD = (float)(1.0 / ct_sqrt((double)D));
    constexpr float f = (float)(ct_sqrt(2.0) / (2.0 * ct_sqrt((double)D)));
    static_for<L>([&](auto k) {
        constexpr int K = decltype(k)::value, kk = P * K + p;
        if constexpr (kk == 0) {
            float z0 = z[0], zH = z[H / P];
            W[K] = {(z0 + zH) * rsD, (z0 - zH) * rsD};
        } else if constexpr (2 * kk == H) {
            W[K] = {(2.0f * f) * z[kk / P], (-2.0f * f) * z[(H + kk) / P]};
        } else if constexpr (2 * kk < H) {
            constexpr int KP = (H - kk - p) / P;
            constexpr float c = (float)((double)f * ct_cos2pi(kk, D)), s = (float)((double)f * ct_sin2pi(kk, D));
            float a = z[kk / P], b = z[(H + kk) / P], cc = z[(H - kk) / P], d = z[(2 * H - kk) / P];
            float Sr = a + cc, Si = b - d, Dr = a - cc, Di = b + d;
            float Pr = fmaf(-s, Di, c * Dr);
            float Pi = fmaf(s, Dr, c * Di);
            W[K] = {fmaf(f, Sr, -Pi), fmaf(f, Si, Pr)};
            W[KP] = {fmaf(f, Sr, Pi), fmaf(-f, Si, Pr)};
        }
    });
}

}  // namespace kvq
