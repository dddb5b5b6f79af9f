// k-dominant frequency hashing (Algorithm 1), batch-mean scope, for the lookback lengths the paper's
// workloads use: a register-blocked two-pass FFT with every index and twiddle fixed at compile time.
//
// Work is laid out by hash row (one variate): a team of 1, 2 or 4 warps owns a row, each warp takes a
// contiguous range of the batch.  Two real windows ride one complex transform of length L = R1 * R2
// (z = x_b + i x_{b+1};  X_b[f] = (Z_f + conj Z_{L-f}) / 2,  X_{b+1}[f] = (Z_f - conj Z_{L-f}) / 2i):
//   pass 1   R2 lanes per transform: lane j2 loads z[j1 R2 + j2] straight from global memory, runs an
//            R1-point DFT in registers, multiplies output k1 by exp(-2 pi i j2 k1 / L) and parks it in the
//            warp's exchange buffer,
//   pass 2   R1 lanes per transform: lane k1 reads its R2 values, runs an R2-point DFT in registers; output
//            k2 is Z[k1 + R1 k2]; only the candidate band and its mirror image are kept,
//   then     lane fi adds the amplitudes of bin f_lo + fi of the warp's windows in ascending instance order.
// Warps never wait for each other inside a row (only __syncwarp); the team's partial sums are added in
// ascending order by its first warp, which ranks the top k bins and packs the hash value.
#include "common.cuh"
#include "kernels.h"

namespace vardrop {

namespace {

// ---- compile-time trigonometry ------------------------------------------------------------------------------
namespace ct {
constexpr double kPi = 3.14159265358979323846264338327950288;
constexpr double sin_small(double x) {          // |x| <= pi / 4
    const double x2 = x * x;
    double term = x, sum = x;
    for (int i = 1; i <= 12; ++i) {
        term *= -x2 / static_cast<double>((2 * i) * (2 * i + 1));
        sum += term;
    }
    return sum;
}
constexpr double cos_small(double x) {
    const double x2 = x * x;
    double term = 1.0, sum = 1.0;
    for (int i = 1; i <= 12; ++i) {
        term *= -x2 / static_cast<double>((2 * i - 1) * (2 * i));
        sum += term;
    }
    return sum;
}
// cos and sin of 2 pi num / den for 0 <= num < den, reduced to the first half-quadrant with integers
constexpr double cos_turn(long long num, long long den);
constexpr double sin_turn(long long num, long long den) {
    if (2 * num > den) return -sin_turn(den - num, den);            // sin(2 pi - a) = -sin a
    if (4 * num > den) return sin_turn(den - 2 * num, 2 * den);     // sin(pi - a) = sin a ; (den/2 - num)/den = (den - 2 num)/(2 den)
    if (8 * num > den) return cos_turn(den - 4 * num, 4 * den);     // sin a = cos(pi/2 - a)
    return sin_small(2.0 * kPi * static_cast<double>(num) / static_cast<double>(den));
}
constexpr double cos_turn(long long num, long long den) {
    if (2 * num > den) return cos_turn(den - num, den);
    if (4 * num > den) return -cos_turn(den - 2 * num, 2 * den);
    if (8 * num > den) return sin_turn(den - 4 * num, 4 * den);
    return cos_small(2.0 * kPi * static_cast<double>(num) / static_cast<double>(den));
}
}  // namespace ct

template <int NUM, int DEN>
struct Turn {                                   // cos and sin of 2 pi NUM / DEN as float constants
    static constexpr float c = static_cast<float>(ct::cos_turn(NUM, DEN));
    static constexpr float s = static_cast<float>(ct::sin_turn(NUM, DEN));
};

template <int I>
struct Int {
    static constexpr int value = I;
};
template <int B, int E, class F>
__device__ __forceinline__ void static_for(F&& f) {
    if constexpr (B < E) {
        f(Int<B>{});
        static_for<B + 1, E>(f);
    }
}

__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }

// v * exp(-2 pi i NUM / DEN)
template <int NUM, int DEN>
__device__ __forceinline__ float2 rotate(float2 v) {
    constexpr int n = ((NUM % DEN) + DEN) % DEN;
    if constexpr (n == 0) return v;
    else if constexpr (4 * n == DEN) return make_float2(v.y, -v.x);
    else if constexpr (2 * n == DEN) return make_float2(-v.x, -v.y);
    else if constexpr (4 * n == 3 * DEN) return make_float2(-v.y, v.x);
    else {
        constexpr float c = Turn<n, DEN>::c, s = Turn<n, DEN>::s;
        return make_float2(fmaf(v.y, s, v.x * c), fmaf(-v.x, s, v.y * c));
    }
}

// ---- prime-size butterflies: y_m = sum_j v_j exp(-2 pi i j m / R), in place --------------------------------
template <int R>
__device__ __forceinline__ void butterfly(float2* v);

template <>
__device__ __forceinline__ void butterfly<2>(float2* v) {
    const float2 a = v[0], b = v[1];
    v[0] = cadd(a, b);
    v[1] = csub(a, b);
}
template <>
__device__ __forceinline__ void butterfly<4>(float2* v) {
    const float2 s02 = cadd(v[0], v[2]), d02 = csub(v[0], v[2]);
    const float2 s13 = cadd(v[1], v[3]), d13 = csub(v[1], v[3]);
    v[0] = cadd(s02, s13);
    v[2] = csub(s02, s13);
    v[1] = make_float2(d02.x + d13.y, d02.y - d13.x);
    v[3] = make_float2(d02.x - d13.y, d02.y + d13.x);
}
// odd prime: pair j with R - j;  y_m = a_m - i b_m,  y_{R-m} = a_m + i b_m  with
// a_m = v_0 + sum_j cos(2 pi j m / R) (v_j + v_{R-j}),  b_m = sum_j sin(2 pi j m / R) (v_j - v_{R-j})
template <int R>
__device__ __forceinline__ void odd_butterfly(float2* v) {
    constexpr int Hh = (R - 1) / 2;
    float2 p[Hh], m[Hh];
    static_for<0, Hh>([&](auto J) {
        constexpr int j = decltype(J)::value;
        p[j] = cadd(v[j + 1], v[R - 1 - j]);
        m[j] = csub(v[j + 1], v[R - 1 - j]);
    });
    float2 out[R];
    out[0] = v[0];
    static_for<0, Hh>([&](auto J) { out[0] = cadd(out[0], p[decltype(J)::value]); });
    static_for<1, Hh + 1>([&](auto M) {
        constexpr int mm = decltype(M)::value;
        float2 a = v[0], b = make_float2(0.f, 0.f);
        static_for<1, Hh + 1>([&](auto J) {
            constexpr int j = decltype(J)::value;
            constexpr int idx = (j * mm) % R;
            constexpr float c = Turn<idx, R>::c, s = Turn<idx, R>::s;
            a.x = fmaf(c, p[j - 1].x, a.x);
            a.y = fmaf(c, p[j - 1].y, a.y);
            b.x = fmaf(s, m[j - 1].x, b.x);
            b.y = fmaf(s, m[j - 1].y, b.y);
        });
        out[mm] = make_float2(a.x + b.y, a.y - b.x);
        out[R - mm] = make_float2(a.x - b.y, a.y + b.x);
    });
    static_for<0, R>([&](auto J) { v[decltype(J)::value] = out[decltype(J)::value]; });
}
template <>
__device__ __forceinline__ void butterfly<3>(float2* v) { odd_butterfly<3>(v); }
template <>
__device__ __forceinline__ void butterfly<5>(float2* v) { odd_butterfly<5>(v); }
template <>
__device__ __forceinline__ void butterfly<7>(float2* v) { odd_butterfly<7>(v); }

template <int N>
struct Radix {                                  // outermost radix of the decimation
    static constexpr int value = N % 4 == 0 ? 4 : N % 2 == 0 ? 2 : N % 3 == 0 ? 3 : N % 5 == 0 ? 5 : 7;
};

// N-point DFT of in[0], in[IS], ... to out[0], out[OS], ... (decimation in time; all indices are constants)
template <int N, int IS, int OS>
__device__ __forceinline__ void dft(const float2* in, float2* out) {
    if constexpr (N == 1) {
        out[0] = in[0];
    } else if constexpr (N == 2 || N == 3 || N == 4 || N == 5 || N == 7) {
        float2 v[N];
        static_for<0, N>([&](auto J) { v[decltype(J)::value] = in[decltype(J)::value * IS]; });
        butterfly<N>(v);
        static_for<0, N>([&](auto J) { out[decltype(J)::value * OS] = v[decltype(J)::value]; });
    } else {
        constexpr int R = Radix<N>::value, M = N / R;
        static_assert(R * M == N, "length must factor into 2, 3, 5, 7");
        float2 sub[N];                                       // sub[r M + k]: DFT of the samples congruent to r
        static_for<0, R>([&](auto Rr) {
            constexpr int r = decltype(Rr)::value;
            dft<M, IS * R, 1>(in + r * IS, sub + r * M);
        });
        static_for<0, M>([&](auto K) {
            constexpr int k = decltype(K)::value;
            float2 v[R];
            static_for<0, R>([&](auto Rr) {
                constexpr int r = decltype(Rr)::value;
                v[r] = rotate<r * k, N>(sub[r * M + k]);
            });
            butterfly<R>(v);
            static_for<0, R>([&](auto Q) {
                constexpr int q = decltype(Q)::value;
                out[(k + M * q) * OS] = v[q];
            });
        });
    }
}

// ---- the kernel ----------------------------------------------------------------------------------------------
constexpr int kRowsWarps = 4;                  // warps per CTA
constexpr int kRowsThreads = kRowsWarps * 32;

struct RowsParams {
    const float* x;
    uint64_t* keys;
    int32_t* freqs;
    float* amp_dbg;
    int* status;
    int B, N, k, f_lo, nf;
    int team;             // warps per row: 1, 2 or 4
    int per_member;       // windows of a row per team member (even)
};

template <int L, int R1, int R2, int PC>
struct RowsPlan {
    static_assert(R1 * R2 == L, "L = R1 * R2");
    static constexpr int P2 = R2 | 1;                                       // exchange row pitch (complex), odd: pass-2 reads are conflict-free
    static constexpr int PS = R1 * P2 + ((R2 - R1 * P2) % 16 + 16) % 16;    // pitch between transforms: consecutive lanes keep consecutive banks
    static constexpr int NACC = (L / 2 + 1 + 31) / 32;                      // accumulators per lane (bins lane, lane + 32, ...)
    static constexpr int exch_elems = PC * PS;
    static size_t smem_bytes(int nf) {
        return sizeof(float2) * (static_cast<size_t>(L) + kRowsWarps * (exch_elems + static_cast<size_t>(PC) * 2 * nf)) +
               sizeof(float) * kRowsWarps * NACC * 32;
    }
};

template <int L, int R1, int R2, int PC, int MINB>
__global__ void __launch_bounds__(kRowsThreads, MINB) hash_rows_kernel(const RowsParams P) {
    using Plan = RowsPlan<L, R1, R2, PC>;
    constexpr int P2 = Plan::P2, PS = Plan::PS, NACC = Plan::NACC;
    extern __shared__ __align__(16) unsigned char smem_rows[];
    const int nf = P.nf, f_lo = P.f_lo, f_hi = P.f_lo + P.nf;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float2* tw = reinterpret_cast<float2*>(smem_rows);                       // tw[k1 R2 + j2] = exp(-2 pi i j2 k1 / L)
    float* part = reinterpret_cast<float*>(tw + L);                          // [warps][NACC * 32] partial sums of the team
    float2* exch = reinterpret_cast<float2*>(part + kRowsWarps * NACC * 32) + static_cast<size_t>(warp) * (Plan::exch_elems + PC * 2 * nf);
    float2* band = exch + Plan::exch_elems;                                  // [PC][2 nf]: Z_f for the band, then Z_{L-f}

    for (int m = threadIdx.x; m < L; m += kRowsThreads) {
        const int k1 = m / R2, j2 = m - k1 * R2;
        int e = (j2 * k1) % L;
        if (2 * e > L) e -= L;                                               // angle folded to |e| <= L / 2
        float s, c;
        sincospif(2.f * static_cast<float>(e) / static_cast<float>(L), &s, &c);
        tw[m] = make_float2(c, -s);
    }
    __syncthreads();
    chain_wait();
    chain_release();

    const int rows_per_cta = kRowsWarps / P.team;
    const int member = warp % P.team;
    const float inv_n = 1.f / static_cast<float>(P.B);

    for (int row_base = blockIdx.x * rows_per_cta; row_base < P.N; row_base += gridDim.x * rows_per_cta) {
        const int row = row_base + warp / P.team;
        const bool active = row < P.N;
        float acc[NACC];
#pragma unroll
        for (int i = 0; i < NACC; ++i) acc[i] = 0.f;

        const int b_lo = member * P.per_member;
        const int b_hi = active ? min(P.B, b_lo + P.per_member) : 0;
        for (int c0 = b_lo; c0 < b_hi; c0 += 2 * PC) {
            const int n_win = min(2 * PC, b_hi - c0);
            const int n_pair = (n_win + 1) >> 1;
            // ---- pass 1 ---------------------------------------------------------------------------------------
            for (int t = lane; t < n_pair * R2; t += 32) {
                const int p = t / R2, j2 = t - p * R2;
                const int b1 = c0 + 2 * p;
                const float* s1 = P.x + (static_cast<size_t>(b1) * P.N + row) * L + j2;
                const bool two = b1 + 1 < b_hi;
                const float* s2 = s1 + (two ? static_cast<size_t>(P.N) * L : 0);
                float2 v[R1], y[R1];
                static_for<0, R1>([&](auto J) {
                    constexpr int j1 = decltype(J)::value;
                    v[j1].x = __ldg(s1 + j1 * R2);
                    v[j1].y = __ldg(s2 + j1 * R2);
                });
                if (!two) {
                    static_for<0, R1>([&](auto J) { v[decltype(J)::value].y = 0.f; });
                }
                dft<R1, 1, 1>(v, y);
                float2* dst = exch + p * PS + j2;
                dst[0] = y[0];
                static_for<1, R1>([&](auto K) {
                    constexpr int k1 = decltype(K)::value;
                    const float2 w = tw[k1 * R2 + j2];
                    dst[k1 * P2] = make_float2(fmaf(-y[k1].y, w.y, y[k1].x * w.x), fmaf(y[k1].x, w.y, y[k1].y * w.x));
                });
            }
            __syncwarp();
            // ---- pass 2 ---------------------------------------------------------------------------------------
            for (int t = lane; t < n_pair * R1; t += 32) {
                const int p = t / R1, k1 = t - p * R1;
                const float2* src = exch + p * PS + k1 * P2;
                float2 v[R2], y[R2];
                static_for<0, R2>([&](auto J) { v[decltype(J)::value] = src[decltype(J)::value]; });
                dft<R2, 1, 1>(v, y);
                float2* bp = band + p * 2 * nf;
                static_for<0, R2>([&](auto K) {
                    constexpr int k2 = decltype(K)::value;
                    const int g = k1 + R1 * k2;                       // y[k2] = Z_g
                    const int gm = g == 0 ? 0 : L - g;                // Z_g is the mirror term of bin gm
                    if (g >= f_lo && g < f_hi) bp[g - f_lo] = y[k2];
                    if (gm >= f_lo && gm < f_hi) bp[nf + gm - f_lo] = y[k2];
                });
            }
            __syncwarp();
            // ---- amplitudes of the warp's windows, ascending instance order ----------------------------------
#pragma unroll
            for (int i = 0; i < NACC; ++i) {
                const int fi = lane + 32 * i;
                if (fi < nf) {
                    float a = acc[i];
                    for (int p = 0; p < n_pair; ++p) {
                        const float2 z1 = band[p * 2 * nf + fi];
                        const float2 z2 = band[p * 2 * nf + nf + fi];
                        const float re1 = z1.x + z2.x, im1 = z1.y - z2.y;
                        a += 0.5f * sqrtf(fmaf(re1, re1, im1 * im1));
                        if (2 * p + 1 < n_win) {
                            const float re2 = z1.y + z2.y, im2 = z2.x - z1.x;
                            a += 0.5f * sqrtf(fmaf(re2, re2, im2 * im2));
                        }
                    }
                    acc[i] = a;
                }
            }
            __syncwarp();
        }

        // ---- team sum in ascending member order ------------------------------------------------------------------
        if (P.team > 1) {
            if (member != 0) {
#pragma unroll
                for (int i = 0; i < NACC; ++i) part[(warp * NACC + i) * 32 + lane] = acc[i];
            }
            __syncthreads();
            if (member == 0) {
                for (int m = 1; m < P.team; ++m) {
#pragma unroll
                    for (int i = 0; i < NACC; ++i) acc[i] += part[((warp + m) * NACC + i) * 32 + lane];
                }
            }
            __syncthreads();
        }

        // ---- top-k ranking (descending amplitude, lower bin first on ties) and packing --------------------------
        if (active && member == 0) {
            bool bad = false;
#pragma unroll
            for (int i = 0; i < NACC; ++i) {
                const int fi = lane + 32 * i;
                if (fi < nf) {
                    bad |= !isfinite(acc[i]);
                    if (P.amp_dbg) P.amp_dbg[static_cast<size_t>(row) * nf + fi] = acc[i] * inv_n;
                } else {
                    acc[i] = -1.f;                                   // not a candidate
                }
            }
            if (__any_sync(0xffffffffu, bad) && lane == 0) set_status(P.status, VARDROP_ERR_NONFINITE);
            uint64_t key = 0;
            for (int rank = 0; rank < P.k; ++rank) {
                // a candidate is coded (amplitude bits, ~bin): amplitudes are non-negative, so unsigned order is
                // amplitude first, then the lower bin; code 0 = nothing left (taken bins are negative)
                uint64_t best = 0;
#pragma unroll
                for (int i = 0; i < NACC; ++i) {
                    const uint64_t code = (static_cast<uint64_t>(__float_as_uint(acc[i])) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(lane + 32 * i));
                    if (acc[i] >= 0.f && code > best) best = code;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    const uint64_t other = __shfl_xor_sync(0xffffffffu, best, off);
                    best = other > best ? other : best;
                }
                const int best_f = best ? static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(best)) : 0;   // 0 only with non-finite input
#pragma unroll
                for (int i = 0; i < NACC; ++i)
                    if (lane + 32 * i == best_f) acc[i] = -1.f;
                if (lane == 0 && P.freqs) P.freqs[static_cast<size_t>(row) * P.k + rank] = f_lo + best_f;
                key = (key << 12) | static_cast<uint64_t>(f_lo + best_f);
            }
            if (lane == 0) P.keys[row] = key;
        }
    }
}

template <int L, int R1, int R2, int PC, int MINB>
int launch_rows(const RowsParams& P, cudaStream_t stream) {
    using Plan = RowsPlan<L, R1, R2, PC>;
    const size_t smem = Plan::smem_bytes(P.nf);
    static thread_local int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(hash_rows_kernel<L, R1, R2, PC, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     static_cast<int>(Plan::smem_bytes(L / 2 + 1))), "hash: smem attribute"))
            return st;
        attr_dev = dev;
    }
    const int rows_per_cta = kRowsWarps / P.team;
    const int want = (P.N + rows_per_cta - 1) / rows_per_cta;
    int per_sm = static_cast<int>((220 * 1024) / (smem + 1024));
    if (per_sm > 16) per_sm = 16;
    if (per_sm < 1) per_sm = 1;
    const int cap = sm_count() * per_sm;
    const int grid = want < cap ? want : cap;
    cudaError_t err;
    { LaunchScope ls_(K_HASH, stream); err = launch_chained(hash_rows_kernel<L, R1, R2, PC, MINB>, dim3(grid), dim3(kRowsThreads), smem, stream, P); }
    return check_cuda(err, "hash: launch");
}

}  // namespace

// Returns -1 when this length has no register-blocked plan (the caller then takes the shared-memory kernel).
int hash_rows_launch(const float* x, const vardrop_hash_cfg& c, int f_lo, int f_hi, uint64_t* keys, int32_t* freqs, float* amp_dbg,
                     int* status, cudaStream_t stream) {
    if (c.scope != 0) return -1;
    if (c.L != 96 && c.L != 192 && c.L != 336 && c.L != 720) return -1;
    RowsParams P{};
    P.x = x; P.keys = keys; P.freqs = freqs; P.amp_dbg = amp_dbg; P.status = status;
    P.B = c.B; P.N = c.N; P.k = c.k; P.f_lo = f_lo; P.nf = f_hi - f_lo;
    // team size: more warps per row while the rows alone do not fill the GPU and every member still gets two transforms
    int team = 1;
    while (team < kRowsWarps && static_cast<long long>(c.N) * team < 8ll * sm_count() && c.B >= 8 * team) team *= 2;
    P.team = team;
    int per = (c.B + team - 1) / team;
    P.per_member = per + (per & 1);
    switch (c.L) {
        case 96: return launch_rows<96, 8, 12, 8, 5>(P, stream);
        case 192: return launch_rows<192, 12, 16, 4, 3>(P, stream);
        case 336: return launch_rows<336, 16, 21, 2, 4>(P, stream);
        default: return launch_rows<720, 24, 30, 1, 4>(P, stream);
    }
}

}  // namespace vardrop
