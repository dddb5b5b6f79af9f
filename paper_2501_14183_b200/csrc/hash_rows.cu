// k-dominant frequency hashing (Algorithm 1), batch-mean scope, for the lookback lengths the paper's
// workloads use: a register-blocked two-pass FFT with every index and twiddle fixed at compile time.
//
// Work is laid out by hash row (one variate): a team of 1, 2 or 4 warps owns a row, each warp takes a
// contiguous range of the batch.  Two real windows ride one complex transform of length L = R1 * R2
// (z = x_b + i x_{b+1};  X_b[f] = (Z_f + conj Z_{L-f}) / 2,  X_{b+1}[f] = (Z_f - conj Z_{L-f}) / 2i):
//   staging  the copy engine brings a warp's next windows into shared memory (one bulk copy a window, counted on the warp's
//            mbarrier) while the warp is in pass 2 of the current ones (x is 16-byte aligned and so is every window),
//   pass 1   R2 lanes per transform: lane j2 takes z[j1 R2 + j2] from the staged windows, runs an
//            R1-point DFT in registers, multiplies output k1 by exp(-2 pi i j2 k1 / L) and parks it in the
//            warp's exchange buffer,
//   pass 2   R1 lanes per transform: lane k1 reads its R2 values and runs an R2-point DFT in registers; output k2 is
//            Z[k1 + R1 k2].  The mirror term Z[L - g] of g = k1 + R1 k2 is output R2 - 1 - k2 of lane R1 - k1 of the same
//            transform (output (R2 - k2) mod R2 of lane 0 itself when k1 = 0), so one shuffle pair fetches it and the lane
//            adds both windows' amplitudes of its bins g <= L / 2 to its accumulators: nothing is parked in between.
// Warps never wait for each other inside a row (only __syncwarp); the transforms that share a warp add their accumulators
// in ascending order, then the team's partial sums are added in ascending order by its first warp, which ranks the top k
// bins and packs the hash value.
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

// Complex sums and differences as one packed instruction each (two IEEE fp32 results per issue slot: the kernel is bound by
// instruction issue, not by the fp32 pipe).
__device__ __forceinline__ unsigned long long pack_c(float2 a) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a.x), "f"(a.y));
    return r;
}
__device__ __forceinline__ float2 unpack_c(unsigned long long v) {
    float2 a;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a.x), "=f"(a.y) : "l"(v));
    return a;
}
__device__ __forceinline__ float2 cadd(float2 a, float2 b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pack_c(a)), "l"(pack_c(b)));
    return unpack_c(d);
}
__device__ __forceinline__ float2 csub(float2 a, float2 b) {
    unsigned long long d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pack_c(a)), "l"(pack_c(b)));
    return unpack_c(d);
}

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
    static_assert(R1 <= 32, "a transform's second pass fits a warp");
    static constexpr int G2 = 32 / R1;                                      // transforms per second pass of a warp
    static_assert(PC % G2 == 0, "whole second passes");
    static constexpr int P2 = R2 | 1;                                       // exchange row pitch (complex), odd: pass-2 reads are conflict-free
    static constexpr int PS = R1 * P2 + ((R2 - R1 * P2) % 16 + 16) % 16;    // pitch between transforms: consecutive lanes keep consecutive banks
    static constexpr int K2N = R2 / 2 + 1;                                  // accumulators per lane for the whole spectrum: bins k1 + R1 k2 <= L / 2
    static constexpr int K2Q = ((L / 2 + 2) / 2 + R1 - 1) / R1;             // for the default band, f < ceil((L / 2 + 1) / 2): bins below R1 K2Q
    static constexpr int exch_elems = PC * PS;
    static constexpr int LP = L + 4;                                        // pitch of a staged window (floats): rows stay 16-byte aligned
    static constexpr int stage_elems = 2 * PC * LP;                         // a warp's staged windows: first of every pair, then second
    static constexpr size_t off_exch = sizeof(float2) * L;
    static_assert(sizeof(float) * K2N * 32 <= sizeof(float2) * exch_elems, "a warp's partial sums fit its exchange buffer");
    static constexpr size_t off_stage = (off_exch + sizeof(float2) * kRowsWarps * exch_elems + 15) / 16 * 16;
    static constexpr size_t off_bar = off_stage + sizeof(float) * kRowsWarps * stage_elems;
    static constexpr size_t smem_bytes() { return off_bar + sizeof(uint64_t) * kRowsWarps; }
    static_assert(L % 4 == 0 && off_exch % 16 == 0, "staged windows and their copies are 16-byte aligned");
};

// One window (bytes, a multiple of 16) from global to shared memory by the copy engine; completion is counted on `bar`.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst_smem)), "l"(src),
                 "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Ask for `bytes` (a multiple of 16) at the 16-byte aligned address `p` to be brought into L2; nothing waits for it.
__device__ __forceinline__ void prefetch_l2(const void* p, unsigned bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ float sqrt_fast(float v) {                      // square root by the special-function unit (about 1 ulp)
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// kWide: candidate bins may lie anywhere up to L / 2; otherwise the band ends below R1 K2Q (the default low-pass band does), and
// a lane evaluates, adds up and ranks only its K2Q lowest bins: the outputs of the second pass that no such bin or mirror term
// reads are never computed.
template <int L, int R1, int R2, int PC, int MINB, bool kWide>
__global__ void __launch_bounds__(kRowsThreads, MINB) hash_rows_kernel(const RowsParams P) {
    using Plan = RowsPlan<L, R1, R2, PC>;
    constexpr int P2 = Plan::P2, PS = Plan::PS, K2N = kWide ? Plan::K2N : Plan::K2Q, G2 = Plan::G2, LP = Plan::LP;
    extern __shared__ __align__(16) unsigned char smem_rows[];
    const int nf = P.nf, f_lo = P.f_lo, f_hi = P.f_lo + P.nf;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float2* tw = reinterpret_cast<float2*>(smem_rows);                       // tw[k1 R2 + j2] = exp(-2 pi i j2 k1 / L)
    float2* exch = reinterpret_cast<float2*>(smem_rows + Plan::off_exch) + static_cast<size_t>(warp) * Plan::exch_elems;
    // partial sums of a team member, [K2N][32]: they live in the member's own exchange buffer, which is idle between rows
    auto part_of = [&](int w) { return reinterpret_cast<float*>(smem_rows + Plan::off_exch) + static_cast<size_t>(w) * Plan::exch_elems * 2; };
    float* stage = reinterpret_cast<float*>(smem_rows + Plan::off_stage) + static_cast<size_t>(warp) * Plan::stage_elems;
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_rows + Plan::off_bar) + warp;     // this warp's staged windows have landed
    if (lane == 0) {
        mbar_init(bar, 1);
        mbar_fence_init();
    }

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
    const float inv_n = 0.5f / static_cast<float>(P.B);                      // the halves of the two-for-one split are taken at the end
    const int grp = lane / R1, k1 = lane - grp * R1;                         // second pass: transform of the pass, first index
    const bool lane_used = grp < G2;
    const int partner = lane_used ? lane - k1 + (R1 - k1) % R1 : lane;       // holds the mirror terms of this lane's outputs
    const int row_step = gridDim.x * rows_per_cta;
    const int b_lo = member * P.per_member, b_end = min(P.B, b_lo + P.per_member);     // this warp's windows of a row
    uint32_t landed = 0;                                                     // parity of the mbarrier phase to wait for next
    // Stage windows [c, c + 2 PC) of `row` (those below b_end): lane 0 announces the bytes, lane w copies window c + w.
    auto stage_windows = [&](int row, int c) {
        const int n = min(2 * PC, b_end - c);
        // (the warp's reads of the staged windows are complete: their values went through the transform before the
        // __syncwarp that precedes this call)
        if (lane == 0) mbar_expect_tx(bar, static_cast<uint32_t>(n) * L * sizeof(float));
        __syncwarp();
        if (lane < n)
            bulk_load(stage + ((lane & 1) * PC + (lane >> 1)) * LP, P.x + (static_cast<size_t>(c + lane) * P.N + row) * L, L * sizeof(float), bar);
    };
    {
        const int row0 = blockIdx.x * rows_per_cta + warp / P.team;
        if (row0 < P.N && b_lo < b_end) stage_windows(row0, b_lo);
    }

    for (int row_base = blockIdx.x * rows_per_cta; row_base < P.N; row_base += gridDim.x * rows_per_cta) {
        const int row = row_base + warp / P.team;
        const bool active = row < P.N;
        float acc[K2N];                                                      // acc[k2]: bin k1 + R1 k2 over this lane's transforms
#pragma unroll
        for (int i = 0; i < K2N; ++i) acc[i] = 0.f;

        const int b_hi = active ? b_end : 0;
        // the windows this warp transforms after this row's: ask for them now, so that they wait in L2 by the time they are copied
        const int next_row = row + row_step;
        if (next_row < P.N) {
            for (int b = b_lo + lane; b < b_end; b += 32)
                prefetch_l2(P.x + (static_cast<size_t>(b) * P.N + next_row) * L, L * sizeof(float));
        }
        for (int c0 = b_lo; c0 < b_hi; c0 += 2 * PC) {
            const int n_win = min(2 * PC, b_hi - c0);
            const int n_pair = (n_win + 1) >> 1;
            if (!__all_sync(0xffffffffu, mbar_wait(bar, landed)) && lane == 0) set_status(P.status, VARDROP_ERR_TIMEOUT);
            landed ^= 1u;
            // ---- pass 1 ---------------------------------------------------------------------------------------
            for (int t = lane; t < n_pair * R2; t += 32) {
                const int p = t / R2, j2 = t - p * R2;
                const int b1 = c0 + 2 * p;
                const bool two = b1 + 1 < b_hi;
                float2 v[R1], y[R1];
                const float* s1 = stage + p * LP + j2;
                const float* s2 = s1 + (two ? PC * LP : 0);
                static_for<0, R1>([&](auto J) {
                    constexpr int j1 = decltype(J)::value;
                    v[j1].x = s1[j1 * R2];
                    v[j1].y = s2[j1 * R2];
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
            // the staged windows are consumed: bring in the next ones
            if (c0 + 2 * PC < b_hi) stage_windows(row, c0 + 2 * PC);
            else if (next_row < P.N && b_lo < b_end) stage_windows(next_row, b_lo);
            // ---- pass 2, amplitudes -------------------------------------------------------------------------------
            for (int p0 = 0; p0 < n_pair; p0 += G2) {
                const int p = p0 + grp;
                const bool live = lane_used && p < n_pair;
                const float2* src = exch + (live ? p : 0) * PS + (lane_used ? k1 : 0) * P2;
                float2 v[R2], y[R2];
                static_for<0, R2>([&](auto J) { v[decltype(J)::value] = src[decltype(J)::value]; });
                dft<R2, 1, 1>(v, y);                                     // y[k2] = Z[k1 + R1 k2]
                const bool two = 2 * p + 1 < n_win;
                static_for<0, K2N>([&](auto K) {
                    constexpr int k2 = decltype(K)::value;
                    constexpr int far = R2 - 1 - k2, own = (R2 - k2) % R2;
                    float mx = __shfl_sync(0xffffffffu, y[far].x, partner), my = __shfl_sync(0xffffffffu, y[far].y, partner);
                    if (k1 == 0) { mx = y[own].x; my = y[own].y; }
                    const float re1 = y[k2].x + mx, im1 = y[k2].y - my;
                    const float re2 = y[k2].y + my, im2 = mx - y[k2].x;
                    const float a1 = sqrt_fast(fmaf(re1, re1, im1 * im1));
                    const float a2 = sqrt_fast(fmaf(re2, re2, im2 * im2));
                    if (live) acc[k2] += two ? a1 + a2 : a1;
                });
            }
            __syncwarp();
        }
        // the transforms that shared a second pass: their sums go to the first of them, in ascending order
#pragma unroll
        for (int j = 1; j < G2; ++j) {
#pragma unroll
            for (int i = 0; i < K2N; ++i) {
                const float other = __shfl_sync(0xffffffffu, acc[i], (lane + j * R1) & 31);
                if (lane < R1) acc[i] += other;
            }
        }

        // ---- team sum in ascending member order ------------------------------------------------------------------
        if (P.team > 1) {
            if (member != 0) {
#pragma unroll
                for (int i = 0; i < K2N; ++i) part_of(warp)[i * 32 + lane] = acc[i];
            }
            __syncthreads();
            if (member == 0) {
                for (int m = 1; m < P.team; ++m) {
#pragma unroll
                    for (int i = 0; i < K2N; ++i) acc[i] += part_of(warp + m)[i * 32 + lane];
                }
            }
            __syncthreads();
        }

        // ---- top-k ranking (descending amplitude, lower bin first on ties) and packing --------------------------
        // lane k1 < R1 holds bin k1 + R1 i in acc[i]
        if (active && member == 0) {
            bool bad = false;
#pragma unroll
            for (int i = 0; i < K2N; ++i) {
                const int bin = lane + R1 * i;
                if (lane < R1 && bin >= f_lo && bin < f_hi) {
                    bad |= !isfinite(acc[i]);
                    if (P.amp_dbg) P.amp_dbg[static_cast<size_t>(row) * nf + bin - f_lo] = acc[i] * inv_n;
                } else {
                    acc[i] = -1.f;                                   // not a candidate
                }
            }
            if (__any_sync(0xffffffffu, bad) && lane == 0) set_status(P.status, VARDROP_ERR_NONFINITE);
            uint64_t key = 0;
            for (int rank = 0; rank < P.k; ++rank) {
                // the largest amplitude left, then the lowest bin that has it: two warp-wide integer reductions.  Amplitudes
                // are non-negative, so their bit patterns order like the values; 0 = nothing left (taken bins are negative).
                float top = -1.f;
#pragma unroll
                for (int i = 0; i < K2N; ++i) top = fmaxf(top, acc[i]);
                const unsigned top_all = __reduce_max_sync(0xffffffffu, top >= 0.f ? __float_as_uint(top) + 1u : 0u);
                unsigned bin = 0xffffffffu;
#pragma unroll
                for (int i = K2N - 1; i >= 0; --i)
                    if (acc[i] >= 0.f && __float_as_uint(acc[i]) + 1u == top_all) bin = static_cast<unsigned>(lane + R1 * i);
                const unsigned bin_all = __reduce_min_sync(0xffffffffu, bin);
                const int best_bin = top_all ? static_cast<int>(bin_all) : f_lo;          // f_lo only with non-finite input
#pragma unroll
                for (int i = 0; i < K2N; ++i)
                    if (lane + R1 * i == best_bin) acc[i] = -1.f;
                if (lane == 0 && P.freqs) P.freqs[static_cast<size_t>(row) * P.k + rank] = best_bin;
                key = (key << 12) | static_cast<uint64_t>(best_bin);
            }
            if (lane == 0) P.keys[row] = key;
        }
    }
}

template <int L, int R1, int R2, int PC, int MINB, bool kWide>
int launch_rows(const RowsParams& P, cudaStream_t stream) {
    using Plan = RowsPlan<L, R1, R2, PC>;
    const size_t smem = Plan::smem_bytes();
    static thread_local int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(hash_rows_kernel<L, R1, R2, PC, MINB, kWide>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     static_cast<int>(smem)), "hash: smem attribute"))
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
    { LaunchScope ls_(K_HASH, stream); err = launch_chained(hash_rows_kernel<L, R1, R2, PC, MINB, kWide>, dim3(grid), dim3(kRowsThreads), smem, stream, P); }
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
    if (reinterpret_cast<uintptr_t>(x) % 16 != 0) return fail(VARDROP_ERR_INVALID_ARG, "hash: x is not 16-byte aligned");
    int per = (c.B + team - 1) / team;
    P.per_member = per + (per & 1);
    switch (c.L) {
        case 96: return f_hi <= 8 * RowsPlan<96, 8, 12, 4>::K2Q ? launch_rows<96, 8, 12, 4, 5, false>(P, stream) : launch_rows<96, 8, 12, 4, 5, true>(P, stream);
        case 192: return f_hi <= 12 * RowsPlan<192, 12, 16, 2>::K2Q ? launch_rows<192, 12, 16, 2, 3, false>(P, stream) : launch_rows<192, 12, 16, 2, 3, true>(P, stream);
        case 336: return f_hi <= 16 * RowsPlan<336, 16, 21, 2>::K2Q ? launch_rows<336, 16, 21, 2, 4, false>(P, stream) : launch_rows<336, 16, 21, 2, 4, true>(P, stream);
        default: return f_hi <= 24 * RowsPlan<720, 24, 30, 1>::K2Q ? launch_rows<720, 24, 30, 1, 4, false>(P, stream) : launch_rows<720, 24, 30, 1, 4, true>(P, stream);
    }
}

}  // namespace vardrop
