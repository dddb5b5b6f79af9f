// k-dominant frequency hashing (Algorithm 1) as one kernel: short real FFTs in shared memory, amplitude,
// low-pass band, fixed-order batch mean, warp-level top-k ranking and hash packing.
//
// Each CTA owns a few hash rows (a variate n in batch-mean scope, an (instance, variate) pair in
// per-instance scope) and all the windows that feed them, so the mean over the batch never leaves the SM
// and is summed in ascending instance order.  Two real windows ride one complex transform
// (z = x1 + i x2; X1_f = (Z_f + conj Z_{L-f}) / 2, X2_f = (Z_f - conj Z_{L-f}) / 2i), which is evaluated by
// a Stockham autosort mixed-radix FFT (radices 4, 2, 3, 5, 7; larger prime factors as plain sums) whose butterflies are spread over the
// whole CTA.  Twiddles are produced once per CTA with sincospif on an angle reduced to half a turn with integers.
#include "common.cuh"
#include "kernels.h"

namespace vardrop {

namespace {

constexpr int kHashThreads = 256;
constexpr int kMaxStages = 16;

struct HashParams {
    const float* x;
    uint64_t* keys;
    int32_t* freqs;
    float* amp_dbg;
    int* status;
    int B, N, L, k, f_lo, nf, scope;
    int rows_total;       // S * N
    int rows_per_cta;     // hash rows per CTA
    int win_per_row;      // windows averaged into one row (B or 1)
    int chunk;            // windows of a row taken per pass
    int n_stages;
    int radix[kMaxStages];
    FastDiv div_L, div_L4, div_nf, div_chunk;
    FastDiv div_lr[kMaxStages];   // L / radix of the stage
    FastDiv div_ns[kMaxStages];   // product of the earlier stages' radices
};

__device__ __forceinline__ float2 cmul(float2 a, float2 b) { return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x); }
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }

// Forward DFT of R points in registers (y_m = sum_j v_j exp(-2 pi i j m / R)).
template <int R>
__device__ __forceinline__ void small_dft(float2* v);

template <>
__device__ __forceinline__ void small_dft<1>(float2*) {}      // the copy-in stage of a length without small factors
template <>
__device__ __forceinline__ void small_dft<2>(float2* v) {
    const float2 a = v[0], b = v[1];
    v[0] = cadd(a, b);
    v[1] = csub(a, b);
}
template <>
__device__ __forceinline__ void small_dft<4>(float2* v) {
    const float2 s02 = cadd(v[0], v[2]), d02 = csub(v[0], v[2]);
    const float2 s13 = cadd(v[1], v[3]), d13 = csub(v[1], v[3]);
    v[0] = cadd(s02, s13);
    v[2] = csub(s02, s13);
    v[1] = make_float2(d02.x + d13.y, d02.y - d13.x);   // d02 - i d13
    v[3] = make_float2(d02.x - d13.y, d02.y + d13.x);   // d02 + i d13
}
// Odd prime R: pair j with R - j;  y_m = a_m - i b_m,  y_{R-m} = a_m + i b_m  with
// a_m = v_0 + sum_j cos(2 pi j m / R) (v_j + v_{R-j}),  b_m = sum_j sin(2 pi j m / R) (v_j - v_{R-j}).
template <int R>
__device__ __forceinline__ void odd_dft(float2* v, const float* cs, const float* sn) {
    constexpr int Hh = (R - 1) / 2;
    float2 p[Hh], m[Hh];
#pragma unroll
    for (int j = 0; j < Hh; ++j) {
        p[j] = cadd(v[j + 1], v[R - 1 - j]);
        m[j] = csub(v[j + 1], v[R - 1 - j]);
    }
    float2 y0 = v[0];
#pragma unroll
    for (int j = 0; j < Hh; ++j) y0 = cadd(y0, p[j]);
    float2 out[R];
    out[0] = y0;
#pragma unroll
    for (int mm = 1; mm <= Hh; ++mm) {
        float2 a = v[0], b = make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 1; j <= Hh; ++j) {
            const int idx = (j * mm) % R;                       // angle index, folded to 1..Hh with a sign on sin
            const int fold = idx <= Hh ? idx : R - idx;
            const float c = cs[fold - 1];
            const float s = idx <= Hh ? sn[fold - 1] : -sn[fold - 1];
            a.x = fmaf(c, p[j - 1].x, a.x);
            a.y = fmaf(c, p[j - 1].y, a.y);
            b.x = fmaf(s, m[j - 1].x, b.x);
            b.y = fmaf(s, m[j - 1].y, b.y);
        }
        out[mm] = make_float2(a.x + b.y, a.y - b.x);
        out[R - mm] = make_float2(a.x - b.y, a.y + b.x);
    }
#pragma unroll
    for (int j = 0; j < R; ++j) v[j] = out[j];
}
template <>
__device__ __forceinline__ void small_dft<3>(float2* v) {
    const float cs[1] = {-0.5f};
    const float sn[1] = {0.8660254037844387f};
    odd_dft<3>(v, cs, sn);
}
template <>
__device__ __forceinline__ void small_dft<5>(float2* v) {
    const float cs[2] = {0.30901699437494745f, -0.8090169943749473f};
    const float sn[2] = {0.9510565162951535f, 0.5877852522924732f};
    odd_dft<5>(v, cs, sn);
}
template <>
__device__ __forceinline__ void small_dft<7>(float2* v) {
    const float cs[3] = {0.6234898018587336f, -0.22252093395631434f, -0.900968867902419f};
    const float sn[3] = {0.7818314824680298f, 0.9749279121818236f, 0.43388373911755823f};
    odd_dft<7>(v, cs, sn);
}

// One Stockham stage over every transform of the pass: butterfly j of a length-L transform reads
// in[j + r L/R], multiplies by w^(r (j mod Ns) L/(Ns R)), transforms the R values and writes
// out[(j div Ns) Ns R + (j mod Ns) + r Ns]  (Ns = product of the radices already done).
template <int R>
__device__ __forceinline__ void fft_stage(const float2* __restrict__ in, float2* __restrict__ out, const float2* __restrict__ tw,
                                          int n_fft, int L, FastDiv div_lr, FastDiv div_ns) {
    const uint32_t LR = div_lr.d, Ns = div_ns.d;
    const uint32_t tw_step = static_cast<uint32_t>(L) / (Ns * R);
    const uint32_t total = static_cast<uint32_t>(n_fft) * LR;
    for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
        const uint32_t p = fd_div(t, div_lr);
        const uint32_t j = t - p * LR;
        const uint32_t q = fd_div(j, div_ns);
        const uint32_t kk = j - q * Ns;
        const float2* src = in + p * L + j;
        float2 v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = src[r * LR];
        if (Ns > 1) {
#pragma unroll
            for (int r = 1; r < R; ++r) v[r] = cmul(v[r], tw[r * kk * tw_step]);
        }
        small_dft<R>(v);
        float2* dst = out + p * L + q * Ns * R + kk;
#pragma unroll
        for (int r = 0; r < R; ++r) dst[r * Ns] = v[r];
    }
}

// The same stage for any radix R (a prime factor above 7), as the plain sum it stands for: one thread per output point
// adds its R inputs times table twiddles.  Output m of butterfly j needs w^(r (kk L/(Ns R) + m L/R)) for input r: the
// exponent advances by a fixed step per input, taken modulo L by one conditional subtraction.  O(L R) per transform.
__device__ __forceinline__ void fft_stage_any(const float2* __restrict__ in, float2* __restrict__ out, const float2* __restrict__ tw,
                                              int n_fft, int L, int R, FastDiv div_lr, FastDiv div_ns) {
    const uint32_t LR = div_lr.d, Ns = div_ns.d, uL = static_cast<uint32_t>(L), uR = static_cast<uint32_t>(R);
    const uint32_t tw_step = uL / (Ns * uR), m_step = uL / uR;
    const uint32_t total = static_cast<uint32_t>(n_fft) * uL;
    for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
        const uint32_t bj = t / uR, m = t - bj * uR;           // m fastest: the threads of a butterfly share its inputs
        const uint32_t p = fd_div(bj, div_lr);
        const uint32_t j = bj - p * LR;
        const uint32_t q = fd_div(j, div_ns);
        const uint32_t kk = j - q * Ns;
        const uint32_t step = (kk * tw_step + m * m_step) % uL;
        const float2* src = in + p * uL + j;
        float2 acc = src[0];
        uint32_t e = 0;
        for (uint32_t r = 1; r < uR; ++r) {
            e += step;
            if (e >= uL) e -= uL;
            const float2 v = src[r * LR], w = tw[e];
            acc.x = fmaf(v.x, w.x, fmaf(-v.y, w.y, acc.x));
            acc.y = fmaf(v.x, w.y, fmaf(v.y, w.x, acc.y));
        }
        out[p * uL + q * Ns * uR + kk + m * Ns] = acc;
    }
}

// First Stockham stage (Ns = 1: no twiddles, butterfly j writes out[j R + r]) reading the windows straight from global
// memory: transform p carries window 2p of the pass in its real part and window 2p + 1 (if any) in its imaginary part.
template <int R>
__device__ __forceinline__ void fft_first_stage(const HashParams& P, float2* __restrict__ out, int n_win, int row0, int b0, int cw,
                                                FastDiv div_lr) {
    const uint32_t L = P.L, LR = div_lr.d;
    const uint32_t n_fft = (n_win + 1) >> 1;
    const uint32_t total = n_fft * LR;
    for (uint32_t t = threadIdx.x; t < total; t += blockDim.x) {
        const uint32_t p = fd_div(t, div_lr);
        const uint32_t j = t - p * LR;
        const float* src[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const uint32_t wl = 2 * p + e;
            const uint32_t r = cw == P.chunk ? fd_div(wl, P.div_chunk) : wl / static_cast<uint32_t>(cw);
            const uint32_t bi = wl - r * cw;
            const size_t w = P.scope == 0 ? static_cast<size_t>(b0 + bi) * P.N + (row0 + r) : static_cast<size_t>(row0 + r);
            src[e] = wl < static_cast<uint32_t>(n_win) ? P.x + w * L + j : nullptr;
        }
        float2 v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = make_float2(__ldg(src[0] + r * LR), src[1] ? __ldg(src[1] + r * LR) : 0.f);
        small_dft<R>(v);
        float2* dst = out + p * L + j * R;
#pragma unroll
        for (int r = 0; r < R; ++r) dst[r] = v[r];
    }
}

__global__ void __launch_bounds__(kHashThreads) hash_kernel(const HashParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int L = P.L, nf = P.nf;
    const int max_win = P.rows_per_cta * P.chunk;           // windows per pass
    const int max_fft = (max_win + 1) / 2;
    float2* tw = reinterpret_cast<float2*>(smem_raw);
    float2* buf0 = tw + L;
    float2* buf1 = buf0 + static_cast<size_t>(max_fft) * L;
    float* acc = reinterpret_cast<float*>(buf1 + static_cast<size_t>(max_fft) * L);   // [rows_per_cta, nf]

    for (int m = threadIdx.x; m < L; m += blockDim.x) {      // w^m = exp(-2 pi i m / L); the angle is folded to |m'| <= L / 2 first
        const int mf = 2 * m > L ? m - L : m;
        float s, c;
        sincospif(2.f * static_cast<float>(mf) / static_cast<float>(L), &s, &c);
        tw[m] = make_float2(c, -s);
    }
    chain_wait();
    chain_release();
    const int row0 = blockIdx.x * P.rows_per_cta;
    const int rows = min(P.rows_per_cta, P.rows_total - row0);
    for (int i = threadIdx.x; i < rows * nf; i += blockDim.x) acc[i] = 0.f;

    for (int b0 = 0; b0 < P.win_per_row; b0 += P.chunk) {
        const int cw = min(P.chunk, P.win_per_row - b0);     // windows of each row in this pass
        const int n_win = rows * cw;
        const int n_fft = (n_win + 1) / 2;
        __syncthreads();
        // ---- mixed-radix Stockham FFT, ping-pong between the two buffers; the first stage reads global memory --
        float2* cur = buf0;
        float2* oth = buf1;
        switch (P.radix[0]) {
            case 2: fft_first_stage<2>(P, cur, n_win, row0, b0, cw, P.div_lr[0]); break;
            case 3: fft_first_stage<3>(P, cur, n_win, row0, b0, cw, P.div_lr[0]); break;
            case 4: fft_first_stage<4>(P, cur, n_win, row0, b0, cw, P.div_lr[0]); break;
            case 5: fft_first_stage<5>(P, cur, n_win, row0, b0, cw, P.div_lr[0]); break;
            case 7: fft_first_stage<7>(P, cur, n_win, row0, b0, cw, P.div_lr[0]); break;
            default: fft_first_stage<1>(P, cur, n_win, row0, b0, cw, P.div_lr[0]); break;      // plain copy-in: every factor is a large prime
        }
        __syncthreads();
        for (int s = 1; s < P.n_stages; ++s) {
            switch (P.radix[s]) {
                case 2: fft_stage<2>(cur, oth, tw, n_fft, L, P.div_lr[s], P.div_ns[s]); break;
                case 3: fft_stage<3>(cur, oth, tw, n_fft, L, P.div_lr[s], P.div_ns[s]); break;
                case 4: fft_stage<4>(cur, oth, tw, n_fft, L, P.div_lr[s], P.div_ns[s]); break;
                case 5: fft_stage<5>(cur, oth, tw, n_fft, L, P.div_lr[s], P.div_ns[s]); break;
                case 7: fft_stage<7>(cur, oth, tw, n_fft, L, P.div_lr[s], P.div_ns[s]); break;
                default: fft_stage_any(cur, oth, tw, n_fft, L, P.radix[s], P.div_lr[s], P.div_ns[s]); break;
            }
            __syncthreads();
            float2* tmp = cur; cur = oth; oth = tmp;
        }
        // ---- amplitudes of the two real windows of every transform, candidate band only ----------------
        float* amp = reinterpret_cast<float*>(oth);          // [n_win, nf]
        for (uint32_t idx = threadIdx.x; idx < static_cast<uint32_t>(n_win) * nf; idx += blockDim.x) {
            const uint32_t wl = fd_div(idx, P.div_nf);
            const uint32_t fi = idx - wl * nf;
            const int f = P.f_lo + fi;
            const float2 z1 = cur[(wl >> 1) * L + f];
            const float2 z2 = cur[(wl >> 1) * L + (f == 0 ? 0 : L - f)];
            float re, im;
            if ((wl & 1) == 0) { re = z1.x + z2.x; im = z1.y - z2.y; }
            else               { re = z1.y + z2.y; im = z2.x - z1.x; }
            amp[idx] = 0.5f * sqrtf(re * re + im * im);
        }
        __syncthreads();
        // ---- running batch sum, ascending instance order ------------------------------------------------
        for (int i = threadIdx.x; i < rows * nf; i += blockDim.x) {
            const int r = i / nf, fi = i - r * nf;
            float a = acc[i];
            for (int bi = 0; bi < cw; ++bi) a += amp[(r * cw + bi) * nf + fi];
            acc[i] = a;
        }
    }
    __syncthreads();

    // ---- top-k ranking (descending amplitude, lower bin first on ties), packing ------------------------------
    // Ranking the batch sums ranks the means.  A candidate is coded as (amplitude bits, ~bin): amplitudes are
    // non-negative, so unsigned comparison of the code orders by amplitude and then by lower bin.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    const float inv_n = 1.f / static_cast<float>(P.win_per_row);
    for (int r = warp; r < rows; r += n_warps) {
        float* a = acc + r * nf;
        const int row = row0 + r;
        bool bad = false;
        for (int fi = lane; fi < nf; fi += 32) {
            const float sum = a[fi];
            bad |= !isfinite(sum);
            if (P.amp_dbg) P.amp_dbg[static_cast<size_t>(row) * nf + fi] = sum * inv_n;
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) set_status(P.status, VARDROP_ERR_NONFINITE);
        uint64_t key = 0;
        for (int rank = 0; rank < P.k; ++rank) {
            uint64_t best = 0;                               // code 0 = nothing found (taken entries are negative)
            for (int fi = lane; fi < nf; fi += 32) {
                const float val = a[fi];
                const uint64_t code = (static_cast<uint64_t>(__float_as_uint(val)) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(fi));
                if (val >= 0.f && code > best) best = code;
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const uint64_t other = __shfl_xor_sync(0xffffffffu, best, off);
                best = other > best ? other : best;
            }
            const int best_f = best ? static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(best)) : 0;      // 0 only with non-finite input
            if (lane == 0) {
                a[best_f] = -1.f;                            // removes the winner
                if (P.freqs) P.freqs[static_cast<size_t>(row) * P.k + rank] = P.f_lo + best_f;
            }
            key = (key << 12) | static_cast<uint64_t>(P.f_lo + best_f);
            __syncwarp();
        }
        if (lane == 0) P.keys[row] = key;
    }
}

}  // namespace

size_t hash_workspace_bytes(const vardrop_hash_cfg&) { return kWsHeaderBytes; }

int hash_validate(const vardrop_hash_cfg& c, int* f_lo, int* f_hi) {
    if (c.B < 1 || c.N < 1 || c.L < 2) return fail(VARDROP_ERR_INVALID_ARG, "hash: B, N >= 1 and L >= 2 required (B=%d N=%d L=%d)", c.B, c.N, c.L);
    if (c.L > 8192) return fail(VARDROP_ERR_UNSUPPORTED, "hash: L=%d above 8192", c.L);
    if (c.k < 1 || c.k > 5) return fail(VARDROP_ERR_INVALID_ARG, "hash: k=%d outside 1..5", c.k);
    if (c.scope != 0 && c.scope != 1) return fail(VARDROP_ERR_INVALID_ARG, "hash: scope=%d (0 batch mean, 1 per instance)", c.scope);
    const int nb = c.L / 2 + 1;
    int lo = c.f_lo, hi = c.f_hi;
    if (lo == 0 && hi == 0) { lo = 1; hi = (nb + 1) / 2; }
    if (lo < 0 || hi > nb || hi > 4096 || lo + c.k > hi)
        return fail(VARDROP_ERR_INVALID_ARG, "hash: band [%d,%d) needs 0 <= f_lo, f_lo + k <= f_hi <= min(L/2+1, 4096)", lo, hi);
    if (static_cast<long long>(c.B) * c.N > (1ll << 31) - 1) return fail(VARDROP_ERR_INVALID_ARG, "hash: B*N too large");
    *f_lo = lo; *f_hi = hi;
    return VARDROP_OK;
}

int hash_launch(const float* x, const vardrop_hash_cfg& c, uint64_t* keys, int32_t* freqs, float* amp_dbg, int* status,
                cudaStream_t stream) {
    int f_lo, f_hi;
    if (int st = hash_validate(c, &f_lo, &f_hi)) return st;
    {
        const int st = hash_rows_launch(x, c, f_lo, f_hi, keys, freqs, amp_dbg, status, stream);
        if (st >= 0) return st;
    }
    HashParams P{};
    P.x = x; P.keys = keys; P.freqs = freqs; P.amp_dbg = amp_dbg; P.status = status;
    P.B = c.B; P.N = c.N; P.L = c.L; P.k = c.k; P.f_lo = f_lo; P.nf = f_hi - f_lo; P.scope = c.scope;
    P.rows_total = c.scope == 0 ? c.N : c.B * c.N;
    P.win_per_row = c.scope == 0 ? c.B : 1;

    // radix plan: fours first, then a two, then the odd primes; prime factors above 7 come last as plain-sum stages (behind
    // a copy-in stage when there is no small factor to read the windows with)
    int rem = c.L, ns = 1;
    P.n_stages = 0;
    auto push = [&](int r) {
        P.radix[P.n_stages] = r;
        P.div_lr[P.n_stages] = make_fastdiv(c.L / r);
        P.div_ns[P.n_stages] = make_fastdiv(ns);
        ns *= r;
        ++P.n_stages;
    };
    while (rem % 4 == 0) { push(4); rem /= 4; }
    for (int p : {2, 3, 5, 7}) while (rem % p == 0) { push(p); rem /= p; }
    if (rem > 1 && P.n_stages == 0) push(1);
    for (int p = 11; rem > 1; p += 2) while (rem % p == 0) { push(p); rem /= p; }

    // windows per pass: about 2048 complex points per buffer, an even count
    int per_pass = 2 * (2048 / c.L);
    if (per_pass < 2) per_pass = 2;
    if (per_pass > 64) per_pass = 64;
    if (P.win_per_row >= per_pass) {
        P.rows_per_cta = 1;
        P.chunk = per_pass;
    } else {
        P.chunk = P.win_per_row;
        P.rows_per_cta = per_pass / P.win_per_row;
        // keep at least a few CTAs per SM in flight
        while (P.rows_per_cta > 1 && (P.rows_total + P.rows_per_cta - 1) / P.rows_per_cta < 592) P.rows_per_cta = (P.rows_per_cta + 1) / 2;
    }
    P.div_L = make_fastdiv(c.L);
    P.div_L4 = make_fastdiv(c.L >= 4 ? c.L / 4 : 1);
    P.div_nf = make_fastdiv(P.nf);
    P.div_chunk = make_fastdiv(P.chunk);

    const int max_fft = (P.rows_per_cta * P.chunk + 1) / 2;
    const size_t smem = sizeof(float2) * (static_cast<size_t>(c.L) + 2ull * max_fft * c.L) + sizeof(float) * P.rows_per_cta * P.nf;
    if (smem > 200 * 1024) return fail(VARDROP_ERR_UNSUPPORTED, "hash: shared memory plan of %zu bytes does not fit", smem);
    static thread_local int attr_done_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_done_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(hash_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024), "hash: smem attribute")) return st;
        attr_done_dev = dev;
    }
    const int grid = (P.rows_total + P.rows_per_cta - 1) / P.rows_per_cta;
    cudaError_t err;
    { LaunchScope ls_(K_HASH, stream); err = launch_chained(hash_kernel, dim3(grid), dim3(kHashThreads), smem, stream, P); }
    return check_cuda(err, "hash: launch");
}

}  // namespace vardrop
