// Gather of the kept raw variates (Sec. 3.3: VarDrop removes the dropped variates of the lookback window before the embedding,
// so the rest of the model sees only N' variates): x_sel[b, j, :] = x[b, sel_idx[j], :] for j < n_sel.
// A pure copy: rows of L floats move as 16-byte chunks when L is a multiple of 4 (4-byte words otherwise), several
// independent loads in flight per thread.
#include "common.cuh"
#include "kernels.h"

namespace vardrop {

namespace {

struct GatherRowsParams {
    const void* x;
    void* x_sel;
    const int32_t* sel_idx;   // [S, N]
    const int32_t* n_sel;     // [S]
    int N, S;
    int words_row;            // copy words (16 or 4 bytes) per row
};

template <class Word>
__global__ void __launch_bounds__(256) gather_rows_kernel(const GatherRowsParams P) {
    chain_wait();
    chain_release();
    const int b = blockIdx.y;
    const int srow = P.S > 1 ? b : 0;
    const int32_t* sel = P.sel_idx + static_cast<size_t>(srow) * P.N;
    const int n_sel = P.n_sel[srow];
    const long long total = static_cast<long long>(n_sel) * P.words_row;
    const Word* src_b = static_cast<const Word*>(P.x) + static_cast<size_t>(b) * P.N * P.words_row;
    Word* dst_b = static_cast<Word*>(P.x_sel) + static_cast<size_t>(b) * P.N * P.words_row;
    constexpr int U = 4;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long base = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; base < total; base += U * stride) {
        const Word* from[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long idx = base + u * stride;
            from[u] = nullptr;
            if (idx < total) {
                const int j = static_cast<int>(idx / P.words_row);
                const int c = static_cast<int>(idx - static_cast<long long>(j) * P.words_row);
                from[u] = src_b + static_cast<size_t>(__ldg(sel + j)) * P.words_row + c;
            }
        }
        Word val[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (from[u]) val[u] = __ldg(from[u]);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long idx = base + u * stride;
            if (idx < total) dst_b[idx] = val[u];
        }
    }
}

}  // namespace

int gather_rows_validate(const vardrop_gather_cfg& c) {
    if (c.B < 1 || c.N < 1 || c.L < 1) return fail(VARDROP_ERR_INVALID_ARG, "gather_rows: B, N, L >= 1 required (B=%d N=%d L=%d)", c.B, c.N, c.L);
    if (c.B > 65535) return fail(VARDROP_ERR_UNSUPPORTED, "gather_rows: B above 65535");
    if (c.S != 0 && c.S != 1 && c.S != c.B) return fail(VARDROP_ERR_INVALID_ARG, "gather_rows: S=%d must be 1 (shared selection) or B (one per instance)", c.S);
    return VARDROP_OK;
}

int gather_rows_launch(const float* x, const int32_t* sel_idx, const int32_t* n_sel, const vardrop_gather_cfg& c, float* x_sel, cudaStream_t stream) {
    GatherRowsParams P{};
    P.x = x; P.x_sel = x_sel; P.sel_idx = sel_idx; P.n_sel = n_sel; P.N = c.N; P.S = c.S > 1 ? c.S : 1;
    const bool wide = c.L % 4 == 0;
    P.words_row = wide ? c.L / 4 : c.L;
    const long long work = static_cast<long long>(c.N) * P.words_row;
    long long gx = (work + 255) / 256;
    const long long cap = max(1, 8 * sm_count() / c.B);        // about eight CTAs per SM in total: the kept count is only known on the device
    if (gx > cap) gx = cap;
    cudaError_t err;
    {
        LaunchScope ls_(K_GATHER_ROWS, stream);
        err = wide ? launch_chained(gather_rows_kernel<uint4>, dim3(static_cast<unsigned>(gx), c.B), dim3(256), 0, stream, P)
                   : launch_chained(gather_rows_kernel<uint32_t>, dim3(static_cast<unsigned>(gx), c.B), dim3(256), 0, stream, P);
    }
    return check_cuda(err, "gather_rows: launch");
}

}  // namespace vardrop
