// Shared pieces of the attention forward / backward: workspace layout, TMA tensor maps, tile geometry.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace vardrop {

constexpr int kTile = 128;          // tokens per query tile and per key tile
constexpr int kDP = 64;             // head dimension the kernels run at (D = 32 is zero-padded to it)
constexpr int kRowBytes = kDP * 2;  // one (token, head) row of bf16: 128 bytes = one swizzle row
constexpr int kTileBytes = kTile * kRowBytes;   // 16 KiB

struct AttnWs {
    size_t qg, kg, vg, dog;   // staged [B, Ncap, H, 64] bf16 copies (gathered and/or padded)
    size_t delta;             // [B, H, Ncap] fp32
    size_t dq_acc;            // [B, Ncap, H, 64] fp32
    size_t tile_done;         // [B, H] int32: key tiles of (b, h) whose backward work is complete
    size_t total;
    int Ncap;
};

inline AttnWs attn_layout(const vardrop_attn_cfg& c) {
    AttnWs w;
    w.Ncap = (c.N + kTile - 1) / kTile * kTile;
    const size_t staged = static_cast<size_t>(c.B) * w.Ncap * c.H * kRowBytes;
    size_t o = kWsHeaderBytes;
    w.qg = o; o += align_up(staged, 1024);
    w.kg = o; o += align_up(staged, 1024);
    w.vg = o; o += align_up(staged, 1024);
    w.dog = o; o += align_up(staged, 1024);
    w.delta = o; o += align_up(sizeof(float) * c.B * c.H * w.Ncap, 1024);
    w.dq_acc = o; o += align_up(staged * 2, 1024);
    w.tile_done = o; o += align_up(sizeof(int32_t) * c.B * c.H, 1024);
    w.total = o;
    return w;
}

// Tensor map over a [B, tokens, H, 64] bf16 tensor: box = one (b, h) tile of 128 tokens x 64 elements,
// 128-byte swizzle, out-of-range rows read as zero.  `tokens` is the extent the copy engine may touch,
// `token_stride` the allocated tokens per instance.
// Tensor map over the same memory seen as [rows, 64] bf16 (rows = B * tokens * H) for row gathers: box = one row,
// 128-byte swizzle, rows outside the tensor read as zero.
int make_row_map(CUtensorMap* map, const void* base, long long rows, long long row_stride_elems);

// Tensor map over the fp32 dQ' accumulator [B, Ncap, H, 64]: box = 128 tokens x 32 floats (one 128-byte swizzled row
// per token) of one head, the unit of the backward kernel's bulk reduce-add.
int make_acc_map(CUtensorMap* map, const void* base, int B, int Ncap, int H);

// Number of SMs of the current device (cached per thread and device).
int sm_count();

int make_tile_map(CUtensorMap* map, const void* base, int B, int tokens, int H, long long sB, long long sN, long long sH);

// Element strides of q, k, v as the kernels see them.  The row view (one 64-element row per (instance, token, head), rows a
// constant distance apart) exists when sN and sB are multiples of sH: row(b, n, h) = b row_b + n row_n + h.
struct QkvLayout {
    long long sB, sN, sH;       // element strides
    bool row_linear;            // the row view exists
    long long rows_total;       // rows of that view (one past the last is the zero row of the gathers)
    long long row_b, row_n;
};
inline QkvLayout qkv_layout(const vardrop_attn_cfg& c) {
    QkvLayout L;
    const bool dflt = c.sB == 0 && c.sN == 0 && c.sH == 0;
    L.sH = dflt ? c.D : c.sH;
    L.sN = dflt ? static_cast<long long>(c.H) * c.D : c.sN;
    L.sB = dflt ? static_cast<long long>(c.N) * c.H * c.D : c.sB;
    L.row_linear = L.sN % L.sH == 0 && L.sB % L.sH == 0;
    L.row_n = L.row_linear ? L.sN / L.sH : 0;
    L.row_b = L.row_linear ? L.sB / L.sH : 0;
    L.rows_total = L.row_linear ? (c.B - 1) * L.row_b + (c.N - 1) * L.row_n + c.H : 0;
    return L;
}

// First 1024-byte boundary at or after p (swizzled tiles need it).
__device__ __forceinline__ unsigned char* align_tiles(unsigned char* p) {
    return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~static_cast<uintptr_t>(1023));
}

// How a 128-token operand tile reaches shared memory.
//   tiled    one 4-D box of the [B, tokens, H, 64] tensor (tokens tok0 .. tok0 + 127 of head h, instance b)
//   gathered 32 row gathers of 4 rows each from the [rows, 64] view: slot j of the tile is variate idx[tok0 + j]
//            (idx = NULL: the slot itself) while tok0 + j < n_valid, and a row past the end (zeros) otherwise.
// Called by all 32 lanes of one warp; `lane0_expect` bytes are announced on the barrier by lane 0 first.
struct TileSource {
    const int32_t* idx;    // gather indices of the instance's selection (NULL: identity)
    int gathered;          // 0: tiled box, 1: row gathers
    int tokens;            // tokens per instance in the gathered tensor
    int rows_total;        // rows of the [rows, 64] view; row(b, n, h) = b row_b + n row_n + h
    int row_b, row_n;
};
// Rows of the [rows, 64] view that the four slots tok0 + 4 lane .. + 3 of a gathered tile name (a row past the end for
// slots at or past n_valid).  `picks` are the four entries idx[tok0 + 4 lane ..] (see tile_picks), fetched ahead of
// time so that several tiles over the same slots share one fetch.
__device__ __forceinline__ int4 tile_picks(const TileSource& src, int tok0) {
    const int lane = threadIdx.x & 31;
    const int slot = tok0 + 4 * lane;
    if (!src.gathered || !src.idx) return make_int4(slot, slot + 1, slot + 2, slot + 3);
    int4 p;
    p.x = slot + 0 < src.tokens ? src.idx[slot + 0] : -1;
    p.y = slot + 1 < src.tokens ? src.idx[slot + 1] : -1;
    p.z = slot + 2 < src.tokens ? src.idx[slot + 2] : -1;
    p.w = slot + 3 < src.tokens ? src.idx[slot + 3] : -1;
    return p;
}
__device__ __forceinline__ void load_tile_picked(unsigned char* dst, const CUtensorMap* map, uint64_t* bar, const TileSource& src, int4 picks,
                                                 int tok0, int n_valid, int h, int b, int H) {
    const int lane = threadIdx.x & 31;
    if (!src.gathered) {
        if (lane == 0) tma_load_4d(dst, map, bar, 0, h, tok0, b);
        return;
    }
    const int slot = tok0 + 4 * lane;
    const int n[4] = {picks.x, picks.y, picks.z, picks.w};
    int rows[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) rows[e] = (slot + e < n_valid && n[e] >= 0) ? b * src.row_b + n[e] * src.row_n + h : src.rows_total;
    tma_gather4(dst + lane * 4 * kRowBytes, map, bar, 0, rows[0], rows[1], rows[2], rows[3]);
}
__device__ __forceinline__ void load_tile(unsigned char* dst, const CUtensorMap* map, uint64_t* bar, const TileSource& src, int tok0, int n_valid,
                                          int h, int b, int H) {
    load_tile_picked(dst, map, bar, src, tile_picks(src, tok0), tok0, n_valid, h, b, H);
}

// Three ways for the operand tiles to reach shared memory:
//   direct   4-D boxes of the caller's tensors                       (no selection, D = 64)
//   gathered row gathers of the kept variates from the caller's tensors   (selection, D = 64, N <= kGatherMaxN: the kept set
//            is at most a few tiles, so re-gathering rows per tile pair costs less than a staging pass)
//   staged   4-D boxes of compacted copies in the workspace, written by the gather kernel   (D = 32, which is also
//            zero-padded to 64 there; or a selection at large N, where every tile is re-read many times and
//            contiguous, L2-resident tiles pay for the extra pass)
constexpr int kGatherMaxN = 512;
// Number of selection rows: one shared by the batch, or one per instance.
inline int attn_sel_rows(const vardrop_attn_cfg& c) { return c.S > 1 ? c.S : 1; }

// Largest kept count over the selection rows (device, whole CTA; `scratch` is one int of shared memory).
__device__ __forceinline__ int max_kept(const int32_t* n_sel, int S, int N, int* scratch) {
    if (!n_sel) return N;
    if (threadIdx.x == 0) *scratch = 0;
    __syncthreads();
    int m = 0;
    for (int s = threadIdx.x; s < S; s += blockDim.x) m = max(m, n_sel[s]);
    if (m > 0) atomicMax(scratch, m);
    __syncthreads();
    return *scratch;
}

// (row gathers also need the row view of the caller's strides and row indices that fit 31 bits; other layouts are staged)
inline bool attn_uses_gather(const vardrop_attn_cfg& c, const int32_t* sel_idx) {
    const QkvLayout L = qkv_layout(c);
    return c.D == kDP && sel_idx != nullptr && c.N <= kGatherMaxN && L.row_linear && L.rows_total < (1ll << 31);
}
inline bool attn_uses_staging(const vardrop_attn_cfg& c, const int32_t* sel_idx) { return c.D != kDP || (sel_idx != nullptr && !attn_uses_gather(c, sel_idx)); }

}  // namespace vardrop
