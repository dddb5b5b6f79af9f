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
    w.total = o;
    return w;
}

// Tensor map over a [B, tokens, H, 64] bf16 tensor: box = one (b, h) tile of 128 tokens x 64 elements,
// 128-byte swizzle, out-of-range rows read as zero.  `tokens` is the extent the copy engine may touch,
// `token_stride` the allocated tokens per instance.
// Number of SMs of the current device (cached per thread and device).
int sm_count();

int make_tile_map(CUtensorMap* map, const void* base, int B, int tokens, int token_stride, int H);

// First 1024-byte boundary at or after p (swizzled tiles need it).
__device__ __forceinline__ unsigned char* align_tiles(unsigned char* p) {
    return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~static_cast<uintptr_t>(1023));
}

// Operands either come straight from the caller's tensors (all-token path at D = 64) or from the staged
// copies in the workspace (a selection is given, or D = 32 needs padding).
inline bool attn_uses_staging(const vardrop_attn_cfg& c, const int32_t* sel_idx) { return sel_idx != nullptr || c.D != kDP; }

}  // namespace vardrop
