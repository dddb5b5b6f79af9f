// Token gather and attention forward (Eq. 3) over the kept variate tokens.
//
// gather_kernel     compacts q/k/v rows named by sel_idx into [B, Ncap, H, 64] staging buffers with 16-byte
//                   copies, zero-pads D = 32 to 64 and zero-fills the ragged end of the last 128-token tile.
// attn_fwd_kernel   one CTA per (128-query tile, head, instance): TMA loads the Q tile once and streams K/V
//                   tiles through a two-stage ring; S = Q K^T and O_j = P V run on the tcgen05 tensor cores
//                   with accumulators in tensor memory; the online softmax is done by 128 threads, one
//                   query row each, straight from tensor memory.
#include "attn_common.cuh"

namespace vardrop {

// ---------------------------------------------------------------------------------------------------------
// host: tensor maps
// ---------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Encoding a tensor map costs a driver call of a microsecond or two and a training loop passes the same buffers step after
// step: a small per-thread cache, keyed by everything the encoding depends on, returns the map of a known buffer.
namespace {
struct MapKey {
    const void* base;
    long long a;
    int kind, b, c, d;
    bool operator==(const MapKey& o) const { return base == o.base && a == o.a && kind == o.kind && b == o.b && c == o.c && d == o.d; }
};
struct alignas(64) MapSlot {
    CUtensorMap map;
    MapKey key;
    bool used;
};
constexpr int kMapSlots = 256;
MapSlot* map_slot(const MapKey& k) {
    static thread_local MapSlot slots[kMapSlots] = {};
    const uintptr_t h = (reinterpret_cast<uintptr_t>(k.base) >> 8) * 0x9E3779B97F4A7C15ull + static_cast<uintptr_t>(k.kind) * 0x632BE5ABull;
    return &slots[(h >> 40) % kMapSlots];
}
}  // namespace

int sm_count() {
    static thread_local int cached_dev = -1, cached = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) cached = n;
        cached_dev = dev;
    }
    return cached;
}

int make_tile_map(CUtensorMap* map, const void* base, int B, int tokens, int token_stride, int H) {
    const MapKey key{base, 0, 1, B, tokens, token_stride * 65536 + H};
    MapSlot* slot = map_slot(key);
    if (slot->used && slot->key == key) { *map = slot->map; return VARDROP_OK; }
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled entry point not available");
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(kDP), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(tokens),
                                static_cast<cuuint64_t>(B)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(kRowBytes), static_cast<cuuint64_t>(H) * kRowBytes,
                                   static_cast<cuuint64_t>(token_stride) * H * kRowBytes};
    const cuuint32_t box[4] = {kDP, 1, kTile, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r));
    slot->map = *map; slot->key = key; slot->used = true;
    return VARDROP_OK;
}

int make_row_map(CUtensorMap* map, const void* base, long long rows) {
    const MapKey key{base, rows, 2, 0, 0, 0};
    MapSlot* slot = map_slot(key);
    if (slot->used && slot->key == key) { *map = slot->map; return VARDROP_OK; }
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled entry point not available");
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(kDP), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(kRowBytes)};
    const cuuint32_t box[2] = {kDP, 1};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled (row view) failed with code %d", static_cast<int>(r));
    slot->map = *map; slot->key = key; slot->used = true;
    return VARDROP_OK;
}

int make_acc_map(CUtensorMap* map, const void* base, int B, int Ncap, int H) {
    const MapKey key{base, 0, 3, B, Ncap, H};
    MapSlot* slot = map_slot(key);
    if (slot->used && slot->key == key) { *map = slot->map; return VARDROP_OK; }
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled entry point not available");
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(kDP), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(Ncap), static_cast<cuuint64_t>(B)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(kDP) * 4, static_cast<cuuint64_t>(H) * kDP * 4, static_cast<cuuint64_t>(Ncap) * H * kDP * 4};
    const cuuint32_t box[4] = {32, 1, kTile, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled (accumulator) failed with code %d", static_cast<int>(r));
    slot->map = *map; slot->key = key; slot->used = true;
    return VARDROP_OK;
}

int attn_validate(const vardrop_attn_cfg& c) {
    if (c.B < 1 || c.N < 1 || c.H < 1) return fail(VARDROP_ERR_INVALID_ARG, "attention: B, N, H >= 1 required (B=%d N=%d H=%d)", c.B, c.N, c.H);
    if (c.D != 32 && c.D != 64) return fail(VARDROP_ERR_UNSUPPORTED, "attention: head dimension %d (32 or 64 supported)", c.D);
    if (c.N > 65536) return fail(VARDROP_ERR_UNSUPPORTED, "attention: N=%d above 65536", c.N);
    if (static_cast<long long>(c.B) * c.N * c.H >= (1ll << 31)) return fail(VARDROP_ERR_UNSUPPORTED, "attention: B*N*H above 2^31");
    if (c.H > 65535 || c.B > 65535) return fail(VARDROP_ERR_UNSUPPORTED, "attention: B or H above 65535");
    if (c.S != 0 && c.S != 1 && c.S != c.B) return fail(VARDROP_ERR_INVALID_ARG, "attention: S=%d must be 1 (shared selection) or B (one per instance)", c.S);
    if (!(c.sm_scale >= 0.f)) return fail(VARDROP_ERR_INVALID_ARG, "attention: sm_scale must be >= 0 (0 selects 1/sqrt(D))");
    return VARDROP_OK;
}

size_t attn_workspace_bytes(const vardrop_attn_cfg& c) { return attn_layout(c).total; }

namespace {

// ---------------------------------------------------------------------------------------------------------
// gather
// ---------------------------------------------------------------------------------------------------------
struct GatherParams {
    const uint4* src[3];
    uint4* dst[3];
    const int32_t* sel_idx;   // NULL: identity
    const int32_t* n_sel;     // NULL with sel_idx NULL
    int N, Ncap, H, D, S;     // S selection rows (1: shared, B: per instance)
};

__global__ void __launch_bounds__(256) gather_kernel(const GatherParams P) {
    chain_wait();
    chain_release();
    const int b = blockIdx.y, t = blockIdx.z;
    const int srow = P.S > 1 ? b : 0;                                         // selection row of this instance
    const int32_t* sel = P.sel_idx ? P.sel_idx + static_cast<size_t>(srow) * P.N : nullptr;
    const int n_sel = P.sel_idx ? P.n_sel[srow] : P.N;
    const int n_fill = min(P.Ncap, (n_sel + kTile - 1) / kTile * kTile);     // rows to define: kept + zero tail of the tile
    const int chunks_row = P.H * (kDP / 8);                                   // 16-byte chunks per staged token
    const int src_chunks_head = P.D / 8;
    const int total = n_fill * chunks_row;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int j = idx / chunks_row;
        const int c = idx - j * chunks_row;
        const int h = c / (kDP / 8), dc = c - h * (kDP / 8);
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (j < n_sel && dc < src_chunks_head) {
            const int n = sel ? sel[j] : j;
            val = __ldg(P.src[t] + (static_cast<size_t>(b) * P.N + n) * (P.H * src_chunks_head) + h * src_chunks_head + dc);
        }
        P.dst[t][(static_cast<size_t>(b) * P.Ncap + j) * chunks_row + c] = val;
    }
}

// ---------------------------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------------------------
struct FwdParams {
    __nv_bfloat16* o;
    float* lse;
    const int32_t* n_sel;   // [S] kept counts; NULL: all N tokens
    int* status;
    float4* dq_acc;         // [B, Ncap, H, 64] fp32: zeroed here for the backward pass when it will accumulate into it
    int32_t* tile_done;     // [B, H] completion counters of the backward pass, zeroed here
    TileSource src;         // where Q, K, V tiles come from
    int B, N, Ncap, H, D, S;
    float scale_log2;       // sm_scale * log2(e)
};

constexpr int kFwdThreads = 128;
constexpr uint32_t kFwdTmemCols = 256;
constexpr int kFwdSmemBytes = 1024 /*barriers + alignment*/ + kTileBytes /*Q*/ + 2 * kTileBytes /*K*/ + 2 * kTileBytes /*V*/ + 2 * kTileBytes /*P*/;

// 2^x by the special-function unit (relative error about 2^-22; -inf gives 0)
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two fp32 values in one 64-bit register pair, for the packed fp32 instructions of sm_100 (one issue slot for two results;
// each half is the IEEE operation of the scalar instruction, so results do not change).
__device__ __forceinline__ uint64_t pair_of(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void halves_of(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma_pair(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_pair(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Writes 32 consecutive columns (c0 .. c0+31, c0 a multiple of 32) of row `r` of a 128 x 128 bf16 tile held as two
// K-major panels of 64 columns, each row 128 bytes with the 128-byte swizzle.
__device__ __forceinline__ void store_row_chunk32(unsigned char* tile, int r, int c0, const float* v) {
    unsigned char* panel = tile + (c0 >> 6) * kTileBytes + r * kRowBytes;
    const int chunk0 = (c0 & 63) >> 3;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint4 w = make_uint4(pack_bf16(v[8 * q + 0], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                                   pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
        *reinterpret_cast<uint4*>(panel + (((chunk0 + q) ^ (r & 7)) << 4)) = w;
    }
}

__global__ void __launch_bounds__(kFwdThreads) attn_fwd_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                const __grid_constant__ CUtensorMap map_k,
                                                                const __grid_constant__ CUtensorMap map_v, const FwdParams P) {
    extern __shared__ unsigned char smem_dyn[];
    // Set-up first (shared-memory carve-up, barriers, tensor memory): it touches nothing another kernel produces, so it runs
    // while the previous kernel of the stream is still finishing.
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_dyn);     // barriers and the TMEM slot sit in front of the tiles
    uint64_t* bar_q = bars + 0;
    uint64_t* bar_kv = bars + 1;                    // [2]
    uint64_t* bar_s = bars + 3;
    uint64_t* bar_o = bars + 4;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
    unsigned char* sQ = align_tiles(smem_dyn + 64);
    unsigned char* sK = sQ + kTileBytes;            // 2 stages
    unsigned char* sV = sK + 2 * kTileBytes;        // 2 stages
    unsigned char* sP = sV + 2 * kTileBytes;        // 128 x 128 bf16, two K-major panels
    if (sP + 2 * kTileBytes > smem_dyn + kFwdSmemBytes) {       // dynamic shared memory base not 1024-byte aligned
        if (threadIdx.x == 0) set_status(P.status, VARDROP_ERR_CUDA);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5;
    if (warp == 0) {
        tmem_alloc(tmem_slot, kFwdTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv + 0, 1);
        mbar_init(bar_kv + 1, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    chain_wait();
    chain_release();
    // kept count of a selection shared by the batch: one broadcast load (per-instance selections take the maximum)
    const int kept_shared = P.n_sel ? (P.S > 1 ? -1 : __ldg(P.n_sel)) : P.N;
    const int n_t_max = ((P.S > 1 ? max_kept(P.n_sel, P.S, P.N, reinterpret_cast<int*>(smem_dyn + 48)) : kept_shared) + kTile - 1) / kTile;     // tiles of the longest selection
    const int n_items = n_t_max * P.H * P.B;                   // work items: (query tile, head, instance); short instances skip tiles
                                                               // (a CTA past the last item falls through the loop and frees its tensor memory)
    // two 128-column buffers: S of tile j lives in buffer j & 1; once the softmax has read it, P V of the same tile
    // lands in its first 64 columns while S of tile j + 1 is produced in the other buffer
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;

    constexpr uint32_t idesc_s = umma_idesc_bf16(128, 128, 0, 0);
    constexpr uint32_t idesc_o = umma_idesc_bf16(128, kDP, 0, 1);

    auto issue_scores = [&](uint32_t tmem_dst, const unsigned char* k_tile) {     // S = Q K^T, completion on bar_s
        const uint32_t a0 = smem_u32(sQ), b0 = smem_u32(k_tile);
#pragma unroll
        for (int ks = 0; ks < kDP / 16; ++ks)
            tc_mma_bf16(tmem_dst, umma_desc_sw128(a0 + ks * 32, 16, 1024), umma_desc_sw128(b0 + ks * 32, 16, 1024), idesc_s, ks > 0);
        tc_commit(bar_s);
    };

    bool ok = true;
    uint32_t kv_count = 0;      // K/V tiles consumed so far by this CTA: ring stage and barrier phase follow from it
    uint32_t n_done = 0;        // work items finished by this CTA (phase of bar_q)

    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const int qt = item % n_t_max;
        const int h = (item / n_t_max) % P.H;
        const int b = item / (n_t_max * P.H);
        const int srow = P.S > 1 ? b : 0;
        const int n_sel = P.S > 1 ? P.n_sel[srow] : kept_shared;       // kept tokens of this instance
        const int n_kv = (n_sel + kTile - 1) / kTile;          // its key tiles = query tiles
        if (qt >= n_kv) continue;
        TileSource src = P.src;
        if (src.idx) src.idx += static_cast<size_t>(srow) * P.N;
        {   // every MMA of the previous item has completed: Q and both ring stages are free.  Warps 0, 1, 2 fetch Q, K, V side
            // by side (each looks up its own gather rows); the byte counts are announced by thread 0, and a barrier phase
            // cannot complete before that arrival, whichever comes first.
            const uint32_t st0 = kv_count & 1;
            if (tid == 0) {
                mbar_expect_tx(bar_q, kTileBytes);
                mbar_expect_tx(bar_kv + st0, 2 * kTileBytes);
            }
            if (warp == 0) load_tile(sQ, &map_q, bar_q, src, qt * kTile, n_sel, h, b, P.H);
            else if (warp == 1) load_tile(sK + st0 * kTileBytes, &map_k, bar_kv + st0, src, 0, n_sel, h, b, P.H);
            else if (warp == 2) load_tile(sV + st0 * kTileBytes, &map_v, bar_kv + st0, src, 0, n_sel, h, b, P.H);
        }
        if (qt == 0 && tid == 0) P.tile_done[b * P.H + h] = 0;
        if (n_kv > 1) {             // the backward pass will add per-key-tile pieces of dQ' into the accumulator: clear this tile's rows
#pragma unroll
            for (int x = 0; x < kDP / 4; ++x) {          // 16 consecutive threads clear one 256-byte row
                const int idx = x * kFwdThreads + tid, r = idx >> 4, c4 = idx & 15;
                P.dq_acc[((static_cast<size_t>(b) * P.Ncap + qt * kTile + r) * P.H + h) * (kDP / 4) + c4] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }

        float o_acc[kDP];
#pragma unroll
        for (int d = 0; d < kDP; ++d) o_acc[d] = 0.f;
        float m_run = -INFINITY, l_run = 0.f, alpha = 0.f;

        for (int j = 0; j < n_kv; ++j, ++kv_count) {
            const uint32_t st = kv_count & 1;
            const uint32_t ph = kv_count & 1;            // bar_s / bar_o complete once per key tile
            if (j + 1 < n_kv) {                          // the other stage was released by the wait on bar_o of the previous tile
                if (tid == 0) mbar_expect_tx(bar_kv + (st ^ 1), 2 * kTileBytes);
                if (warp == 1) load_tile(sK + (st ^ 1) * kTileBytes, &map_k, bar_kv + (st ^ 1), src, (j + 1) * kTile, n_sel, h, b, P.H);
                else if (warp == 2) load_tile(sV + (st ^ 1) * kTileBytes, &map_v, bar_kv + (st ^ 1), src, (j + 1) * kTile, n_sel, h, b, P.H);
            }
            if (tid == 0) {
                if (j == 0) {                            // later tiles: issued right behind the previous tile's P V
                    ok &= mbar_wait(bar_q, n_done & 1);
                    ok &= mbar_wait(bar_kv + st, (kv_count >> 1) & 1);
                    tc_fence_after();
                    issue_scores(tmem + st * 128, sK + st * kTileBytes);
                }
            }
            const uint32_t tmem_s = tmem + st * 128;     // S of this tile; its first 64 columns are reused for P V
            const uint32_t tmem_o = tmem_s;
            ok &= mbar_wait(bar_s, ph);
            tc_fence_after();

            // ---- online softmax of this thread's query row over the 128 keys of the tile ------------------
            const int valid = min(kTile, n_sel - j * kTile);      // keys of this tile that exist
            float s[kTile];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tmem_s + lane_sel + c * 32, s + c * 32);
            tmem_ld_wait();
            if (valid < kTile) {                                  // ragged last tile: keys past n_sel never win the max
#pragma unroll
                for (int i = 0; i < kTile; ++i)
                    if (i >= valid) s[i] = -INFINITY;
            }
            float mx[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) mx[i] = s[i];
#pragma unroll
            for (int i = 8; i < kTile - 8; i += 16) {             // three-input maximum: two new values per instruction
#pragma unroll
                for (int u = 0; u < 8; ++u) mx[u] = max3(mx[u], s[i + u], s[i + 8 + u]);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) mx[u] = fmaxf(mx[u], s[kTile - 8 + u]);
            const float m_tile = fmaxf(max3(mx[0], mx[1], mx[2]), max3(max3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
            const float m_new = fmaxf(m_run, m_tile * P.scale_log2);
            alpha = fast_exp2(m_run - m_new);
            float l4[4];
            {
                const uint64_t scale2 = pair_of(P.scale_log2, P.scale_log2), shift2 = pair_of(-m_new, -m_new);
                uint64_t l2[2] = {pair_of(0.f, 0.f), pair_of(0.f, 0.f)};          // four running sums: keys i = 0..3 mod 4
#pragma unroll
                for (int i = 0; i < kTile; i += 2) {              // exp2(-inf) = 0 for the masked keys
                    float x0, x1;
                    halves_of(fma_pair(pair_of(s[i], s[i + 1]), scale2, shift2), x0, x1);
                    s[i] = fast_exp2(x0);
                    s[i + 1] = fast_exp2(x1);
                    l2[(i >> 1) & 1] = add_pair(l2[(i >> 1) & 1], pair_of(s[i], s[i + 1]));
                }
                halves_of(l2[0], l4[0], l4[1]);
                halves_of(l2[1], l4[2], l4[3]);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) store_row_chunk32(sP, tid, c * 32, s + c * 32);
            l_run = l_run * alpha + ((l4[0] + l4[1]) + (l4[2] + l4[3]));
            m_run = m_new;

            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                const uint32_t a0 = smem_u32(sP), b0 = smem_u32(sV + st * kTileBytes);
#pragma unroll
                for (int ks = 0; ks < kTile / 16; ++ks)
                    tc_mma_bf16(tmem_o, umma_desc_sw128(a0 + (ks >> 2) * kTileBytes + (ks & 3) * 32, 16, 1024),
                                umma_desc_sw128(b0 + ks * 2048, kTileBytes, 1024), idesc_o, ks > 0);
                tc_commit(bar_o);
                if (j + 1 < n_kv) {                      // scores of the next key tile queue up behind P V, in the other buffer
                    ok &= mbar_wait(bar_kv + (st ^ 1), ((kv_count + 1) >> 1) & 1);
                    tc_fence_after();
                    issue_scores(tmem + (st ^ 1) * 128, sK + (st ^ 1) * kTileBytes);
                }
            }
            ok &= mbar_wait(bar_o, ph);
            tc_fence_after();
#pragma unroll
            {
                float ov[kDP];
#pragma unroll
                for (int c = 0; c < kDP / 32; ++c) tmem_ld32(tmem_o + lane_sel + c * 32, ov + c * 32);
                tmem_ld_wait();
#pragma unroll
                for (int d = 0; d < kDP; d += 2)                                          // rescale and add in one step
                    halves_of(fma_pair(pair_of(o_acc[d], o_acc[d + 1]), pair_of(alpha, alpha), pair_of(ov[d], ov[d + 1])), o_acc[d], o_acc[d + 1]);
            }
            tc_fence_before();
            ok = __syncthreads_and(ok);                  // a wait gave up somewhere in the CTA: stop issuing work
            if (!ok) break;
        }

        const int row = qt * kTile + tid;
        if (ok && row < n_sel) {
            const float inv_l = 1.f / l_run;
            __nv_bfloat16* dst = P.o + ((static_cast<size_t>(b) * P.N + row) * P.H + h) * P.D;
#pragma unroll
            for (int q = 0; q < kDP / 8; ++q) {
                if (q * 8 < P.D) {
                    const uint4 w = make_uint4(pack_bf16(o_acc[8 * q + 0] * inv_l, o_acc[8 * q + 1] * inv_l),
                                               pack_bf16(o_acc[8 * q + 2] * inv_l, o_acc[8 * q + 3] * inv_l),
                                               pack_bf16(o_acc[8 * q + 4] * inv_l, o_acc[8 * q + 5] * inv_l),
                                               pack_bf16(o_acc[8 * q + 6] * inv_l, o_acc[8 * q + 7] * inv_l));
                    *reinterpret_cast<uint4*>(dst + 8 * q) = w;
                }
            }
            P.lse[(static_cast<size_t>(b) * P.H + h) * P.N + row] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
        ++n_done;
    }

    if (!ok) set_status(P.status, VARDROP_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kFwdTmemCols);
}

}  // namespace

int attn_fwd_launch(const void* q, const void* k, const void* v, const int32_t* sel_idx, const int32_t* n_sel,
                    const vardrop_attn_cfg& c, void* o, float* lse, void* ws, cudaStream_t stream) {
    const AttnWs w = attn_layout(c);
    char* base = static_cast<char*>(ws);
    const bool staged = attn_uses_staging(c, sel_idx);
    CUtensorMap mq, mk, mv;
    if (staged) {
        GatherParams G{};
        G.src[0] = static_cast<const uint4*>(q); G.src[1] = static_cast<const uint4*>(k); G.src[2] = static_cast<const uint4*>(v);
        G.dst[0] = reinterpret_cast<uint4*>(base + w.qg); G.dst[1] = reinterpret_cast<uint4*>(base + w.kg);
        G.dst[2] = reinterpret_cast<uint4*>(base + w.vg);
        G.sel_idx = sel_idx; G.n_sel = sel_idx ? n_sel : nullptr;
        G.N = c.N; G.Ncap = w.Ncap; G.H = c.H; G.D = c.D; G.S = attn_sel_rows(c);
        const long long work = static_cast<long long>(w.Ncap) * c.H * (kDP / 8);
        int gx = static_cast<int>((work + 255) / 256);
        const int cap = max(1, 4 * sm_count() / (3 * c.B));        // about four CTAs per SM in total; each strides over its rows
        if (gx > cap) gx = cap;
        cudaError_t gerr;
        { LaunchScope ls_(K_GATHER, stream); gerr = launch_chained(gather_kernel, dim3(gx, c.B, 3), dim3(256), 0, stream, G); }
        if (int st = check_cuda(gerr, "attention: gather launch")) return st;
        if (int st = make_tile_map(&mq, base + w.qg, c.B, w.Ncap, w.Ncap, c.H)) return st;
        if (int st = make_tile_map(&mk, base + w.kg, c.B, w.Ncap, w.Ncap, c.H)) return st;
        if (int st = make_tile_map(&mv, base + w.vg, c.B, w.Ncap, w.Ncap, c.H)) return st;
    } else if (attn_uses_gather(c, sel_idx)) {
        const long long rows = static_cast<long long>(c.B) * c.N * c.H;
        if (int st = make_row_map(&mq, q, rows)) return st;
        if (int st = make_row_map(&mk, k, rows)) return st;
        if (int st = make_row_map(&mv, v, rows)) return st;
    } else {
        if (int st = make_tile_map(&mq, q, c.B, c.N, c.N, c.H)) return st;
        if (int st = make_tile_map(&mk, k, c.B, c.N, c.N, c.H)) return st;
        if (int st = make_tile_map(&mv, v, c.B, c.N, c.N, c.H)) return st;
    }
    FwdParams P{};
    P.o = static_cast<__nv_bfloat16*>(o); P.lse = lse; P.n_sel = sel_idx ? n_sel : nullptr;
    P.status = reinterpret_cast<int*>(base);
    P.dq_acc = reinterpret_cast<float4*>(base + w.dq_acc);
    P.tile_done = reinterpret_cast<int32_t*>(base + w.tile_done);
    P.src.idx = sel_idx; P.src.gathered = attn_uses_gather(c, sel_idx) ? 1 : 0; P.src.tokens = c.N;
    P.src.rows_total = c.B * c.N * c.H;
    P.B = c.B; P.N = c.N; P.Ncap = w.Ncap; P.H = c.H; P.D = c.D; P.S = attn_sel_rows(c);
    const float scale = c.sm_scale > 0.f ? c.sm_scale : 1.f / sqrtf(static_cast<float>(c.D));
    P.scale_log2 = scale * 1.4426950408889634f;
    static thread_local int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFwdSmemBytes), "attention: smem attribute")) return st;
        attr_dev = dev;
    }
    cudaError_t err;
    {
        const long long worst = static_cast<long long>(w.Ncap / kTile) * c.H * c.B;
        const int grid = static_cast<int>(worst < 2ll * sm_count() ? worst : 2ll * sm_count());      // two CTAs fit per SM
        LaunchScope ls_(K_ATTN_FWD, stream);
        err = launch_chained(attn_fwd_kernel, dim3(grid), dim3(kFwdThreads), kFwdSmemBytes, stream, mq, mk, mv, P);
    }
    return check_cuda(err, "attention: forward launch");
}

}  // namespace vardrop
