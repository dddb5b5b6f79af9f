// Token gather and attention forward (Eq. 3) over the kept variate tokens.
//
// gather_kernel     compacts q/k/v rows named by sel_idx into [B, Ncap, H, 64] staging buffers with 16-byte
//                   copies, zero-pads D = 32 to 64 and zero-fills the ragged end of the last 128-token tile.
// attn_fwd_kernel   one persistent CTA per SM over (pair of 128-query tiles, head, instance): a load warp streams Q
//                   and a four-stage ring of K/V tiles, one thread issues S = Q K^T and O += P V on the tcgen05
//                   tensor cores (accumulators, and P itself, in tensor memory), and two softmax warpgroups, one per
//                   query tile of the pair and one thread per query row, turn S into P, so that one tile's
//                   exponentials run while the other tile's products do.
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
    long long aux[3];      // strides of a tile map (the key only carries a mix of them)
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

int make_tile_map(CUtensorMap* map, const void* base, int B, int tokens, int H, long long sB, long long sN, long long sH) {
    const MapKey key{base, sB * 131 + sN * 31 + sH, 1, B, tokens, H};
    MapSlot* slot = map_slot(key);
    if (slot->used && slot->key == key && slot->aux[0] == sB && slot->aux[1] == sN && slot->aux[2] == sH) { *map = slot->map; return VARDROP_OK; }
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled entry point not available");
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(kDP), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(tokens),
                                static_cast<cuuint64_t>(B)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(sH) * 2, static_cast<cuuint64_t>(sN) * 2, static_cast<cuuint64_t>(sB) * 2};
    const cuuint32_t box[4] = {kDP, 1, kTile, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r));
    slot->map = *map; slot->key = key; slot->used = true;
    slot->aux[0] = sB; slot->aux[1] = sN; slot->aux[2] = sH;
    return VARDROP_OK;
}

int make_row_map(CUtensorMap* map, const void* base, long long rows, long long row_stride_elems) {
    const MapKey key{base, rows, 2, static_cast<int>(row_stride_elems), 0, 0};
    MapSlot* slot = map_slot(key);
    if (slot->used && slot->key == key) { *map = slot->map; return VARDROP_OK; }
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(VARDROP_ERR_CUDA, "attention: cuTensorMapEncodeTiled entry point not available");
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(kDP), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(row_stride_elems) * 2};
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
    if (c.sB != 0 || c.sN != 0 || c.sH != 0) {
        if (c.sH < c.D || c.sN < c.sH || c.sB < c.sN || (c.sH | c.sN | c.sB) % 8 != 0)
            return fail(VARDROP_ERR_INVALID_ARG, "attention: strides sB=%lld sN=%lld sH=%lld must be multiples of 8 with sB >= sN >= sH >= D (or all 0)",
                        static_cast<long long>(c.sB), static_cast<long long>(c.sN), static_cast<long long>(c.sH));
        if (c.sB > (1ll << 38)) return fail(VARDROP_ERR_UNSUPPORTED, "attention: sB above 2^38 elements");
    }
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
    long long cB, cN, cH;     // strides of the sources in 16-byte chunks
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
    const uint4* src_b = P.src[t] + static_cast<size_t>(b) * P.cB;
    uint4* dst_b = P.dst[t] + static_cast<size_t>(b) * P.Ncap * chunks_row;
    // four chunks per thread and trip, a whole CTA apart, so that four independent row lookups and four 16-byte loads are in
    // flight per thread before the first store (one load per trip leaves the memory system idle most of the time)
    constexpr int U = 4;
    const int stride = gridDim.x * blockDim.x;
    for (int base = blockIdx.x * blockDim.x + threadIdx.x; base < total; base += U * stride) {
        const uint4* from[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * stride;
            from[u] = nullptr;
            if (idx < total) {
                const int j = idx / chunks_row;
                const int c = idx - j * chunks_row;
                const int h = c / (kDP / 8), dc = c - h * (kDP / 8);
                if (j < n_sel && dc < src_chunks_head) {
                    const int n = sel ? __ldg(sel + j) : j;
                    from[u] = src_b + static_cast<size_t>(n) * P.cN + static_cast<size_t>(h) * P.cH + dc;
                }
            }
        }
        uint4 val[U];
#pragma unroll
        for (int u = 0; u < U; ++u) val[u] = from[u] ? __ldg(from[u]) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * stride;
            if (idx < total) dst_b[idx] = val[u];
        }
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

// Roles of a CTA (one CTA per SM, persistent over work items = (four consecutive 128-query tiles, head, instance)):
//   warps 0, 1       issue the tensor-core products, warp 0 for softmax warpgroups 0 and 1, warp 1 for 2 and 3 (every lane runs
//                    the issue code so that operands stay in uniform registers, an elected lane executes each product); they come
//                    first because the warp schedulers favour the oldest ready warp and their short dependent chains sit on the
//                    critical path of the softmax warpgroups
//   warp 2           fetches Q, K, V tiles (TMA boxes or row gathers); warp 3 idles (it completes the register-donor warpgroup)
//   warps 4-19       four softmax warpgroups: warpgroup w owns query tile w of the item, one thread per query row
// Keys are processed 64 at a time: S_w (128 x 64, fp32) and O_w (128 x 64) of the four warpgroups fill the 512 columns of
// tensor memory, P_w (bf16) overlays the first 32 columns of S_w.  A warpgroup's chain per 64 keys is
//   S ready -> tensor-memory load -> row maximum -> exponentials -> P stored -> (issue warp) O += P V, next S = Q K^T -> S ready,
// a latency chain of a couple of thousand cycles of which the exponentials, the one throughput limit (16 per cycle and SM
// on the special-function units against 256 flop per score on the tensor cores at D = 64), are a quarter: four chains in
// flight keep those units busy where two could not.
constexpr int kFwdGroups = 4;
constexpr int kFwdGroupThreads = 128;
constexpr int kFwdThreads = (kFwdGroups + 1) * kFwdGroupThreads;
constexpr int kHalf = 64;                        // keys per softmax step
// Register split (setmaxnreg works on whole warpgroups): launched with 640 x 96 = 61440 registers; the softmax warpgroups
// take 104 a thread and the first warpgroup keeps 64: 512 x 104 + 128 x 64 = 61440.
constexpr int kFwdSoftmaxRegs = 104;
constexpr int kFwdOtherRegs = 64;
constexpr int kFwdStages = 3;                    // K/V ring (stages of one 128-key K tile and V tile)
constexpr uint32_t kFwdTmemCols = 512;           // per warpgroup w: S_w at column 128 w (P overlays its first 32), O_w at 128 w + 64
constexpr int kFwdSmemBytes = 1024 /*barriers + alignment*/ + kFwdGroups * kTileBytes /*Q tiles*/ + kFwdStages * 2 * kTileBytes /*K, V ring*/ +
                              kFwdGroups * kTileBytes /*O staging*/;
constexpr float kRescaleStep = 8.f;              // the reference maximum of a row moves only when the running maximum has grown by 2^8

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

// every lane of the warp waits; the result is the same in all of them
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(bar, parity)); }
// the same with a sleep between polls: for warps whose reaction time is not on the critical path
__device__ __forceinline__ bool warp_wait_relaxed(uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait_relaxed(bar, parity)); }

__global__ void __launch_bounds__(kFwdThreads, 1) attn_fwd_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                   const __grid_constant__ CUtensorMap map_k,
                                                                   const __grid_constant__ CUtensorMap map_v, const FwdParams P) {
    extern __shared__ unsigned char smem_dyn[];
    // Set-up first (shared-memory carve-up, barriers, tensor memory): it touches nothing another kernel produces, so it runs
    // while the previous kernel of the stream is still finishing.
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_dyn);     // barriers and the TMEM slot sit in front of the tiles
    uint64_t* bar_q_full = bars + 0;                // Q tiles of the item have landed
    uint64_t* bar_q_free = bars + 1;                // every S product of the item has completed: the Q buffers may be refilled (both issue warps)
    uint64_t* bar_kv_full = bars + 2;               // [kFwdStages]
    uint64_t* bar_kv_free = bar_kv_full + kFwdStages;  // [kFwdStages] every product reading the stage has completed (both issue warps)
    uint64_t* bar_s = bar_kv_free + kFwdStages;     // [4] S of warpgroup w's next 64 keys is in tensor memory
    uint64_t* bar_p = bar_s + kFwdGroups;           // [4] P of warpgroup w is in tensor memory (128 arrivals)
    uint64_t* bar_o = bar_p + kFwdGroups;           // [4] the last P V of the item has completed: O of warpgroup w is final
    uint64_t* bar_e = bar_o + kFwdGroups;           // [4] the O staging tile of warpgroup w is written (128 arrivals)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_e + kFwdGroups);
    int* s_scratch = reinterpret_cast<int*>(tmem_slot + 1);
    unsigned char* sQ = align_tiles(smem_dyn + 256);
    unsigned char* sK = sQ + kFwdGroups * kTileBytes;           // kFwdStages stages of (K tile, V tile)
    unsigned char* sOut = sK + kFwdStages * 2 * kTileBytes;     // one staging tile per warpgroup
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (sOut + kFwdGroups * kTileBytes > smem_dyn + kFwdSmemBytes) {     // dynamic shared memory base not 1024-byte aligned
        chain_wait();
        if (tid == 0) set_status(P.status, VARDROP_ERR_CUDA);
        return;
    }

    if (warp == 0) {
        tmem_alloc(tmem_slot, kFwdTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_free, 2);
        for (int st = 0; st < kFwdStages; ++st) {
            mbar_init(bar_kv_full + st, 1);
            mbar_init(bar_kv_free + st, 2);
        }
        for (int w = 0; w < kFwdGroups; ++w) {
            mbar_init(bar_s + w, 1);
            mbar_init(bar_p + w, kFwdGroupThreads);
            mbar_init(bar_o + w, 1);
            mbar_init(bar_e + w, kFwdGroupThreads);
        }
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
    if (blockIdx.x == 0 && threadIdx.x == 0) P.status[kWsPairingWord] = 1;      // this workspace now holds a forward pass that no backward pass has consumed
    // kept count of a selection shared by the batch: one broadcast load (per-instance selections take the maximum)
    const int kept_shared = P.n_sel ? (P.S > 1 ? -1 : __ldg(P.n_sel)) : P.N;
    const int n_t_max = ((P.S > 1 ? max_kept(P.n_sel, P.S, P.N, s_scratch) : kept_shared) + kTile - 1) / kTile;     // tiles of the longest selection
    const int n_quads = (n_t_max + kFwdGroups - 1) / kFwdGroups;       // query tiles are handled four at a time
    const int n_items = n_quads * P.H * P.B;                   // work items: (four query tiles, head, instance); short instances skip items
                                                               // (a CTA past the last item falls through its loops and frees its tensor memory)
    constexpr uint32_t idesc_o = umma_idesc_bf16(128, kDP, 0, 1);
    bool ok = true;

    // decode of a work item, the same in every role
    struct Item { int p, h, b, n_sel, n_kv, n_half, n_act; };
    auto decode = [&](int item) {
        Item it;
        it.p = item % n_quads;
        it.h = (item / n_quads) % P.H;
        it.b = item / (n_quads * P.H);
        it.n_sel = P.S > 1 ? P.n_sel[it.b] : kept_shared;      // kept tokens of this instance
        it.n_kv = (it.n_sel + kTile - 1) / kTile;              // its key tiles = query tiles
        it.n_half = (it.n_sel + kHalf - 1) / kHalf;            // its 64-key steps
        it.n_act = min(kFwdGroups, it.n_kv - kFwdGroups * it.p);   // query tiles of the item that exist (<= 0: skip the item)
        return it;
    };

    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kFwdOtherRegs));
    if (warp == 2) {
        // ---------------------------------------------------------------- loads ----------------------------------
        uint32_t kv_iter = 0, n_done = 0;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode(item);
            if (it.n_act <= 0) continue;
            TileSource src = P.src;
            if (src.idx) src.idx += static_cast<size_t>(P.S > 1 ? it.b : 0) * P.N;
            ok = warp_wait_relaxed(bar_q_free, (n_done & 1) ^ 1);
            if (!ok) break;
            if (lane == 0) mbar_expect_tx(bar_q_full, it.n_act * kTileBytes);
            for (int w = 0; w < it.n_act; ++w)
                load_tile(sQ + w * kTileBytes, &map_q, bar_q_full, src, (kFwdGroups * it.p + w) * kTile, it.n_sel, it.h, it.b, P.H);
            for (int j = 0; j < it.n_kv; ++j, ++kv_iter) {
                const uint32_t st = kv_iter % kFwdStages;
                ok = warp_wait_relaxed(bar_kv_free + st, ((kv_iter / kFwdStages) & 1) ^ 1);
                if (!ok) break;
                if (lane == 0) mbar_expect_tx(bar_kv_full + st, 2 * kTileBytes);
                load_tile(sK + st * 2 * kTileBytes, &map_k, bar_kv_full + st, src, j * kTile, it.n_sel, it.h, it.b, P.H);
                load_tile(sK + st * 2 * kTileBytes + kTileBytes, &map_v, bar_kv_full + st, src, j * kTile, it.n_sel, it.h, it.b, P.H);
            }
            ++n_done;
        }
    } else if (warp < 2) {
        // ---------------------------------------------------------------- tensor-core issue ----------------------
        // Issue warp `iw` serves warpgroups 2 iw and 2 iw + 1.  Both warps follow every K/V stage and release it with a commit of
        // their own (a commit with nothing outstanding arrives at once), so the release counts are fixed at two.
        const int iw = warp;
        uint32_t kv_iter = 0, n_done = 0, t_w[2] = {0, 0};
        // Operand descriptors are built once and stepped by additions.
        const uint64_t d_q = umma_desc_sw128(smem_u32(sQ), 16, 1024);                       // K-major: + 32 bytes per 16 head dimensions
        const uint64_t d_k = umma_desc_sw128(smem_u32(sK), 16, 1024);                       //          + 8192 bytes per 64 keys
        const uint64_t d_v = umma_desc_sw128(smem_u32(sK + kTileBytes), kTileBytes, 1024);  // MN-major: + 2048 bytes per 16 keys
        // S_w = Q_w K^T over the 64 keys of step `hh` of the stage; N = the key count of the step rounded up to 16
        auto issue_scores = [&](int w, uint32_t st, int hh, int n_cols) {
            const uint64_t a = umma_desc_advance(d_q, w * kTileBytes), bdesc = umma_desc_advance(d_k, st * 2 * kTileBytes + hh * (kHalf * kRowBytes));
            const uint32_t idesc = umma_idesc_bf16(128, n_cols, 0, 0);
            const uint32_t d_s = tmem + w * 128;
            tc_mma_bf16_w(d_s, a, bdesc, idesc, 0u);
            tc_mma_bf16_w(d_s, umma_desc_advance(a, 32), umma_desc_advance(bdesc, 32), idesc, 1u);
            tc_mma_bf16_w(d_s, umma_desc_advance(a, 64), umma_desc_advance(bdesc, 64), idesc, 1u);
            tc_mma_bf16_w(d_s, umma_desc_advance(a, 96), umma_desc_advance(bdesc, 96), idesc, 1u);
            tc_commit_w(bar_s + w);
        };
        // O_w (+)= P_w V over the step's keys: P is read from tensor memory (it overlays the first 32 columns of S_w), V from the stage
        auto issue_pv = [&](int w, uint32_t st, int hh, int k_steps, uint32_t acc) {
            const uint64_t bdesc = umma_desc_advance(d_v, st * 2 * kTileBytes + hh * 4 * 2048);
            const uint32_t d_o = tmem + w * 128 + 64, a_p = tmem + w * 128;
            if (k_steps == 4) {                     // the usual case, straight-line
                tc_mma_bf16_ta_w(d_o, a_p, bdesc, idesc_o, acc);
                tc_mma_bf16_ta_w(d_o, a_p + 8, umma_desc_advance(bdesc, 2048), idesc_o, 1u);
                tc_mma_bf16_ta_w(d_o, a_p + 16, umma_desc_advance(bdesc, 4096), idesc_o, 1u);
                tc_mma_bf16_ta_w(d_o, a_p + 24, umma_desc_advance(bdesc, 6144), idesc_o, 1u);
            } else {
                for (int ks = 0; ks < k_steps; ++ks)
                    tc_mma_bf16_ta_w(d_o, a_p + ks * 8, umma_desc_advance(bdesc, ks * 2048), idesc_o, ks > 0 ? 1u : acc);
            }
        };
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode(item);
            if (it.n_act <= 0) continue;
            const int n_w = max(0, min(2, it.n_act - 2 * iw));        // warpgroups of this issue warp that have a query tile
            ok &= warp_wait(bar_q_full, n_done & 1);
            for (int g = 0; g < it.n_half && ok; ++g) {
                const int j = g >> 1, hh = g & 1;
                const uint32_t st = (kv_iter + j) % kFwdStages;
                const int valid = min(kHalf, it.n_sel - g * kHalf);
                if (hh == 0) {
                    ok &= warp_wait(bar_kv_full + st, ((kv_iter + j) / kFwdStages) & 1);
                    tc_fence_after();
                }
                if (g == 0) {
                    for (int w = 0; w < n_w; ++w) issue_scores(2 * iw + w, st, 0, (valid + 15) & ~15);
                    if (it.n_half == 1) tc_commit_w(bar_q_free);
                }
                for (int w = 0; w < n_w && ok; ++w) {
                    ok &= warp_wait(bar_p + 2 * iw + w, t_w[w] & 1);
                    ++t_w[w];
                    tc_fence_after();
                    issue_pv(2 * iw + w, st, hh, (valid + 15) >> 4, g > 0);
                    if (g + 1 < it.n_half) {
                        const uint32_t st1 = (kv_iter + ((g + 1) >> 1)) % kFwdStages;
                        if (w == 0 && hh == 1) {         // the next step starts a new stage
                            ok &= warp_wait(bar_kv_full + st1, ((kv_iter + ((g + 1) >> 1)) / kFwdStages) & 1);
                            tc_fence_after();
                        }
                        issue_scores(2 * iw + w, st1, (g + 1) & 1, (min(kHalf, it.n_sel - (g + 1) * kHalf) + 15) & ~15);
                    } else {
                        tc_commit_w(bar_o + 2 * iw + w);
                    }
                }
                if (g + 2 == it.n_half) tc_commit_w(bar_q_free);                      // the last S products of the item are queued
                if (hh == 1 || g + 1 == it.n_half) tc_commit_w(bar_kv_free + st);     // every product reading the stage is queued
            }
            kv_iter += it.n_kv;
            ++n_done;
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kFwdSoftmaxRegs));
        // ---------------------------------------------------------------- softmax warpgroups ---------------------
        const int w = (warp >> 2) - 1;                  // query tile of the item
        const int r = tid & (kFwdGroupThreads - 1);     // query row inside the tile = tensor-memory lane
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tm_s = tmem + w * 128 + lane_sel, tm_o = tm_s + 64;
        unsigned char* stage = sOut + w * kTileBytes;
        uint32_t t_cnt = 0, n_done = 0;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode(item);
            if (w >= it.n_act) continue;
            const int qt = kFwdGroups * it.p + w;
            if (qt == 0 && r == 0) P.tile_done[it.b * P.H + it.h] = 0;
            if (it.n_kv > 1) {          // the backward pass will add per-key-tile pieces of dQ' into the accumulator: clear this tile's rows
#pragma unroll
                for (int x = 0; x < kDP / 4; ++x) {          // 16 consecutive threads clear one 256-byte row
                    const int idx = x * kFwdGroupThreads + r, rr = idx >> 4, c4 = idx & 15;
                    P.dq_acc[((static_cast<size_t>(it.b) * P.Ncap + qt * kTile + rr) * P.H + it.h) * (kDP / 4) + c4] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            float m_ref = -INFINITY, l_run = 0.f;       // exponentials are taken against m_ref (log2 domain), which trails the running maximum
            for (int g = 0; g < it.n_half; ++g, ++t_cnt) {
                ok = warp_wait_relaxed(bar_s + w, t_cnt & 1);
                if (!ok) break;
                tc_fence_after();
                const int valid = min(kHalf, it.n_sel - g * kHalf);      // keys of this step that exist
                float s[kHalf];
                tmem_ld32(tm_s, s);
                if (valid > 32) tmem_ld32(tm_s + 32, s + 32);
                tmem_ld_wait();
                if (valid < kHalf) {                                  // ragged last step: keys past n_sel never win the max
#pragma unroll
                    for (int i = 0; i < kHalf; ++i)
                        if (i >= valid) s[i] = -INFINITY;
                }
                float mx[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) mx[i] = s[i];
#pragma unroll
                for (int i = 4; i < kHalf - 4; i += 8) {              // three-input maximum: two new values per instruction
#pragma unroll
                    for (int u = 0; u < 4; ++u) mx[u] = max3(mx[u], s[i + u], s[i + 4 + u]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) mx[u] = fmaxf(mx[u], s[kHalf - 4 + u]);
                const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * P.scale_log2;
                if (g == 0) {
                    m_ref = m_tile;
                } else {
                    // O accumulates in tensor memory against m_ref.  It is rescaled only when a row's maximum has outgrown m_ref by
                    // 2^8 (probabilities then stay below 256, exact enough in bf16 and far from overflow); S of this step being
                    // complete implies P V of the previous step is, so O may be touched here.
                    const bool grow = m_tile > m_ref + kRescaleStep;
                    if (__any_sync(0xffffffffu, grow)) {
                        const float alpha = grow ? fast_exp2(m_ref - m_tile) : 1.f;
                        if (grow) m_ref = m_tile;
                        l_run *= alpha;
#pragma unroll 1
                        for (int c = 0; c < kDP; c += 16) {           // sixteen columns at a time: the scores stay in registers meanwhile
                            float ov[16];
                            tmem_ld16(tm_o + c, ov);
                            tmem_ld_wait();
#pragma unroll
                            for (int d = 0; d < 16; ++d) ov[d] *= alpha;
                            tmem_st16(tm_o + c, reinterpret_cast<const uint32_t*>(ov));
                        }
                    }
                }
                const uint64_t scale2 = pair_of(P.scale_log2, P.scale_log2), shift2 = pair_of(-m_ref, -m_ref);
                uint64_t l2[2] = {pair_of(0.f, 0.f), pair_of(0.f, 0.f)};          // four running sums: keys i = 0..3 mod 4
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    if (c * 32 < valid) {
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {             // exp2(-inf) = 0 for the masked keys
                            float x0, x1;
                            halves_of(fma_pair(pair_of(s[c * 32 + i], s[c * 32 + i + 1]), scale2, shift2), x0, x1);
                            const float e0 = fast_exp2(x0), e1 = fast_exp2(x1);
                            l2[(i >> 1) & 1] = add_pair(l2[(i >> 1) & 1], pair_of(e0, e1));
                            pk[i >> 1] = pack_bf16(e0, e1);
                        }
                        tmem_st16(tm_s + c * 16, pk);                 // P overlays S: key 2 c' and 2 c' + 1 in column c'
                    }
                }
                {
                    float a0, a1, a2, a3;
                    halves_of(l2[0], a0, a1);
                    halves_of(l2[1], a2, a3);
                    l_run += (a0 + a1) + (a2 + a3);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_p + w);
            }
            if (!ok) break;
            // ---- epilogue: O / l, rounded to bf16, through a staging tile so that whole 128-byte rows are written -------------
            ok = warp_wait_relaxed(bar_o + w, n_done & 1);
            if (!ok) break;
            tc_fence_after();
            {
                const float inv_l = 1.f / l_run;
                unsigned char* rowp = stage + r * kRowBytes;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    float ov[32];
                    tmem_ld32(tm_o + hf * 32, ov);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4*>(rowp + (((hf * 4 + q) ^ (r & 7)) << 4)) =
                            make_uint4(pack_bf16(ov[8 * q + 0] * inv_l, ov[8 * q + 1] * inv_l), pack_bf16(ov[8 * q + 2] * inv_l, ov[8 * q + 3] * inv_l),
                                       pack_bf16(ov[8 * q + 4] * inv_l, ov[8 * q + 5] * inv_l), pack_bf16(ov[8 * q + 6] * inv_l, ov[8 * q + 7] * inv_l));
                }
                const int row = qt * kTile + r;
                if (row < it.n_sel) P.lse[(static_cast<size_t>(it.b) * P.H + it.h) * P.N + row] = (m_ref + log2f(l_run)) * 0.6931471805599453f;
            }
            tc_fence_before();
            mbar_arrive(bar_e + w);
            ok = warp_wait_relaxed(bar_e + w, n_done & 1);
            if (!ok) break;
            {
                const int c = r & 7;
                if (c * 8 < P.D) {
                    for (int rr = r >> 3; rr < kTile; rr += kFwdGroupThreads / 8) {
                        const int row = qt * kTile + rr;
                        if (row >= it.n_sel) break;
                        *reinterpret_cast<uint4*>(P.o + ((static_cast<size_t>(it.b) * P.N + row) * P.H + it.h) * P.D + c * 8) =
                            *reinterpret_cast<const uint4*>(stage + rr * kRowBytes + ((c ^ (rr & 7)) << 4));
                    }
                }
            }
            ++n_done;
        }
    }

    if (!ok) set_status(P.status, VARDROP_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kFwdTmemCols);
}

// ---------------------------------------------------------------------------------------------------------
// forward, few tiles: one query tile per CTA, two CTAs per SM
// ---------------------------------------------------------------------------------------------------------
// With only a few work items per SM (the kept sets of the paper's workloads: one or two tiles per head and instance) the step is
// a chain of latencies and what counts is how many independent (query tile, head, instance) items are in flight: this kernel runs
// one item per 128-thread CTA, two CTAs per SM, and keeps P in shared memory.  The four-warpgroup kernel above takes over
// when there are enough query tiles to fill its groups of four.
constexpr int kTileFwdThreads = 128;
constexpr uint32_t kTileFwdTmemCols = 256;
constexpr int kTileFwdSmemBytes = 1024 /*barriers + alignment*/ + kTileBytes /*Q*/ + 2 * kTileBytes /*K*/ + 2 * kTileBytes /*V*/ + 2 * kTileBytes /*P*/;

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

__global__ void __launch_bounds__(kTileFwdThreads) attn_fwd_tile_kernel(const __grid_constant__ CUtensorMap map_q,
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
    if (sP + 2 * kTileBytes > smem_dyn + kTileFwdSmemBytes) {       // dynamic shared memory base not 1024-byte aligned
        chain_wait();
        if (threadIdx.x == 0) set_status(P.status, VARDROP_ERR_CUDA);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5;
    if (warp == 0) {
        tmem_alloc(tmem_slot, kTileFwdTmemCols);
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
    if (blockIdx.x == 0 && threadIdx.x == 0) P.status[kWsPairingWord] = 1;      // this workspace now holds a forward pass that no backward pass has consumed
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
                const int idx = x * kTileFwdThreads + tid, r = idx >> 4, c4 = idx & 15;
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
    if (warp == 0) tmem_dealloc(tmem, kTileFwdTmemCols);
}


}  // namespace

// Which forward kernel: the kept count is only known on the device, so the host goes by the largest it can be.  A selection
// keeps a fraction of the variates (a tenth to a third in the paper's settings); up to 2048 variates that is a handful of tiles
// per head and instance.  Without a selection every token is kept.
static bool attn_fwd_uses_groups(const vardrop_attn_cfg& c, const int32_t* sel_idx) { return sel_idx ? c.N > 2048 : c.N > 2 * kTile; }

int attn_fwd_launch(const void* q, const void* k, const void* v, const int32_t* sel_idx, const int32_t* n_sel,
                    const vardrop_attn_cfg& c, void* o, float* lse, void* ws, cudaStream_t stream) {
    const AttnWs w = attn_layout(c);
    const QkvLayout L = qkv_layout(c);
    char* base = static_cast<char*>(ws);
    const bool staged = attn_uses_staging(c, sel_idx);
    const long long Hd = static_cast<long long>(c.H) * kDP;          // staged copies: [B, Ncap, H, 64] contiguous
    CUtensorMap mq, mk, mv;
    if (staged) {
        GatherParams G{};
        G.src[0] = static_cast<const uint4*>(q); G.src[1] = static_cast<const uint4*>(k); G.src[2] = static_cast<const uint4*>(v);
        G.dst[0] = reinterpret_cast<uint4*>(base + w.qg); G.dst[1] = reinterpret_cast<uint4*>(base + w.kg);
        G.dst[2] = reinterpret_cast<uint4*>(base + w.vg);
        G.sel_idx = sel_idx; G.n_sel = sel_idx ? n_sel : nullptr;
        G.N = c.N; G.Ncap = w.Ncap; G.H = c.H; G.D = c.D; G.S = attn_sel_rows(c);
        G.cB = L.sB / 8; G.cN = L.sN / 8; G.cH = L.sH / 8;
        const long long work = static_cast<long long>(w.Ncap) * c.H * (kDP / 8);
        int gx = static_cast<int>((work + 255) / 256);
        const int cap = max(1, 8 * sm_count() / (3 * c.B));        // about eight CTAs per SM in total (the kept count is only known on the
                                                                   // device: a grid sized for every variate would be mostly empty CTAs)
        if (gx > cap) gx = cap;
        cudaError_t gerr;
        { LaunchScope ls_(K_GATHER, stream); gerr = launch_chained(gather_kernel, dim3(gx, c.B, 3), dim3(256), 0, stream, G); }
        if (int st = check_cuda(gerr, "attention: gather launch")) return st;
        if (int st = make_tile_map(&mq, base + w.qg, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
        if (int st = make_tile_map(&mk, base + w.kg, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
        if (int st = make_tile_map(&mv, base + w.vg, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
    } else if (attn_uses_gather(c, sel_idx)) {
        if (int st = make_row_map(&mq, q, L.rows_total, L.sH)) return st;
        if (int st = make_row_map(&mk, k, L.rows_total, L.sH)) return st;
        if (int st = make_row_map(&mv, v, L.rows_total, L.sH)) return st;
    } else {
        if (int st = make_tile_map(&mq, q, c.B, c.N, c.H, L.sB, L.sN, L.sH)) return st;
        if (int st = make_tile_map(&mk, k, c.B, c.N, c.H, L.sB, L.sN, L.sH)) return st;
        if (int st = make_tile_map(&mv, v, c.B, c.N, c.H, L.sB, L.sN, L.sH)) return st;
    }
    FwdParams P{};
    P.o = static_cast<__nv_bfloat16*>(o); P.lse = lse; P.n_sel = sel_idx ? n_sel : nullptr;
    P.status = reinterpret_cast<int*>(base);
    P.dq_acc = reinterpret_cast<float4*>(base + w.dq_acc);
    P.tile_done = reinterpret_cast<int32_t*>(base + w.tile_done);
    P.src.idx = sel_idx; P.src.gathered = attn_uses_gather(c, sel_idx) ? 1 : 0; P.src.tokens = c.N;
    P.src.rows_total = static_cast<int>(L.rows_total); P.src.row_b = static_cast<int>(L.row_b); P.src.row_n = static_cast<int>(L.row_n);
    P.B = c.B; P.N = c.N; P.Ncap = w.Ncap; P.H = c.H; P.D = c.D; P.S = attn_sel_rows(c);
    const float scale = c.sm_scale > 0.f ? c.sm_scale : 1.f / sqrtf(static_cast<float>(c.D));
    P.scale_log2 = scale * 1.4426950408889634f;
    static thread_local int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFwdSmemBytes), "attention: smem attribute")) return st;
        if (int st = check_cuda(cudaFuncSetAttribute(attn_fwd_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileFwdSmemBytes), "attention: smem attribute")) return st;
        attr_dev = dev;
    }
    cudaError_t err;
    if (attn_fwd_uses_groups(c, sel_idx)) {
        const long long worst = static_cast<long long>((w.Ncap / kTile + kFwdGroups - 1) / kFwdGroups) * c.H * c.B;       // groups of four query tiles
        const int grid = static_cast<int>(worst < sm_count() ? worst : sm_count());                 // one CTA per SM
        LaunchScope ls_(K_ATTN_FWD, stream);
        err = launch_chained(attn_fwd_kernel, dim3(grid), dim3(kFwdThreads), kFwdSmemBytes, stream, mq, mk, mv, P);
    } else {
        const long long worst = static_cast<long long>(w.Ncap / kTile) * c.H * c.B;
        const int grid = static_cast<int>(worst < 2ll * sm_count() ? worst : 2ll * sm_count());      // two CTAs fit per SM
        LaunchScope ls_(K_ATTN_FWD, stream);
        err = launch_chained(attn_fwd_tile_kernel, dim3(grid), dim3(kTileFwdThreads), kTileFwdSmemBytes, stream, mq, mk, mv, P);
    }
    return check_cuda(err, "attention: forward launch");
}

}  // namespace vardrop
