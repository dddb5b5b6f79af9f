// Attention backward over the kept variate tokens and the scatter of the gradients to the full layout.
//
// bwd_prep_kernel    Delta_i = sum_d dO'_id O'_id and a zero-filled staged copy of dO' (rows past n_sel may hold
//                    anything in the caller's buffer).  The fp32 dQ' accumulator is cleared by the forward kernel.
// attn_bwd_kernel    one persistent CTA per SM (384 threads: 256 workers and a third warpgroup whose first thread issues
//                    the products) over (128-key tile, head, instance), looping over the query tiles.  Scores are
//                    formed transposed (S^T = K Q^T, dP^T = V dO^T) so that two workers own each key row of tensor
//                    memory; P^T and dS^T are written to shared memory once and feed three tensor-core products:
//                    dV += P^T dO, dK += dS^T Q (accumulated in tensor memory across the query loop) and
//                    dQ_i = dS K (added into the fp32 accumulator by bulk reduce-adds).
//                    The same kernel writes the zero rows of every dropped variate (by a warp that is off the critical
//                    path, a slice ahead of every query tile) and, when the CTA that finishes the last key tile of an (instance, head) pair sees the
//                    pair complete, converts that pair's dQ' accumulator to bf16 rows of dq: each row of dq / dk / dv
//                    is written exactly once and no further launch is needed.
#include "attn_common.cuh"

namespace vardrop {

namespace {

__device__ __forceinline__ uint32_t pack2(float a, float b) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w));
}

// ---------------------------------------------------------------------------------------------------------
// prep
// ---------------------------------------------------------------------------------------------------------
struct PrepParams {
    const uint4* o;       // [B, N, H, D] bf16
    const uint4* d_o;     // [B, N, H, D] bf16
    uint4* dog;           // [B, Ncap, H, 64] bf16 staged dO (NULL: not needed)
    float* delta;         // [B, H, Ncap]
    float4* dq_acc;       // [B, Ncap, H, 64] fp32
    const int32_t* n_sel; // [S] kept counts; NULL: N
    int N, Ncap, H, D, S;
};

// one thread per 16-byte chunk of a staged (token, head) row; the 8 threads of a row reduce Delta by shuffles
__global__ void __launch_bounds__(256) bwd_prep_kernel(const PrepParams P) {
    chain_wait();
    chain_release();
    const int b = blockIdx.y;
    const int n_sel = P.n_sel ? P.n_sel[P.S > 1 ? b : 0] : P.N;
    if (!P.dog && n_sel <= kTile) return;            // a single key tile: the main kernel computes Delta itself
    const int n_fill = min(P.Ncap, (n_sel + kTile - 1) / kTile * kTile);
    const int chunks_row = P.H * 8;
    const int src_chunks_head = P.D / 8;
    const int total = n_fill * chunks_row;            // a multiple of 8; blockDim is a multiple of 8
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int i = idx / chunks_row;
        const int c = idx - i * chunks_row;
        const int h = c >> 3, dc = c & 7;
        uint4 vo = make_uint4(0u, 0u, 0u, 0u), vd = vo;
        if (i < n_sel && dc < src_chunks_head) {
            const size_t src = (static_cast<size_t>(b) * P.N + i) * (P.H * src_chunks_head) + h * src_chunks_head + dc;
            vo = __ldg(P.o + src);
            vd = __ldg(P.d_o + src);
        }
        const float2 a0 = unpack2(vo.x), a1 = unpack2(vo.y), a2 = unpack2(vo.z), a3 = unpack2(vo.w);
        const float2 g0 = unpack2(vd.x), g1 = unpack2(vd.y), g2 = unpack2(vd.z), g3 = unpack2(vd.w);
        float part = a0.x * g0.x + a0.y * g0.y + a1.x * g1.x + a1.y * g1.y + a2.x * g2.x + a2.y * g2.y + a3.x * g3.x + a3.y * g3.y;
        part += __shfl_xor_sync(0xffffffffu, part, 1);
        part += __shfl_xor_sync(0xffffffffu, part, 2);
        part += __shfl_xor_sync(0xffffffffu, part, 4);
        if (P.delta && dc == 0) P.delta[(static_cast<size_t>(b) * P.H + h) * P.Ncap + i] = part;
        const size_t dst = (static_cast<size_t>(b) * P.Ncap + i) * chunks_row + c;
        if (P.dog) P.dog[dst] = vd;
        if (P.dq_acc && n_sel > kTile) {              // a single key tile writes dq directly, nothing to accumulate
            P.dq_acc[2 * dst] = make_float4(0.f, 0.f, 0.f, 0.f);
            P.dq_acc[2 * dst + 1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// main
// ---------------------------------------------------------------------------------------------------------
struct BwdParams {
    const float* lse;       // [B, H, N]
    const __nv_bfloat16* o; // [B, N, H, D] forward output (rows 0 .. n_sel-1), for Delta
    const float* delta;     // [B, H, Ncap] precomputed Delta, or NULL: computed here from o and dO
    TileSource src;         // where Q, K, V tiles come from
    TileSource src_do;      // where dO tiles come from
    float* dq_acc;          // [B, Ncap, H, 64]
    __nv_bfloat16* dq;      // [B, N, H, D]; written here only when there is a single key tile
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    const int32_t* sel_idx; // [S, N]; NULL: identity
    const int32_t* inv_idx; // [S, N]; NULL: identity (nothing dropped)
    int32_t* tile_done;     // [B, H] key tiles finished per (instance, head); zeroed by the forward pass
    int convert_here;       // 1: the CTA that completes an (instance, head) pair converts its dQ' accumulator to dq rows
                            // 0: a separate kernel does (many tiles: the conversion wants the whole GPU)
    const int32_t* n_sel;   // [S]; NULL: N
    int* status;
    int B, N, Ncap, H, D, S;
    float scale, scale_log2;
};

constexpr int kBwdWorkers = 256;       // two threads per tensor-memory lane: each takes one 64-column half
constexpr int kBwdThreads = kBwdWorkers + 128; // plus a third warpgroup: its first warp's first lane issues every tensor-core product,
                                               // the rest of it only gives its registers to the workers
// Register split (setmaxnreg works on whole warpgroups): the kernel is launched with 384 x 168 = 64512 registers; the
// third warpgroup keeps 152 a thread and the two worker warpgroups take 176: 256 x 176 + 128 x 152 = 64512 (with less than
// 152 the third warpgroup, which also takes dQ out of tensor memory, spills).
constexpr int kBwdWorkerRegs = 176;
constexpr int kBwdIssuerRegs = 152;
constexpr uint32_t kBwdTmemCols = 512;
constexpr int kQStages = 3;            // ring of query-tile operands (Q and dO), fetched two tiles ahead
constexpr int kBwdSmemBytes = 3072 /*barriers, row statistics, alignment*/ + 2 * kTileBytes /*K, V*/ + 2 * kQStages * kTileBytes /*Q, dO ring*/ +
                              4 * kTileBytes /*P^T, dS^T*/ + 2 * kTileBytes /*dQ tile, fp32, two 32-column halves*/;     // 227 KiB: all an SM offers a CTA

// barrier among the worker threads only (the issuing warp never joins it)
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kBwdWorkers) : "memory"); }
__device__ __forceinline__ bool worker_sync_and(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\n"
        "setp.ne.b32 q, %1, 0;\n"
        "bar.red.and.pred p, 1, %2, q;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(ok)), "n"(kBwdWorkers)
        : "memory");
    return r != 0;
}

// the same for the third warpgroup (128 threads, barrier 2)
__device__ __forceinline__ void group3_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }
__device__ __forceinline__ bool group3_sync_and(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\n"
        "setp.ne.b32 q, %1, 0;\n"
        "bar.red.and.pred p, 2, 128, q;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(ok))
        : "memory");
    return r != 0;
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
__device__ __forceinline__ uint64_t mul_pair(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// every lane of the warp waits; the result is the same in all of them
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(bar, parity)); }
// the same with a sleep between polls: for warps whose reaction time is not on the critical path
__device__ __forceinline__ bool warp_wait_relaxed(uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait_relaxed(bar, parity)); }

__device__ __forceinline__ float fast_exp2(float x) {      // special-function unit; exp2(-inf) = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 16 consecutive columns (c0 a multiple of 16) of row r of a 128 x 128 bf16 tile stored as two 64-column panels
// (128-byte swizzled rows)
__device__ __forceinline__ void store_chunk16(unsigned char* tile, int r, int c0, const float* v) {
    unsigned char* panel = tile + (c0 >> 6) * kTileBytes + r * kRowBytes;
    const int chunk0 = (c0 & 63) >> 3;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const uint4 w = make_uint4(pack2(v[8 * q + 0], v[8 * q + 1]), pack2(v[8 * q + 2], v[8 * q + 3]), pack2(v[8 * q + 4], v[8 * q + 5]),
                                   pack2(v[8 * q + 6], v[8 * q + 7]));
        *reinterpret_cast<uint4*>(panel + (((chunk0 + q) ^ (r & 7)) << 4)) = w;
    }
}

// Zero rows of dq, dk, dv for every dropped variate, by one warp of the CTA that is off the critical path, so that the zeros
// are written beside the products instead of in front of them.  The rows of all instances are dealt to the CTAs in rounds of
// 32: in round k the warp of CTA c looks rows (c + k gridDim.x) 32 .. + 31 up in inv_idx, one a lane, and writes the dropped
// ones, 512 bytes a store instruction.
__device__ __forceinline__ int zero_row_rounds(const BwdParams& P) {
    return P.inv_idx ? (P.B * P.N + static_cast<int>(gridDim.x) * 32 - 1) / (static_cast<int>(gridDim.x) * 32) : 0;
}
__device__ __forceinline__ void zero_rows_round(const BwdParams& P, int round) {
    const int lane = threadIdx.x & 31;
    const int chunks_row = P.H * (P.D / 8);                    // 16-byte chunks per (instance, variate) row
    const int total_rows = P.B * P.N;
    const int base = (static_cast<int>(blockIdx.x) + round * static_cast<int>(gridDim.x)) * 32;
    const int r = base + lane;
    bool dropped = false;
    if (r < total_rows) {
        const int b = r / P.N, n = r - b * P.N;
        dropped = __ldg(P.inv_idx + static_cast<size_t>(P.S > 1 ? b : 0) * P.N + n) < 0;
    }
    unsigned mask = __ballot_sync(0xffffffffu, dropped);
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    uint4* dq4 = reinterpret_cast<uint4*>(P.dq);
    uint4* dk4 = reinterpret_cast<uint4*>(P.dk);
    uint4* dv4 = reinterpret_cast<uint4*>(P.dv);
    while (mask) {
        const int l = __ffs(mask) - 1;
        mask &= mask - 1;
        const size_t row0 = static_cast<size_t>(base + l) * chunks_row;
        for (int c = lane; c < chunks_row; c += 32) { dq4[row0 + c] = z; dk4[row0 + c] = z; dv4[row0 + c] = z; }
    }
}

__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                   const __grid_constant__ CUtensorMap map_k,
                                                                   const __grid_constant__ CUtensorMap map_v,
                                                                   const __grid_constant__ CUtensorMap map_do,
                                                                   const __grid_constant__ CUtensorMap map_acc, const BwdParams P) {
    extern __shared__ unsigned char smem_dyn[];
    // Set-up first (shared-memory carve-up, barriers, tensor memory): it touches nothing another kernel produces, so it runs
    // while the previous kernel of the stream is still finishing.
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_dyn);
    uint64_t* bar_kv = bars + 0;
    uint64_t* bar_qdo = bars + 1;                   // [3]
    uint64_t* bar_s = bars + 4;                     // S^T of a query tile complete
    uint64_t* bar_dp = bars + 5;                    // dP^T of a query tile complete (and every product issued before it)
    uint64_t* bar_g = bars + 6;                     // dQ of a query tile complete
    uint64_t* bar_acc = bars + 7;                   // every product of the item complete: dV, dK final, operands free
    uint64_t* bar_p = bars + 8;                     // P^T of a query tile written by every worker thread
    uint64_t* bar_ds = bars + 9;                    // dS^T of a query tile written by every worker thread
    uint64_t* bar_conv = bars + 10;                 // the "last key tile of its (instance, head)" flag of an item is written
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_dyn + 96);
    float* s_stat = reinterpret_cast<float*>(smem_dyn + 128);     // [3 stages][128] minus the lse of the query tile, log2 domain
    float* s_dpart = s_stat + kQStages * kTile;                   // [2][128] Delta of the query tile: with precomputed Delta, one array per
                                                                  // tile parity (written a barrier ahead of its use); otherwise the two
                                                                  // halves' partial sums over 32 head dimensions of dO O
    unsigned char* sK = align_tiles(smem_dyn + 128 + (kQStages + 2) * kTile * sizeof(float));
    unsigned char* sV = sK + kTileBytes;
    unsigned char* sQ = sV + kTileBytes;            // 3 stages
    unsigned char* sdO = sQ + kQStages * kTileBytes;   // 3 stages
    unsigned char* sPt = sdO + kQStages * kTileBytes;  // P^T  : rows = keys, columns = queries (two 64-query panels)
    unsigned char* sdSt = sPt + 2 * kTileBytes;     // dS^T : same shape
    unsigned char* sDQ = sdSt + 2 * kTileBytes;     // dQ_i as fp32: panel `half` = head dimensions 32 half .. 32 half + 31, 128-byte swizzled rows
    if (sDQ + 2 * kTileBytes > smem_dyn + kBwdSmemBytes) {
        chain_wait();
        if (threadIdx.x == 0) set_status(P.status, VARDROP_ERR_CUDA);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5;
    const int row = tid & (kTile - 1);              // tensor-memory lane this thread reads
    const int half = tid >> 7;                      // which 64-column half of the lane
    if (warp == 0) {
        tmem_alloc(tmem_slot, kBwdTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_kv, 1);
        for (int st = 0; st < kQStages; ++st) mbar_init(bar_qdo + st, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_dp, 1);
        mbar_init(bar_g, 1);
        mbar_init(bar_acc, 1);
        mbar_init(bar_p, kBwdWorkers);
        mbar_init(bar_ds, kBwdWorkers);
        mbar_init(bar_conv, 1);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
        tma_prefetch_desc(&map_do);
        tma_prefetch_desc(&map_acc);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    chain_wait();
    chain_release();
    // One backward pass per forward pass: the forward kernel cleared this workspace's dQ' accumulator and tile counters and left a
    // mark; a backward pass that does not find the mark (a second backward for the same forward, or two forwards sharing the
    // workspace before their backwards) would add into stale state, so it reports the call instead of returning wrong gradients.
    if (blockIdx.x == 0 && threadIdx.x == 0 && atomicExch(P.status + kWsPairingWord, 0) != 1) set_status(P.status, VARDROP_ERR_INVALID_ARG);
    // kept count of a selection shared by the batch: one broadcast load (per-instance selections take the maximum)
    const int kept_shared = P.n_sel ? (P.S > 1 ? -1 : __ldg(P.n_sel)) : P.N;
    const int n_t_max = ((P.S > 1 ? max_kept(P.n_sel, P.S, P.N, reinterpret_cast<int*>(smem_dyn + 100)) : kept_shared) + kTile - 1) / kTile;     // tiles of the longest selection
    const int n_items = n_t_max * P.H * P.B;                   // work items: (key tile, head, instance); short instances skip tiles
    // Zero rows of dq, dk, dv for every dropped variate: the last warp of the third warpgroup, which only helps with taking dQ out
    // of tensor memory, writes a slice of its CTA's share ahead of every query tile (see zero_rows_round) and the rest at the end.
    const bool zero_warp = warp == kBwdThreads / 32 - 1 && P.inv_idx != nullptr;
    // (a CTA past the last item runs no loop below: it writes its share of the zero rows and frees its tensor memory)

    const uint32_t tm_st = tmem;            // [0,128)   S^T
    const uint32_t tm_dpt = tmem + 128;     // [128,256) dP^T
    const uint32_t tm_dv = tmem + 256;      // [256,320) dV
    const uint32_t tm_dk = tmem + 320;      // [320,384) dK
    const uint32_t tm_dq = tmem + 384;      // [384,448) dQ of the current query tile
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;

    constexpr uint32_t idesc_kk = umma_idesc_bf16(128, 128, 0, 0);     // K-major x K-major, N = 128
    constexpr uint32_t idesc_kmn = umma_idesc_bf16(128, kDP, 0, 1);    // A K-major, B MN-major, N = 64
    constexpr uint32_t idesc_mnmn = umma_idesc_bf16(128, kDP, 1, 1);   // A MN-major, B MN-major, N = 64

    int n_sel = P.N;            // kept tokens of the instance being processed (set per work item)
    bool use_delta = false;     // precomputed Delta in use for this instance
    bool ok = true;
    uint32_t q_count = 0;       // query tiles consumed so far by this CTA: ring stage = q_count mod 3
    uint32_t n_done = 0;        // work items finished by this CTA (phase of bar_kv)
    uint32_t n_conv = 0;        // items whose "last key tile" flag has been read (phase of bar_conv)

    // operand descriptors, built once and stepped by additions: K-major views for the scores and the P^T / dS^T panels,
    // MN-major views where the reduction runs over the rows of the tile
    // (every tile sits at a fixed distance from the K tile, so two descriptors of the K tile and constant steps give them all)
    const uint64_t d_k = umma_desc_sw128(smem_u32(sK), 16, 1024), m_k = umma_desc_sw128(smem_u32(sK), kTileBytes, 1024);
    const uint64_t d_v = umma_desc_advance(d_k, kTileBytes);
    const uint64_t d_q0 = umma_desc_advance(d_k, 2 * kTileBytes), d_do0 = umma_desc_advance(d_k, (2 + kQStages) * kTileBytes);
    const uint64_t d_pt = umma_desc_advance(d_k, (2 + 2 * kQStages) * kTileBytes), d_dst = umma_desc_advance(d_k, (4 + 2 * kQStages) * kTileBytes);
    const uint64_t m_q0 = umma_desc_advance(m_k, 2 * kTileBytes), m_do0 = umma_desc_advance(m_k, (2 + kQStages) * kTileBytes);
    const uint64_t m_dst = umma_desc_advance(m_k, (4 + 2 * kQStages) * kTileBytes);
    // The five products of a (key tile, query tile) pair, each issued by one thread.  S^T = K Q^T and dP^T = V dO^T read the
    // query tile in ring stage `stage`; dV += P^T dO and dK += dS^T Q accumulate over the query loop; dQ_i = dS K.
    auto issue_st = [&](uint32_t stage) {
        const uint64_t dq_ = umma_desc_advance(d_q0, stage * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kDP / 16; ++ks)
            tc_mma_bf16(tm_st, umma_desc_advance(d_k, ks * 32), umma_desc_advance(dq_, ks * 32), idesc_kk, ks > 0);
        tc_commit(bar_s);
    };
    auto issue_dpt = [&](uint32_t stage) {
        const uint64_t dd_ = umma_desc_advance(d_do0, stage * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kDP / 16; ++ks)
            tc_mma_bf16(tm_dpt, umma_desc_advance(d_v, ks * 32), umma_desc_advance(dd_, ks * 32), idesc_kk, ks > 0);
        tc_commit(bar_dp);
    };
    auto issue_dv = [&](uint32_t stage, uint32_t acc_on) {           // reduction over the 128 queries
        const uint64_t mdo = umma_desc_advance(m_do0, stage * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kTile / 16; ++ks)
            tc_mma_bf16(tm_dv, umma_desc_advance(d_pt, (ks >> 2) * kTileBytes + (ks & 3) * 32), umma_desc_advance(mdo, ks * 2048), idesc_kmn,
                        ks > 0 ? 1u : acc_on);
    };
    auto issue_dk = [&](uint32_t stage, uint32_t acc_on) {
        const uint64_t mq = umma_desc_advance(m_q0, stage * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kTile / 16; ++ks)
            tc_mma_bf16(tm_dk, umma_desc_advance(d_dst, (ks >> 2) * kTileBytes + (ks & 3) * 32), umma_desc_advance(mq, ks * 2048), idesc_kmn,
                        ks > 0 ? 1u : acc_on);
    };
    auto issue_dq = [&]() {                                           // reduction over the 128 keys
#pragma unroll
        for (int ks = 0; ks < kTile / 16; ++ks)
            tc_mma_bf16(tm_dq, umma_desc_advance(m_dst, ks * 2048), umma_desc_advance(m_k, ks * 2048), idesc_mnmn, ks > 0);
        tc_commit(bar_g);
    };

    // minus the lse of query `qrow` in the log2 domain (fetched by the threads of half 0; -inf switches a missing query off)
    auto load_lse = [&](int b, int h, int qrow) -> float {
        if (half != 0) return 0.f;
        return qrow < n_sel ? P.lse[(static_cast<size_t>(b) * P.H + h) * P.N + qrow] * -1.4426950408889634f : -INFINITY;
    };
    // this thread's 32 head dimensions (64 bytes) of forward-output row `qrow`, zeros when there is no such row
    auto load_o = [&](int b, int h, int qrow, uint4* dst) {
        const bool have = qrow < n_sel && half * 32 < P.D;
        const uint4* src = reinterpret_cast<const uint4*>(P.o + ((static_cast<size_t>(b) * P.N + (have ? qrow : 0)) * P.H + h) * P.D + (have ? half * 32 : 0));
#pragma unroll
        for (int x = 0; x < 4; ++x) dst[x] = have ? __ldg(src + x) : make_uint4(0u, 0u, 0u, 0u);
    };
    // precomputed Delta of query `qrow` (fetched by the threads of half 1)
    auto load_delta = [&](int b, int h, int qrow) -> float {
        if (half != 1 || !use_delta) return 0.f;
        return qrow < n_sel ? P.delta[(static_cast<size_t>(b) * P.H + h) * P.Ncap + qrow] : 0.f;
    };
    auto dot8 = [](uint4 a, uint4 g) -> float {
        const float2 a0 = unpack2(a.x), a1 = unpack2(a.y), a2 = unpack2(a.z), a3 = unpack2(a.w);
        const float2 g0 = unpack2(g.x), g1 = unpack2(g.y), g2 = unpack2(g.z), g3 = unpack2(g.w);
        return a0.x * g0.x + a0.y * g0.y + a1.x * g1.x + a1.y * g1.y + a2.x * g2.x + a2.y * g2.y + a3.x * g3.x + a3.y * g3.y;
    };

    if (warp >= kBwdWorkers / 32) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kBwdIssuerRegs));
        // The third warpgroup.  Its first thread queues the products as their operands become ready: the workers announce P^T
        // and dS^T on bar_p / bar_ds; the tensor core runs dV and the next S^T while they compute dS^T, and dQ, dK and the next
        // dP^T while they compute the next P^T.  All four warps (one per quarter of the tensor-memory lanes) then take dQ of the
        // tile out of tensor memory into the fp32 shared-memory tile, which one bulk reduction adds to the accumulator.
        const bool issuer = tid == kBwdWorkers;
        const int qrow_l = tid - kBwdWorkers;           // query row this thread drains
        const int z_rounds = zero_warp ? zero_row_rounds(P) : 0;
        const int tiles_cta = (n_items > static_cast<int>(blockIdx.x) ? (n_items - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0) * n_t_max;
        const int z_slice = tiles_cta > 0 ? (z_rounds + tiles_cta - 1) / tiles_cta : z_rounds;      // rounds ahead of every query tile
        int z_round = 0;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const int jt = item % n_t_max;
            const int h = (item / n_t_max) % P.H;
            const int b = item / (n_t_max * P.H);
            const int kept = P.S > 1 ? P.n_sel[b] : kept_shared;
            const int n_q = (kept + kTile - 1) / kTile;
            if (jt >= n_q) continue;
            const bool single_tile = n_q == 1;
            if (issuer) {
                const uint32_t st0 = q_count % kQStages;
                ok &= mbar_wait(bar_kv, n_done & 1);
                ok &= mbar_wait(bar_qdo + st0, (q_count / kQStages) & 1);
                tc_fence_after();
                issue_st(st0);
                issue_dpt(st0);
            }
            for (int i = 0; i < n_q; ++i) {
                const uint32_t qc = q_count + i, st = qc % kQStages, st1 = (qc + 1) % kQStages, ph = qc & 1;
                for (int zs = 0; zs < z_slice && z_round < z_rounds; ++zs, ++z_round) zero_rows_round(P, z_round);
                if (issuer) {
                    ok &= mbar_wait(bar_p, ph);
                    tc_fence_after();
                    issue_dv(st, i > 0);
                    if (i + 1 < n_q) {                   // S^T of the next query tile queues up behind dV
                        ok &= mbar_wait(bar_qdo + st1, ((qc + 1) / kQStages) & 1);
                        tc_fence_after();
                        issue_st(st1);
                    }
                    ok &= mbar_wait(bar_ds, ph);
                    tc_fence_after();
                    issue_dq();
                    issue_dk(st, i > 0);
                    if (i + 1 < n_q) issue_dpt(st1);     // Q, dO of the next tile arrived before its S^T was issued
                    else tc_commit(bar_acc);
                }
                __syncwarp();                            // the issuer's warp waits for it here instead of polling beside it
                if (!single_tile) {                      // (a single key tile: the workers write dQ with dV and dK at the end)
                    ok &= mbar_wait(bar_g, ph);
                    tc_fence_after();
                    if (issuer) bulk_wait_group_read0(); // the previous reduction has read the shared-memory tile
                    group3_sync();
                    float dqv[32];
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {     // rows past n_sel are exact zeros (their probabilities are zero)
                        tmem_ld32(tm_dq + lane_sel + hf * 32, dqv);
                        tmem_ld_wait();
                        unsigned char* rowp = sDQ + hf * kTileBytes + qrow_l * kRowBytes;
#pragma unroll
                        for (int x = 0; x < 8; ++x)
                            *reinterpret_cast<float4*>(rowp + ((x ^ (qrow_l & 7)) << 4)) = make_float4(dqv[4 * x], dqv[4 * x + 1], dqv[4 * x + 2], dqv[4 * x + 3]);
                    }
                    fence_proxy_async_smem();
                    tc_fence_before();
                    ok = group3_sync_and(ok);            // dQ is out of tensor memory: the next one may be issued
                    if (issuer) {                        // one bulk reduce-add per half: dq_acc[b, 128 i .., h, 32 half ..] += tile
                        tma_reduce_add_4d(&map_acc, sDQ, 0, h, i * kTile, b);
                        tma_reduce_add_4d(&map_acc, sDQ + kTileBytes, 32, h, i * kTile, b);
                        bulk_commit_group();
                    }
                    if (!ok) break;
                }
            }
            ok = group3_sync_and(ok);                    // the warpgroup leaves together if a wait gave up
            if (!ok) break;
            if (P.convert_here && !single_tile) {        // tell the workers whether this was the last key tile of its (instance, head)
                if (issuer) {
                    int* flag = reinterpret_cast<int*>(smem_dyn + 104);
                    bulk_wait_group0();                  // this item's reductions have landed
                    __threadfence();
                    *flag = atomicAdd(P.tile_done + b * P.H + h, 1) == n_q - 1;
                    mbar_arrive(bar_conv);
                }
            }
            q_count += n_q;
            ++n_done;
        }
        for (; z_round < z_rounds; ++z_round) zero_rows_round(P, z_round);    // what is left of the zero rows
        if (tid == kBwdWorkers) bulk_wait_group0();      // the last dQ reductions have landed
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kBwdWorkerRegs));
    // Operand fetches of a work item: K, V and the first two query tiles' Q, dO, by warps 0 .. 3 side by side (each looks up its own
    // gather rows); a barrier phase cannot complete before the thread that announces its bytes has arrived, whichever comes
    // first.  `qc` is the number of query tiles this CTA has consumed before the item (its first ring stage).
    auto fetch_item = [&](int jt_, int h_, int b_, int kept_, uint32_t qc) {
        const int srow_ = P.S > 1 ? b_ : 0;
        TileSource src_ = P.src, src_do_ = P.src_do;
        if (src_.idx) src_.idx += static_cast<size_t>(srow_) * P.N;
        const int n_q_ = (kept_ + kTile - 1) / kTile;
        if (tid == 0) mbar_expect_tx(bar_kv, 2 * kTileBytes);
        if (warp == 0) load_tile(sK, &map_k, bar_kv, src_, jt_ * kTile, kept_, h_, b_, P.H);
        else if (warp == 1) load_tile(sV, &map_v, bar_kv, src_, jt_ * kTile, kept_, h_, b_, P.H);
        for (int i = 0; i < 2 && i < n_q_; ++i) {
            const uint32_t stage = (qc + i) % kQStages;
            if (warp == 2) {
                if ((tid & 31) == 0) mbar_expect_tx(bar_qdo + stage, 2 * kTileBytes);
                load_tile(sQ + stage * kTileBytes, &map_q, bar_qdo + stage, src_, i * kTile, kept_, h_, b_, P.H);
            } else if (warp == 3) {
                load_tile(sdO + stage * kTileBytes, &map_do, bar_qdo + stage, src_do_, i * kTile, kept_, h_, b_, P.H);
            }
        }
    };
    bool fetched = false;       // the operands of the item at hand were requested behind the products of the item before it
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const int jt = item % n_t_max;
        const int h = (item / n_t_max) % P.H;
        const int b = item / (n_t_max * P.H);
        const int srow = P.S > 1 ? b : 0;
        n_sel = P.S > 1 ? P.n_sel[srow] : kept_shared;
        const int n_q = (n_sel + kTile - 1) / kTile;               // query tiles = key tiles of this instance
        if (jt >= n_q) continue;
        const bool single_tile = n_q == 1;     // one key tile: dQ' needs no accumulation across CTAs
        use_delta = P.delta != nullptr && n_q > 1;                 // precomputed Delta exists only when there are several key tiles
        const int32_t* sel = P.sel_idx ? P.sel_idx + static_cast<size_t>(srow) * P.N : nullptr;
        TileSource src = P.src, src_do = P.src_do;
        if (src.idx) src.idx += static_cast<size_t>(srow) * P.N;
        // Query tile i of this item rides ring stage (q_count at item start + i) mod 3; the k-th use of a stage completes
        // phase k of its barrier.  Tiles are fetched two ahead of the one being processed.
        auto fetch_qdo = [&](int i, uint32_t stage) {    // warps 2 and 3 fetch Q and dO of query tile i; one thread announces the bytes
            if (warp == 2) {
                if ((tid & 31) == 0) mbar_expect_tx(bar_qdo + stage, 2 * kTileBytes);
                load_tile(sQ + stage * kTileBytes, &map_q, bar_qdo + stage, src, i * kTile, n_sel, h, b, P.H);
            } else if (warp == 3) {
                load_tile(sdO + stage * kTileBytes, &map_do, bar_qdo + stage, src_do, i * kTile, n_sel, h, b, P.H);
            }
        };
        // plain loads first (row statistics, forward output, the variate this thread's key row scatters to): they are in
        // flight while the tile fetches are issued
        const int key = jt * kTile + row;               // this thread's key row
        const bool key_valid = key < n_sel;
        const uint32_t st0 = q_count % kQStages;
        const float lse_first = load_lse(b, h, row);
        const float lse_second = n_q > 1 ? load_lse(b, h, kTile + row) : 0.f;
        uint4 o_cur[4], o_next[4];
        float dl_cur = load_delta(b, h, row), dl_next = 0.f;
        if (!use_delta) load_o(b, h, row, o_cur);
        const int n_out = key_valid ? (sel ? sel[key] : key) : 0;
        if (!fetched) fetch_item(jt, h, b, n_sel, q_count);      // (the CTA's first item: nothing came before it)
        fetched = false;
        if (half == 0) {
            s_stat[st0 * kTile + row] = lse_first;
            if (n_q > 1) s_stat[((st0 + 1) % kQStages) * kTile + row] = lse_second;
        }
        if (use_delta && half == 1) s_dpart[(q_count & 1) * kTile + row] = dl_cur;      // Delta of the first tile, in its parity's array
        worker_sync();                                   // row statistics of the first tiles visible

        // The query loop is a two-phase pipeline.  Phase A turns S^T into P^T while the tensor core still runs dK, dP^T of the
        // previous tile; once P^T is in shared memory dV and the next S^T are issued.  Phase B turns dP^T into dS^T while
        // those run; then dQ, dK and the next dP^T are issued.  dQ of a tile is drained one phase later, behind the next
        // tile's phase A, when it is surely complete.
        for (int i = 0; i < n_q; ++i, ++q_count) {
            const uint32_t st = q_count % kQStages, ph = q_count & 1;
            const uint32_t st2 = (q_count + 2) % kQStages;
            float lse_ahead = 0.f;
            if (i + 2 < n_q) lse_ahead = load_lse(b, h, (i + 2) * kTile + row);       // lands while this tile is processed
            if (i + 1 < n_q) {
                dl_next = load_delta(b, h, (i + 1) * kTile + row);
                if (!use_delta) load_o(b, h, (i + 1) * kTile + row, o_next);
            }
            if (!use_delta) {   // Delta of query `row`, this thread's 32 head dimensions: dO from the tile in shared memory, O from registers
                ok &= mbar_wait(bar_qdo + st, (q_count / kQStages) & 1);
                const unsigned char* do_row = sdO + st * kTileBytes + row * kRowBytes;
                float part = 0.f;
#pragma unroll
                for (int x = 0; x < 4; ++x)
                    part += dot8(o_cur[x], *reinterpret_cast<const uint4*>(do_row + (((half * 4 + x) ^ (row & 7)) << 4)));
                s_dpart[half * kTile + row] = part;
                worker_sync();                           // every partial sum is in place before phase B reads them
            }

            // ---- phase A: P^T of this thread's key row, its 64 queries (kept in registers for phase B) ----------
            ok &= mbar_wait(bar_s, ph);
            tc_fence_after();
            float pv[64];
            {   // 16 queries at a time; the next piece is read from tensor memory while the current one is processed
                const float* lse2 = s_stat + st * kTile + half * 64;
                const uint64_t scale2 = pair_of(P.scale_log2, P.scale_log2);
                float sv[2][16];
                tmem_ld16(tm_st + lane_sel + half * 64, sv[0]);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    tmem_ld_wait();
                    if (c < 3) tmem_ld16(tm_st + lane_sel + half * 64 + (c + 1) * 16, sv[(c + 1) & 1]);
#pragma unroll
                    for (int x = 0; x < 16; x += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(lse2 + c * 16 + x);       // minus lse
                        float e0, e1, e2, e3;
                        halves_of(fma_pair(pair_of(sv[c & 1][x + 0], sv[c & 1][x + 1]), scale2, pair_of(l4.x, l4.y)), e0, e1);
                        halves_of(fma_pair(pair_of(sv[c & 1][x + 2], sv[c & 1][x + 3]), scale2, pair_of(l4.z, l4.w)), e2, e3);
                        pv[c * 16 + x + 0] = key_valid ? fast_exp2(e0) : 0.f;    // rows past n_sel hold zero
                        pv[c * 16 + x + 1] = key_valid ? fast_exp2(e1) : 0.f;    // keys: they must not count
                        pv[c * 16 + x + 2] = key_valid ? fast_exp2(e2) : 0.f;
                        pv[c * 16 + x + 3] = key_valid ? fast_exp2(e3) : 0.f;
                    }
                    store_chunk16(sPt, row, half * 64 + c * 16, pv + c * 16);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar_p);                          // dV and the next S^T may go

            // ---- phase B: dS^T = P^T o (dP^T - Delta) ----------------------------------------------------------
            ok &= mbar_wait(bar_dp, ph);                 // dP^T done => every product of the previous tile is done: its ring stage is free
            tc_fence_after();
            if (i + 2 < n_q) fetch_qdo(i + 2, st2);
            {
                const float* dlt = s_dpart + (use_delta ? (q_count & 1) * kTile : 0) + half * 64;
                float dp[2][16];
                tmem_ld16(tm_dpt + lane_sel + half * 64, dp[0]);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    tmem_ld_wait();
                    if (c < 3) tmem_ld16(tm_dpt + lane_sel + half * 64 + (c + 1) * 16, dp[(c + 1) & 1]);
                    float* d = dp[c & 1];
                    if (use_delta) {                     // one array holds the complete Delta
#pragma unroll
                        for (int x = 0; x < 16; x += 4) {
                            const float4 da = *reinterpret_cast<const float4*>(dlt + c * 16 + x);
                            const uint64_t minus1 = pair_of(-1.f, -1.f);               // d - Delta as fma(Delta, -1, d): one rounding, as the subtraction
                            halves_of(mul_pair(pair_of(pv[c * 16 + x + 0], pv[c * 16 + x + 1]),
                                               fma_pair(pair_of(da.x, da.y), minus1, pair_of(d[x + 0], d[x + 1]))), d[x + 0], d[x + 1]);
                            halves_of(mul_pair(pair_of(pv[c * 16 + x + 2], pv[c * 16 + x + 3]),
                                               fma_pair(pair_of(da.z, da.w), minus1, pair_of(d[x + 2], d[x + 3]))), d[x + 2], d[x + 3]);
                        }
                    } else {                             // two partial sums, one per 32 head dimensions
#pragma unroll
                        for (int x = 0; x < 16; x += 4) {
                            const float4 da = *reinterpret_cast<const float4*>(dlt + c * 16 + x);
                            const float4 db = *reinterpret_cast<const float4*>(dlt + kTile + c * 16 + x);
                            d[x + 0] = pv[c * 16 + x + 0] * (d[x + 0] - (da.x + db.x));
                            d[x + 1] = pv[c * 16 + x + 1] * (d[x + 1] - (da.y + db.y));
                            d[x + 2] = pv[c * 16 + x + 2] * (d[x + 2] - (da.z + db.z));
                            d[x + 3] = pv[c * 16 + x + 3] * (d[x + 3] - (da.w + db.w));
                        }
                    }
                    store_chunk16(sdSt, row, half * 64 + c * 16, d);
                }
            }
            if (i + 2 < n_q && half == 0) s_stat[st2 * kTile + row] = lse_ahead;       // read two tiles from now, behind several barriers
            if (i + 1 < n_q) {
                // precomputed Delta of the next tile goes into the other parity's array now: the barrier at the end of this
                // iteration stands between this store and its readers, and that array's last readers are a barrier behind
                if (use_delta && half == 1) s_dpart[((q_count + 1) & 1) * kTile + row] = dl_next;
                dl_cur = dl_next;
                if (!use_delta) {
#pragma unroll
                    for (int x = 0; x < 4; ++x) o_cur[x] = o_next[x];
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar_ds);                         // dQ, dK and the next dP^T may go
            ok = worker_sync_and(ok);                    // a wait gave up somewhere among the workers: stop
            if (!ok) break;
        }
        if (!ok) break;

        ok &= mbar_wait(bar_acc, n_done & 1);
        tc_fence_after();
        // Every product of this item has completed: K, V and every Q / dO stage are free, and nothing below touches them.  The
        // operands of this CTA's next item are requested now, so that they travel while the gradients of this one are written;
        // the issuing thread then queues that item's first S^T and dP^T (tensor-memory columns the write-out does not read).
        if (ok) {
            for (int nx = item + gridDim.x; nx < n_items; nx += gridDim.x) {
                const int jt_n = nx % n_t_max, h_n = (nx / n_t_max) % P.H, b_n = nx / (n_t_max * P.H);
                const int kept_n = P.S > 1 ? P.n_sel[b_n] : kept_shared;
                if (jt_n >= (kept_n + kTile - 1) / kTile) continue;
                fetch_item(jt_n, h_n, b_n, kept_n, q_count);
                fetched = true;
                break;
            }
        }
        {   // dV, dK of this key tile (and dQ when this is the only key tile: key row = query row): every thread rounds its 32
            // columns to bf16 into a staging tile (the P^T / dS^T tiles are free now), then eight threads write each 128-byte
            // row of the full-layout gradients in one piece.
            unsigned char* stage_dv = sPt;
            unsigned char* stage_dk = sPt + kTileBytes;
            unsigned char* stage_dq = sdSt;
            int* s_nout = reinterpret_cast<int*>(sdSt + kTileBytes);           // variate of each key row, -1: no such row
            auto stage = [&](unsigned char* tile, uint32_t tm, float mul) {
                float acc[32];
                tmem_ld32(tm + lane_sel + half * 32, acc);
                tmem_ld_wait();
                unsigned char* rowp = tile + row * kRowBytes;
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4*>(rowp + (((half * 4 + q) ^ (row & 7)) << 4)) =
                        make_uint4(pack2(acc[8 * q + 0] * mul, acc[8 * q + 1] * mul), pack2(acc[8 * q + 2] * mul, acc[8 * q + 3] * mul),
                                   pack2(acc[8 * q + 4] * mul, acc[8 * q + 5] * mul), pack2(acc[8 * q + 6] * mul, acc[8 * q + 7] * mul));
            };
            stage(stage_dv, tm_dv, 1.f);
            stage(stage_dk, tm_dk, P.scale);
            if (single_tile) stage(stage_dq, tm_dq, P.scale);                   // complete: bar_acc covers every product of the item
            if (half == 0) s_nout[row] = key_valid ? n_out : -1;
            tc_fence_before();
            ok = worker_sync_and(ok);                    // the workers go on (or give up) together
            const int c = tid & 7;
            if (ok && c * 8 < P.D) {
                for (int r = tid >> 3; r < kTile; r += kBwdWorkers / 8) {
                    const int n = s_nout[r];
                    if (n < 0) continue;
                    const size_t out = ((static_cast<size_t>(b) * P.N + n) * P.H + h) * P.D + c * 8;
                    const int off = r * kRowBytes + ((c ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(P.dv + out) = *reinterpret_cast<const uint4*>(stage_dv + off);
                    *reinterpret_cast<uint4*>(P.dk + out) = *reinterpret_cast<const uint4*>(stage_dk + off);
                    if (single_tile) *reinterpret_cast<uint4*>(P.dq + out) = *reinterpret_cast<const uint4*>(stage_dq + off);
                }
            }
            worker_sync();          // staging tiles, statistics and accumulators are free for the next item
        }
        if (P.convert_here && !single_tile && ok) {   // dQ' of this (instance, head) is complete once all its key tiles are: the last one converts it
            int* flag = reinterpret_cast<int*>(smem_dyn + 104);
            ok &= mbar_wait(bar_conv, n_conv & 1);       // the third warpgroup has seen this item's reductions land and counted the tile
            ++n_conv;
            if (*flag) {
                __threadfence();
                const int chunks_head = P.D / 8;         // 16-byte output chunks per row
                for (int idx = tid; idx < n_sel * chunks_head; idx += kBwdWorkers) {
                    const int j = idx / chunks_head, dc = idx - j * chunks_head;
                    const float4* acc = reinterpret_cast<const float4*>(P.dq_acc + ((static_cast<size_t>(b) * P.Ncap + j) * P.H + h) * kDP) + dc * 2;
                    const float4 a0 = __ldcg(acc), a1 = __ldcg(acc + 1);
                    const int n = sel ? sel[j] : j;
                    *reinterpret_cast<uint4*>(P.dq + ((static_cast<size_t>(b) * P.N + n) * P.H + h) * P.D + dc * 8) =
                        make_uint4(pack2(a0.x * P.scale, a0.y * P.scale), pack2(a0.z * P.scale, a0.w * P.scale),
                                   pack2(a1.x * P.scale, a1.y * P.scale), pack2(a1.z * P.scale, a1.w * P.scale));
                }
            }
            worker_sync();          // `flag` is free for the next item
        }
        ++n_done;
    }
    }   // workers
    if (!ok) set_status(P.status, VARDROP_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kBwdTmemCols);
}

// ---------------------------------------------------------------------------------------------------------
// main, many tiles: the two phases of a (key tile, query tile) pair on warpgroups of their own
// ---------------------------------------------------------------------------------------------------------
// In the kernel above the same 256 threads turn S^T into P^T and then dP^T into dS^T, and the tensor core waits for each.
// With many query tiles per key tile that serial worker time is the whole step, so this kernel gives each phase its own 256
// threads and lets phase A of query tile i + 1 run beside phase B of tile i:
//   warps 0-2    issue the products, each its own chain (all lanes run the issue code, an elected lane executes each product);
//                warp 3 completes the register-donor warpgroup
//   warps 4-11   phase A: P^T = exp2(S^T scale - lse), written to tensor memory as bf16 (the A operand of dV += P^T dO); they
//                also take dQ of the previous tile out of tensor memory for the bulk reduce-add
//   warps 12-19  phase B: dS^T = P^T o (dP^T - Delta) with P^T read back from tensor memory, written to tensor memory
//                over the consumed columns of dP^T (the A operand of dK += dS^T Q) and to shared memory (dQ = dS K
//                reads it transposed)
// P^T and dS^T never pass through shared memory on their way to dV and dK, which takes 128 KB of shared-memory traffic
// off every tile pair (shared-memory bandwidth, not the tensor pipe, bounds these products at a head dimension of 64).
// Tensor memory: S^T [0,128) dP^T / dS^T [128,256) dV [256,320) dK [320,384) dQ [384,448) P^T [448,512).
// Delta is always precomputed here (the host takes this kernel only where the prep kernel runs) and tiles arrive as
// boxes (direct or staged).
constexpr int kPipeThreads = 640;
constexpr int kPipeGroup = 256;
constexpr int kPipeSmallRegs = 64;     // launched with 640 x 96 = 61440 registers: 128 x 64 + 512 x 104
constexpr int kPipeBigRegs = 104;
constexpr int kPipeHeader = 4096;      // barriers, row statistics, scatter indices
constexpr int kPipeSmemBytes = kPipeHeader + 2 * kTileBytes /*K, V*/ + 2 * kQStages * kTileBytes /*Q, dO ring*/ + 2 * kTileBytes /*dS^T*/ +
                               2 * kTileBytes /*dQ tile, fp32, two 32-column halves*/;

template <int kId>
__device__ __forceinline__ bool group_sync_and(bool ok) {      // named barrier kId among 256 threads, and-reduction of ok
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\n"
        "setp.ne.b32 q, %1, 0;\n"
        "bar.red.and.pred p, %2, 256, q;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(ok)), "n"(kId)
        : "memory");
    return r != 0;
}

__global__ void __launch_bounds__(kPipeThreads, 1) attn_bwd_pipe_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                         const __grid_constant__ CUtensorMap map_k,
                                                                         const __grid_constant__ CUtensorMap map_v,
                                                                         const __grid_constant__ CUtensorMap map_do,
                                                                         const __grid_constant__ CUtensorMap map_acc, const BwdParams P) {
    extern __shared__ unsigned char smem_dyn[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_dyn);
    uint64_t* bar_kv = bars + 0;
    uint64_t* bar_qdo = bars + 1;                   // [3]
    uint64_t* bar_s = bars + 4;                     // S^T of a query tile complete
    uint64_t* bar_sfree = bars + 5;                 // phase A holds S^T in registers (256 arrivals): the next S^T may be produced
    uint64_t* bar_p = bars + 6;                     // P^T in tensor memory (256 arrivals)
    uint64_t* bar_pfree = bars + 7;                 // phase B holds P^T in registers (256 arrivals) and dV has read it (1 commit)
    uint64_t* bar_dp = bars + 8;                    // dP^T of a query tile complete (and every product issued before it)
    uint64_t* bar_ds = bars + 9;                    // dS^T in tensor and shared memory (256 arrivals)
    uint64_t* bar_g = bars + 10;                    // dQ of a query tile complete
    uint64_t* bar_acc = bars + 11;                  // every product of the item complete: dV, dK final, operands free
    uint64_t* bar_dqfree = bars + 12;               // dQ of a query tile has left tensor memory (256 arrivals): the next one may be produced
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_dyn + 128);
    int* s_scratch = reinterpret_cast<int*>(smem_dyn + 132);
    float* s_stat = reinterpret_cast<float*>(smem_dyn + 256);     // [3 stages][128] minus the lse of the query tile, log2 domain
    float* s_delta = s_stat + kQStages * kTile;                   // [2][128] Delta of the query tile, one array per tile parity
    int* s_nout = reinterpret_cast<int*>(s_delta + 2 * kTile);    // [2][128] variate of each key row (-1: no such row), one array per item parity
    unsigned char* sK = align_tiles(smem_dyn + 256 + (kQStages + 4) * kTile * sizeof(float));
    unsigned char* sV = sK + kTileBytes;
    unsigned char* sQ = sV + kTileBytes;               // 3 stages
    unsigned char* sdO = sQ + kQStages * kTileBytes;   // 3 stages
    unsigned char* sdSt = sdO + kQStages * kTileBytes; // dS^T : rows = keys, columns = queries (two 64-query panels); dV / dK staging at the end of an item
    unsigned char* sDQ = sdSt + 2 * kTileBytes;        // dQ_i as fp32: panel `half` = head dimensions 32 half .. 32 half + 31, 128-byte swizzled rows
    const int tid = threadIdx.x, warp = tid >> 5;
    if (sDQ + 2 * kTileBytes > smem_dyn + kPipeSmemBytes) {
        chain_wait();
        if (tid == 0) set_status(P.status, VARDROP_ERR_CUDA);
        return;
    }
    if (warp == 0) {
        tmem_alloc(tmem_slot, kBwdTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_kv, 1);
        for (int st = 0; st < kQStages; ++st) mbar_init(bar_qdo + st, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_sfree, kPipeGroup);
        mbar_init(bar_p, kPipeGroup);
        mbar_init(bar_pfree, kPipeGroup + 1);
        mbar_init(bar_dp, 1);
        mbar_init(bar_ds, kPipeGroup);
        mbar_init(bar_g, 1);
        mbar_init(bar_acc, 3);
        mbar_init(bar_dqfree, kPipeGroup);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
        tma_prefetch_desc(&map_do);
        tma_prefetch_desc(&map_acc);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    chain_wait();
    chain_release();
    // One backward pass per forward pass: the forward kernel cleared this workspace's dQ' accumulator and tile counters and left a
    // mark; a backward pass that does not find the mark (a second backward for the same forward, or two forwards sharing the
    // workspace before their backwards) would add into stale state, so it reports the call instead of returning wrong gradients.
    if (blockIdx.x == 0 && threadIdx.x == 0 && atomicExch(P.status + kWsPairingWord, 0) != 1) set_status(P.status, VARDROP_ERR_INVALID_ARG);
    const int kept_shared = P.n_sel ? (P.S > 1 ? -1 : __ldg(P.n_sel)) : P.N;
    const int n_t_max = ((P.S > 1 ? max_kept(P.n_sel, P.S, P.N, s_scratch) : kept_shared) + kTile - 1) / kTile;
    const int n_items = n_t_max * P.H * P.B;                   // work items: (key tile, head, instance); short instances skip tiles

    const uint32_t tm_st = tmem;            // [0,128)   S^T
    const uint32_t tm_dpt = tmem + 128;     // [128,256) dP^T; dS^T (bf16) over its consumed columns: queries 64 half .. at column 64 half
    const uint32_t tm_dv = tmem + 256;      // [256,320) dV
    const uint32_t tm_dk = tmem + 320;      // [320,384) dK
    const uint32_t tm_dq = tmem + 384;      // [384,448) dQ of the current query tile
    const uint32_t tm_pt = tmem + 448;      // [448,512) P^T (bf16): queries 2 c, 2 c + 1 in column c
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    bool ok = true;
    uint32_t q_count = 0;       // query tiles consumed so far by this CTA: ring stage = q_count mod 3
    uint32_t n_done = 0;        // work items finished by this CTA

    struct Item { int jt, h, b, n_sel, n_q; };
    auto decode = [&](int item) {
        Item it;
        it.jt = item % n_t_max;
        it.h = (item / n_t_max) % P.H;
        it.b = item / (n_t_max * P.H);
        it.n_sel = P.S > 1 ? P.n_sel[it.b] : kept_shared;
        it.n_q = (it.n_sel + kTile - 1) / kTile;               // query tiles = key tiles of this instance
        return it;
    };
    // bf16 staging of a 64-column accumulator (this thread's 32 columns of its key row), then whole 128-byte rows to the
    // full-layout gradient: used by phase A for dV and by phase B for dK (and dQ of a single-tile instance)
    auto stage_acc = [&](unsigned char* tile, uint32_t tm, float mul, int row, int half) {
        float acc[32];
        tmem_ld32(tm + lane_sel + half * 32, acc);
        tmem_ld_wait();
        unsigned char* rowp = tile + row * kRowBytes;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4*>(rowp + (((half * 4 + q) ^ (row & 7)) << 4)) =
                make_uint4(pack2(acc[8 * q + 0] * mul, acc[8 * q + 1] * mul), pack2(acc[8 * q + 2] * mul, acc[8 * q + 3] * mul),
                           pack2(acc[8 * q + 4] * mul, acc[8 * q + 5] * mul), pack2(acc[8 * q + 6] * mul, acc[8 * q + 7] * mul));
    };
    auto store_rows = [&](const unsigned char* tile, __nv_bfloat16* dst, const int* nout, int gt, int b, int h) {     // gt: thread index in its group
        const int c = gt & 7;
        if (c * 8 >= P.D) return;
        for (int r = gt >> 3; r < kTile; r += kPipeGroup / 8) {
            const int n = nout[r];
            if (n < 0) continue;
            *reinterpret_cast<uint4*>(dst + ((static_cast<size_t>(b) * P.N + n) * P.H + h) * P.D + c * 8) =
                *reinterpret_cast<const uint4*>(tile + r * kRowBytes + ((c ^ (r & 7)) << 4));
        }
    };

    if (warp < 4) {
        // ------------------------------------------------------------ issue and dQ drain --------------------------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPipeSmallRegs));
        constexpr uint32_t idesc_kk = umma_idesc_bf16(128, 128, 0, 0);     // K-major x K-major, N = 128
        constexpr uint32_t idesc_kmn = umma_idesc_bf16(128, kDP, 0, 1);    // A K-major (tensor memory), B MN-major, N = 64
        constexpr uint32_t idesc_mnmn = umma_idesc_bf16(128, kDP, 1, 1);   // A MN-major, B MN-major, N = 64
        const uint64_t d_k = umma_desc_sw128(smem_u32(sK), 16, 1024), m_k = umma_desc_sw128(smem_u32(sK), kTileBytes, 1024);
        const uint64_t d_v = umma_desc_advance(d_k, kTileBytes);
        const uint64_t d_q0 = umma_desc_advance(d_k, 2 * kTileBytes), d_do0 = umma_desc_advance(d_k, (2 + kQStages) * kTileBytes);
        const uint64_t m_q0 = umma_desc_advance(m_k, 2 * kTileBytes), m_do0 = umma_desc_advance(m_k, (2 + kQStages) * kTileBytes);
        const uint64_t m_dst = umma_desc_advance(m_k, (2 + 2 * kQStages) * kTileBytes);
        auto issue_st = [&](uint32_t stage) {
            const uint64_t dq_ = umma_desc_advance(d_q0, stage * kTileBytes);
#pragma unroll
            for (int ks = 0; ks < kDP / 16; ++ks)
                tc_mma_bf16_w(tm_st, umma_desc_advance(d_k, ks * 32), umma_desc_advance(dq_, ks * 32), idesc_kk, ks > 0);
            tc_commit_w(bar_s);
        };
        auto issue_dpt = [&](uint32_t stage) {
            const uint64_t dd_ = umma_desc_advance(d_do0, stage * kTileBytes);
#pragma unroll
            for (int ks = 0; ks < kDP / 16; ++ks)
                tc_mma_bf16_w(tm_dpt, umma_desc_advance(d_v, ks * 32), umma_desc_advance(dd_, ks * 32), idesc_kk, ks > 0);
            tc_commit_w(bar_dp);
        };
        auto issue_dv = [&](uint32_t stage, uint32_t acc_on) {           // reduction over the 128 queries; P^T from tensor memory
            const uint64_t mdo = umma_desc_advance(m_do0, stage * kTileBytes);
#pragma unroll
            for (int ks = 0; ks < kTile / 16; ++ks)
                tc_mma_bf16_ta_w(tm_dv, tm_pt + ks * 8, umma_desc_advance(mdo, ks * 2048), idesc_kmn, ks > 0 ? 1u : acc_on);
            tc_commit_w(bar_pfree);
        };
        auto issue_dk = [&](uint32_t stage, uint32_t acc_on) {           // dS^T from tensor memory: queries 0..63 at column 0, 64..127 at column 64
            const uint64_t mq = umma_desc_advance(m_q0, stage * kTileBytes);
#pragma unroll
            for (int ks = 0; ks < kTile / 16; ++ks)
                tc_mma_bf16_ta_w(tm_dk, tm_dpt + (ks >> 2) * 64 + (ks & 3) * 8, umma_desc_advance(mq, ks * 2048), idesc_kmn, ks > 0 ? 1u : acc_on);
        };
        auto issue_dq = [&]() {                                           // reduction over the 128 keys; dS from shared memory, transposed view
#pragma unroll
            for (int ks = 0; ks < kTile / 16; ++ks)
                tc_mma_bf16_w(tm_dq, umma_desc_advance(m_dst, ks * 2048), umma_desc_advance(m_k, ks * 2048), idesc_mnmn, ks > 0);
            tc_commit_w(bar_g);
        };
        uint32_t n_drained = 0;                          // dQ tiles handed to phase A for draining so far
        // Three warps issue, each its own chain of products, so that no chain waits behind another's operands (every lane runs the
        // code, an elected lane executes each product; within a warp products complete in issue order):
        //   warp 0   S^T and dV: the chain through P^T          warp 1   dK and dP^T: the chain through dS^T in tensor memory
        //   warp 2   dQ: the chain through dS^T in shared memory and the drained dQ tile
        // bar_acc collects one commit from each at the end of an item.
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode(item);
            if (it.jt >= it.n_q) continue;
            const bool single_tile = it.n_q == 1;
            const uint32_t st0 = q_count % kQStages;
            if (warp < 3) {
                ok &= warp_wait(bar_kv, n_done & 1);
                if (warp < 2) ok &= warp_wait(bar_qdo + st0, (q_count / kQStages) & 1);
                tc_fence_after();
                if (warp == 0) issue_st(st0);
                else if (warp == 1) issue_dpt(st0);
            }
            for (int i = 0; i < it.n_q; ++i) {
                const uint32_t qc = q_count + i, st = qc % kQStages, st1 = (qc + 1) % kQStages, ph = qc & 1;
                if (warp == 0) {
                    ok &= warp_wait(bar_sfree, ph);      // phase A holds S^T of this tile: the next one may overwrite it
                    if (i + 1 < it.n_q) {
                        ok &= warp_wait(bar_qdo + st1, ((qc + 1) / kQStages) & 1);
                        tc_fence_after();
                        issue_st(st1);
                    }
                    ok &= warp_wait(bar_p, ph);
                    tc_fence_after();
                    issue_dv(st, i > 0);
                } else if (warp == 1) {
                    ok &= warp_wait(bar_ds, ph);
                    tc_fence_after();
                    issue_dk(st, i > 0);
                    if (i + 1 < it.n_q) {                // over dS^T in tensor memory, behind dK which reads it
                        ok &= warp_wait(bar_qdo + st1, ((qc + 1) / kQStages) & 1);
                        tc_fence_after();
                        issue_dpt(st1);
                    }
                } else if (warp == 2) {
                    ok &= warp_wait(bar_ds, ph);
                    if (n_drained > 0) ok &= warp_wait(bar_dqfree, (n_drained - 1) & 1);      // phase A has taken the previous dQ out of tensor memory
                    tc_fence_after();
                    issue_dq();
                    if (!single_tile) ++n_drained;
                }
            }
            if (warp < 3) tc_commit_w(bar_acc);          // this warp's products of the item
            if (!ok) break;
            q_count += it.n_q;
            ++n_done;
        }
        // The fourth warp of this group issues nothing and falls through the loop above at once: it writes the zero rows of the
        // dropped variates while the others work.  (Placed behind the loop, this code shares no live range with the issue code.)
        if (warp == 3) {
            const int z_rounds = zero_row_rounds(P);
            for (int z_round = 0; z_round < z_rounds; ++z_round) zero_rows_round(P, z_round);
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ phase A: P^T --------------------------------------
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPipeBigRegs));
        const int gt = tid - 128, row = gt & (kTile - 1), half = gt >> 7;
        const bool owner = gt == 0;                      // the one thread that owns the bulk reductions of dQ
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode(item);
            if (it.jt >= it.n_q) continue;
            const int n_sel = it.n_sel;
            const bool key_valid = it.jt * kTile + row < n_sel;
            const bool single_tile = it.n_q == 1;
            // dQ of query tile i out of tensor memory (this thread's 32 head dimensions of query row `row`) into the fp32 staging tile,
            // which one thread adds to the accumulator with two bulk reductions; called behind a group barrier that follows the
            // owner's wait for the previous reduction
            auto drain = [&](int i) {
                tc_fence_after();
                float dqv[32];
                tmem_ld32(tm_dq + lane_sel + half * 32, dqv);
                tmem_ld_wait();
                unsigned char* rowp = sDQ + half * kTileBytes + row * kRowBytes;
#pragma unroll
                for (int x = 0; x < 8; ++x)
                    *reinterpret_cast<float4*>(rowp + ((x ^ (row & 7)) << 4)) = make_float4(dqv[4 * x], dqv[4 * x + 1], dqv[4 * x + 2], dqv[4 * x + 3]);
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(bar_dqfree);                 // the next dQ may be produced
                ok = group_sync_and<1>(ok);              // the staging tile is complete
                if (owner) {
                    tma_reduce_add_4d(&map_acc, sDQ, 0, it.h, i * kTile, it.b);
                    tma_reduce_add_4d(&map_acc, sDQ + kTileBytes, 32, it.h, i * kTile, it.b);
                    bulk_commit_group();
                }
            };
            auto load_lse = [&](int qrow) -> float {     // minus the lse of query `qrow` in the log2 domain; -inf switches a missing query off
                return qrow < n_sel ? P.lse[(static_cast<size_t>(it.b) * P.H + it.h) * P.N + qrow] * -1.4426950408889634f : -INFINITY;
            };
            const uint32_t st0 = q_count % kQStages;
            if (half == 0) {
                s_stat[st0 * kTile + row] = load_lse(row);
                if (it.n_q > 1) s_stat[((st0 + 1) % kQStages) * kTile + row] = load_lse(kTile + row);
            }
            ok = group_sync_and<1>(ok);                  // row statistics of the first tiles visible
            for (int i = 0; i < it.n_q; ++i, ++q_count) {
                const uint32_t st = q_count % kQStages, ph = q_count & 1, st2 = (q_count + 2) % kQStages;
                float lse_ahead = 0.f;
                if (i + 2 < it.n_q && half == 0) lse_ahead = load_lse((i + 2) * kTile + row);       // lands while this tile is processed
                ok &= warp_wait_relaxed(bar_s, ph);
                tc_fence_after();
                float sv[64];
                tmem_ld32(tm_st + lane_sel + half * 64, sv);
                tmem_ld32(tm_st + lane_sel + half * 64 + 32, sv + 32);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(bar_sfree);                  // S^T is in registers
                uint32_t pw[32];
                {
                    const float* lse2 = s_stat + st * kTile + half * 64;
                    const uint64_t scale2 = pair_of(P.scale_log2, P.scale_log2);
#pragma unroll
                    for (int x = 0; x < 64; x += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(lse2 + x);       // minus lse
                        float e0, e1, e2, e3;
                        halves_of(fma_pair(pair_of(sv[x + 0], sv[x + 1]), scale2, pair_of(l4.x, l4.y)), e0, e1);
                        halves_of(fma_pair(pair_of(sv[x + 2], sv[x + 3]), scale2, pair_of(l4.z, l4.w)), e2, e3);
                        pw[(x >> 1) + 0] = pack2(fast_exp2(e0), fast_exp2(e1));
                        pw[(x >> 1) + 1] = pack2(fast_exp2(e2), fast_exp2(e3));
                    }
                    if (!key_valid) {                    // rows past n_sel hold zero keys: they must not count
#pragma unroll
                        for (int x = 0; x < 32; ++x) pw[x] = 0u;
                    }
                }
                if (q_count > 0) ok &= warp_wait_relaxed(bar_pfree, (q_count - 1) & 1);     // the previous P^T has been read by phase B and by dV
                tc_fence_after();
                tmem_st16(tm_pt + lane_sel + half * 32, pw);
                tmem_st16(tm_pt + lane_sel + half * 32 + 16, pw + 16);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_p);                      // dV may go, phase B may read P^T
                // dQ of the previous query tile: it was issued when phase B finished that tile
                if (!single_tile && i > 0) {
                    ok &= warp_wait_relaxed(bar_g, (q_count - 1) & 1);
                    if (owner) bulk_wait_group_read0();  // the previous reduction has read the shared-memory tile
                }
                ok = group_sync_and<1>(ok);              // everyone is done with this tile's statistics (and agrees on ok)
                if (!ok) break;
                if (i + 2 < it.n_q && half == 0) s_stat[st2 * kTile + row] = lse_ahead;       // read two tiles from now, behind this barrier's successor
                if (!single_tile && i > 0) drain(i - 1);
            }
            if (!ok) break;
            if (!single_tile) {                          // dQ of the last query tile
                ok &= warp_wait_relaxed(bar_g, (q_count - 1) & 1);
                if (owner) bulk_wait_group_read0();
                ok = group_sync_and<1>(ok);
                if (!ok) break;
                drain(it.n_q - 1);
            }
            // dV of this key tile
            ok &= warp_wait_relaxed(bar_acc, n_done & 1);
            tc_fence_after();
            stage_acc(sdSt, tm_dv, 1.f, row, half);
            if (owner) bulk_wait_group_read0();          // the fp32 staging tile is free (phase B may use it for a single-tile instance next)
            tc_fence_before();
            ok = group_sync_and<1>(ok);                  // the staging tile is complete
            if (!ok) break;
            // the scatter indices were written by phase B before its first arrival on bar_ds, which the products behind bar_acc waited for
            store_rows(sdSt, P.dv, s_nout + (n_done & 1) * kTile, gt, it.b, it.h);
            ++n_done;
        }
        if (owner) bulk_wait_group0();                   // the last dQ reductions have landed
    } else {
        // ------------------------------------------------------------ phase B: dS^T -------------------------------------
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPipeBigRegs));
        const int gt = tid - 384, row = gt & (kTile - 1), half = gt >> 7, gwarp = gt >> 5;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode(item);
            if (it.jt >= it.n_q) continue;
            const int n_sel = it.n_sel, srow = P.S > 1 ? it.b : 0;
            const bool single_tile = it.n_q == 1;
            const int32_t* sel = P.sel_idx ? P.sel_idx + static_cast<size_t>(srow) * P.N : nullptr;
            TileSource src = P.src, src_do = P.src_do;
            if (src.idx) src.idx += static_cast<size_t>(srow) * P.N;
            auto fetch_qdo = [&](int i, uint32_t stage) {    // warps 2 and 3 of the group fetch Q and dO of query tile i
                if (gwarp == 2) {
                    if ((tid & 31) == 0) mbar_expect_tx(bar_qdo + stage, 2 * kTileBytes);
                    load_tile(sQ + stage * kTileBytes, &map_q, bar_qdo + stage, src, i * kTile, n_sel, it.h, it.b, P.H);
                } else if (gwarp == 3) {
                    load_tile(sdO + stage * kTileBytes, &map_do, bar_qdo + stage, src_do, i * kTile, n_sel, it.h, it.b, P.H);
                }
            };
            auto load_delta = [&](int qrow) -> float {
                return qrow < n_sel ? P.delta[(static_cast<size_t>(it.b) * P.H + it.h) * P.Ncap + qrow] : 0.f;
            };
            const int key = it.jt * kTile + row;
            const bool key_valid = key < n_sel;
            const uint32_t st0 = q_count % kQStages;
            float dl_next = 0.f;
            const float dl_first = half == 1 ? load_delta(row) : 0.f;
            const int n_out = key_valid ? (sel ? sel[key] : key) : -1;
            {   // every MMA of the previous item has completed: K, V and every Q/dO stage are free
                if (gt == 0) mbar_expect_tx(bar_kv, 2 * kTileBytes);
                if (gwarp == 0) load_tile(sK, &map_k, bar_kv, src, it.jt * kTile, n_sel, it.h, it.b, P.H);
                else if (gwarp == 1) load_tile(sV, &map_v, bar_kv, src, it.jt * kTile, n_sel, it.h, it.b, P.H);
                fetch_qdo(0, st0);
                if (it.n_q > 1) fetch_qdo(1, (st0 + 1) % kQStages);
            }
            if (half == 1) s_delta[(q_count & 1) * kTile + row] = dl_first;
            else s_nout[(n_done & 1) * kTile + row] = n_out;     // phase A reads it at the end of the item; the array of two items ago is free
            ok = group_sync_and<3>(ok);
            for (int i = 0; i < it.n_q; ++i, ++q_count) {
                const uint32_t ph = q_count & 1, st2 = (q_count + 2) % kQStages;
                if (i + 1 < it.n_q && half == 1) dl_next = load_delta((i + 1) * kTile + row);
                ok &= warp_wait_relaxed(bar_p, ph);
                tc_fence_after();
                uint32_t pw[32];                         // this thread's 64 probabilities, bf16 pairs
                tmem_ld32(tm_pt + lane_sel + half * 32, reinterpret_cast<float*>(pw));
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(bar_pfree);
                ok &= warp_wait_relaxed(bar_dp, ph);             // dP^T done => dK, dP^T of the previous tile are done; its S^T, dV were done when
                                                         // P^T of this tile could be written: the ring stage of the previous tile is free
                if (q_count > 0) ok &= warp_wait_relaxed(bar_g, (q_count - 1) & 1);      // dQ of the previous tile has read the dS^T tile in shared memory
                tc_fence_after();
                if (i + 2 < it.n_q) fetch_qdo(i + 2, st2);
                {
                    const float* dlt = s_delta + (q_count & 1) * kTile + half * 64;
                    const uint64_t minus1 = pair_of(-1.f, -1.f);
                    float dp[2][16];
                    uint32_t dsw[16];
                    // destination of this thread's key row in the two 64-query panels of the dS^T tile (128-byte swizzled rows)
                    unsigned char* srow = sdSt + half * kTileBytes + row * kRowBytes;
                    const int sw = row & 7;
                    tmem_ld16(tm_dpt + lane_sel + half * 64, dp[0]);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        tmem_ld_wait();
                        if (c < 3) tmem_ld16(tm_dpt + lane_sel + half * 64 + (c + 1) * 16, dp[(c + 1) & 1]);
                        const float* d = dp[c & 1];
                        uint32_t* out = dsw + (c & 1) * 8;
#pragma unroll
                        for (int x = 0; x < 16; x += 4) {
                            const float4 da = *reinterpret_cast<const float4*>(dlt + c * 16 + x);
                            const uint32_t w0 = pw[c * 8 + (x >> 1)], w1 = pw[c * 8 + (x >> 1) + 1];
                            const uint64_t p01 = pair_of(__uint_as_float(w0 << 16), __uint_as_float(w0 & 0xFFFF0000u));
                            const uint64_t p23 = pair_of(__uint_as_float(w1 << 16), __uint_as_float(w1 & 0xFFFF0000u));
                            float r0, r1, r2, r3;
                            halves_of(mul_pair(p01, fma_pair(pair_of(da.x, da.y), minus1, pair_of(d[x + 0], d[x + 1]))), r0, r1);
                            halves_of(mul_pair(p23, fma_pair(pair_of(da.z, da.w), minus1, pair_of(d[x + 2], d[x + 3]))), r2, r3);
                            out[(x >> 1) + 0] = pack2(r0, r1);        // rounded once: the same words go to shared and to tensor memory
                            out[(x >> 1) + 1] = pack2(r2, r3);
                        }
                        *reinterpret_cast<uint4*>(srow + (((2 * c) ^ sw) << 4)) = make_uint4(out[0], out[1], out[2], out[3]);
                        *reinterpret_cast<uint4*>(srow + (((2 * c + 1) ^ sw) << 4)) = make_uint4(out[4], out[5], out[6], out[7]);
                        if (c & 1) tmem_st16(tm_dpt + lane_sel + half * 64 + (c >> 1) * 16, dsw);      // over columns this thread has consumed
                    }
                }
                if (i + 1 < it.n_q && half == 1) s_delta[((q_count + 1) & 1) * kTile + row] = dl_next;
                tmem_st_wait();
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(bar_ds);                     // dQ, dK and the next dP^T may go
                ok = group_sync_and<3>(ok);
                if (!ok) break;
            }
            if (!ok) break;
            ok &= warp_wait_relaxed(bar_acc, n_done & 1);
            tc_fence_after();
            stage_acc(sdSt + kTileBytes, tm_dk, P.scale, row, half);
            if (single_tile) stage_acc(sDQ, tm_dq, P.scale, row, half);         // complete: bar_acc covers every product of the item
            tc_fence_before();
            ok = group_sync_and<3>(ok);
            if (!ok) break;
            store_rows(sdSt + kTileBytes, P.dk, s_nout + (n_done & 1) * kTile, gt, it.b, it.h);
            if (single_tile) store_rows(sDQ, P.dq, s_nout + (n_done & 1) * kTile, gt, it.b, it.h);
            ++n_done;
        }
    }
    if (!ok) set_status(P.status, VARDROP_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kBwdTmemCols);
}

// ---------------------------------------------------------------------------------------------------------
// dq from the accumulator (paths with many key tiles)
// ---------------------------------------------------------------------------------------------------------
struct ConvertParams {
    const float4* dq_acc;    // [B, Ncap, H, 64] fp32
    uint4* dq;               // [B, N, H, D] bf16
    const int32_t* inv_idx;  // [S, N]; NULL: identity
    const int32_t* n_sel;    // [S]; NULL: N
    int N, Ncap, H, D, S;
    float scale;
};

__global__ void __launch_bounds__(256) bwd_convert_kernel(const ConvertParams P) {
    chain_wait();
    chain_release();
    const int b = blockIdx.y;
    const int srow = P.S > 1 ? b : 0;
    if ((P.n_sel ? P.n_sel[srow] : P.N) <= kTile) return;       // single key tile: the main kernel wrote the kept dq rows
    const int32_t* inv = P.inv_idx ? P.inv_idx + static_cast<size_t>(srow) * P.N : nullptr;
    const int chunks_head = P.D / 8;
    const int chunks_row = P.H * chunks_head;
    const int total = P.N * chunks_row;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int n = idx / chunks_row;
        const int c = idx - n * chunks_row;
        const int h = c / chunks_head, dc = c - h * chunks_head;
        const int j = inv ? inv[n] : n;
        if (j < 0) continue;                                     // dropped rows were zeroed by the main kernel
        const float4* src = P.dq_acc + ((static_cast<size_t>(b) * P.Ncap + j) * P.H + h) * (kDP / 4) + dc * 2;
        const float4 a = __ldcg(src), c2 = __ldcg(src + 1);
        P.dq[static_cast<size_t>(b) * total + idx] = make_uint4(pack2(a.x * P.scale, a.y * P.scale), pack2(a.z * P.scale, a.w * P.scale),
                                                                pack2(c2.x * P.scale, c2.y * P.scale), pack2(c2.z * P.scale, c2.w * P.scale));
    }
}

}  // namespace

int attn_bwd_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                    const int32_t* sel_idx, const int32_t* n_sel, const int32_t* inv_idx, const vardrop_attn_cfg& c, void* dq,
                    void* dk, void* dv, void* ws, cudaStream_t stream) {
    const AttnWs w = attn_layout(c);
    const QkvLayout L = qkv_layout(c);
    char* base = static_cast<char*>(ws);
    const bool staged = attn_uses_staging(c, sel_idx);
    const long long Hd = static_cast<long long>(c.H) * kDP, HD = static_cast<long long>(c.H) * c.D;
    const float scale = c.sm_scale > 0.f ? c.sm_scale : 1.f / sqrtf(static_cast<float>(c.D));

    const bool gathered = attn_uses_gather(c, sel_idx);
    // Delta is precomputed by a small kernel when there can be many key tiles (every key-tile CTA would otherwise
    // recompute it): without a selection, and on the staged path, where that kernel runs anyway to stage dO.  On the
    // gathered path (few tiles) the main kernel computes Delta itself.
    const bool pre_delta = sel_idx == nullptr ? c.N > kTile : staged;
    if (staged || pre_delta) {       // D = 32 also needs a zero-padded copy of dO next to the staged Q', K', V'
        PrepParams R{};
        R.o = static_cast<const uint4*>(o); R.d_o = static_cast<const uint4*>(d_o);
        R.dog = staged ? reinterpret_cast<uint4*>(base + w.dog) : nullptr;
        R.delta = pre_delta ? reinterpret_cast<float*>(base + w.delta) : nullptr;
        R.dq_acc = nullptr;
        R.n_sel = sel_idx ? n_sel : nullptr;
        R.N = c.N; R.Ncap = w.Ncap; R.H = c.H; R.D = c.D; R.S = attn_sel_rows(c);
        const long long work = static_cast<long long>(w.Ncap) * c.H * 8;
        int gx = static_cast<int>((work + 255) / 256);
        const int cap = max(1, 4 * sm_count() / c.B);              // about four CTAs per SM in total
        if (gx > cap) gx = cap;
        cudaError_t perr;
        { LaunchScope ls_(K_BWD_PREP, stream); perr = launch_chained(bwd_prep_kernel, dim3(gx, c.B), dim3(256), 0, stream, R); }
        if (int st = check_cuda(perr, "attention: backward prep launch")) return st;
    }

    CUtensorMap mq, mk, mv, mdo;
    if (staged) {
        if (int st = make_tile_map(&mq, base + w.qg, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
        if (int st = make_tile_map(&mk, base + w.kg, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
        if (int st = make_tile_map(&mv, base + w.vg, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
        if (int st = make_tile_map(&mdo, base + w.dog, c.B, w.Ncap, c.H, w.Ncap * Hd, Hd, kDP)) return st;
    } else if (gathered) {
        if (int st = make_row_map(&mq, q, L.rows_total, L.sH)) return st;
        if (int st = make_row_map(&mk, k, L.rows_total, L.sH)) return st;
        if (int st = make_row_map(&mv, v, L.rows_total, L.sH)) return st;
        if (int st = make_row_map(&mdo, d_o, static_cast<long long>(c.B) * c.N * c.H, kDP)) return st;      // d_o is contiguous
    } else {
        if (int st = make_tile_map(&mq, q, c.B, c.N, c.H, L.sB, L.sN, L.sH)) return st;
        if (int st = make_tile_map(&mk, k, c.B, c.N, c.H, L.sB, L.sN, L.sH)) return st;
        if (int st = make_tile_map(&mv, v, c.B, c.N, c.H, L.sB, L.sN, L.sH)) return st;
        if (int st = make_tile_map(&mdo, d_o, c.B, c.N, c.H, c.N * HD, HD, c.D)) return st;
    }
    CUtensorMap macc;
    if (int st = make_acc_map(&macc, base + w.dq_acc, c.B, w.Ncap, c.H)) return st;
    BwdParams P{};
    P.lse = lse; P.o = static_cast<const __nv_bfloat16*>(o); P.delta = pre_delta ? reinterpret_cast<const float*>(base + w.delta) : nullptr;
    P.dq_acc = reinterpret_cast<float*>(base + w.dq_acc);
    P.src.idx = sel_idx; P.src.gathered = gathered ? 1 : 0; P.src.tokens = c.N;
    P.src.rows_total = static_cast<int>(L.rows_total); P.src.row_b = static_cast<int>(L.row_b); P.src.row_n = static_cast<int>(L.row_n);
    P.src_do = P.src;
    P.src_do.idx = nullptr;         // dO rows are already compact: slot j is row j (and d_o is contiguous)
    P.src_do.rows_total = c.B * c.N * c.H; P.src_do.row_b = c.N * c.H; P.src_do.row_n = c.H;
    P.dq = static_cast<__nv_bfloat16*>(dq); P.dk = static_cast<__nv_bfloat16*>(dk); P.dv = static_cast<__nv_bfloat16*>(dv);
    P.sel_idx = sel_idx; P.n_sel = sel_idx ? n_sel : nullptr;
    P.inv_idx = sel_idx ? inv_idx : nullptr;
    P.tile_done = reinterpret_cast<int32_t*>(base + w.tile_done);
    P.convert_here = gathered ? 1 : 0;
    P.status = reinterpret_cast<int*>(base);
    P.B = c.B; P.N = c.N; P.Ncap = w.Ncap; P.H = c.H; P.D = c.D; P.S = attn_sel_rows(c);
    P.scale = scale; P.scale_log2 = scale * 1.4426950408889634f;
    static thread_local int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(attn_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemBytes), "attention: smem attribute")) return st;
        if (int st = check_cuda(cudaFuncSetAttribute(attn_bwd_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPipeSmemBytes), "attention: smem attribute")) return st;
        attr_dev = dev;
    }
    // Many query tiles per key tile: the kernel with one warpgroup pair per phase (it needs the precomputed Delta and boxed tiles,
    // which is what these shapes have).  The kept count is only known on the device, so the host goes by the largest it can be.
    const bool pipelined = !gathered && pre_delta && (sel_idx ? c.N > 2048 : c.N > 2 * kTile);
    {
        const long long worst = static_cast<long long>(w.Ncap / kTile) * c.H * c.B;
        const int grid = static_cast<int>(worst < sm_count() ? worst : sm_count());      // one CTA per SM (all of tensor memory)
        LaunchScope ls_(K_ATTN_BWD, stream);
        const cudaError_t err = pipelined
            ? launch_chained(attn_bwd_pipe_kernel, dim3(grid), dim3(kPipeThreads), kPipeSmemBytes, stream, mq, mk, mv, mdo, macc, P)
            : launch_chained(attn_bwd_kernel, dim3(grid), dim3(kBwdThreads), kBwdSmemBytes, stream, mq, mk, mv, mdo, macc, P);
        if (int st = check_cuda(err, "attention: backward launch")) return st;
    }
    if (!gathered && c.N > kTile) {         // several key tiles possible: dq comes from the accumulator in a pass of its own
        ConvertParams F{};
        F.dq_acc = reinterpret_cast<const float4*>(base + w.dq_acc);
        F.dq = static_cast<uint4*>(dq);
        F.inv_idx = sel_idx ? inv_idx : nullptr;
        F.n_sel = sel_idx ? n_sel : nullptr;
        F.N = c.N; F.Ncap = w.Ncap; F.H = c.H; F.D = c.D; F.S = attn_sel_rows(c); F.scale = scale;
        const long long work = static_cast<long long>(c.N) * c.H * (c.D / 8);
        int gx = static_cast<int>((work + 255) / 256);
        const int cap = max(1, 8 * sm_count() / c.B);
        if (gx > cap) gx = cap;
        cudaError_t cerr;
        { LaunchScope ls_(K_BWD_CONVERT, stream); cerr = launch_chained(bwd_convert_kernel, dim3(gx, c.B), dim3(256), 0, stream, F); }
        if (int st = check_cuda(cerr, "attention: backward convert launch")) return st;
    }
    return VARDROP_OK;

}

}  // namespace vardrop
