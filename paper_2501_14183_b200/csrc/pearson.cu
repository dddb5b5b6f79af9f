// Variate redundancy of a batch (Appendix A, Eq. 4): for every instance and variate, the largest Pearson correlation
// coefficient with any other variate of the same window, and how many variates exceed a threshold (Sec. 1 quotes the
// share above 0.9).  This is the O(N^2 T) similarity the paper argues against computing per batch; here it checks how
// redundant a workload is.
//
// pearson_normalize_kernel   one warp per (instance, variate): mean and centred norm in fp32, then the unit vector
//                            z = (x - mean) / |x - mean| is stored as two bf16 terms, z = hi + lo (16 mantissa bits),
//                            in [B, Npad, Lpad] arrays padded with zeros (Npad a multiple of 256, Lpad of 64).
// pearson_max_kernel         one CTA per (128-variate row tile, instance) walks over 256-variate column tiles: rho = z_v . z_w is
//                            a dense contraction, so it runs on the tcgen05 tensor cores (hi hi + hi lo + lo hi, fp32
//                            accumulator in tensor memory); operand chunks are fetched into registers one step ahead of
//                            the products; two threads per row take the maximum over the other variates.
#include "attn_common.cuh"

namespace vardrop {

namespace {

struct PearsonParams {
    const float* x;          // [B, N, L]
    __nv_bfloat16* z_hi;     // [B, Npad, Lpad]
    __nv_bfloat16* z_lo;
    float* max_rho;          // [B, N]
    int32_t* n_above;        // [B]
    int* status;
    int B, N, L, Npad, Lpad;
    float threshold;
};

__global__ void __launch_bounds__(256) pearson_normalize_kernel(const PearsonParams P) {
    chain_wait();
    chain_release();
    const int b = blockIdx.y, lane = threadIdx.x & 31;
    const int n = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (blockIdx.x == 0 && threadIdx.x == 0) P.n_above[b] = 0;
    if (n >= P.Npad) return;
    __nv_bfloat16* hi = P.z_hi + (static_cast<size_t>(b) * P.Npad + n) * P.Lpad;
    __nv_bfloat16* lo = P.z_lo + (static_cast<size_t>(b) * P.Npad + n) * P.Lpad;
    float mean = 0.f, inv = 0.f;
    const float* row = P.x + (static_cast<size_t>(b) * P.N + (n < P.N ? n : 0)) * P.L;
    if (n < P.N) {
        float s = 0.f;
        for (int t = lane; t < P.L; t += 32) s += row[t];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        mean = s / static_cast<float>(P.L);
        float ss = 0.f;
        for (int t = lane; t < P.L; t += 32) {
            const float d = row[t] - mean;
            ss = fmaf(d, d, ss);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if (!isfinite(ss) && lane == 0) set_status(P.status, VARDROP_ERR_NONFINITE);
        inv = ss > 0.f ? 1.f / sqrtf(ss) : 0.f;               // a constant variate correlates 0 with everything
    }
    for (int t = lane; t < P.Lpad; t += 32) {
        const float z = (n < P.N && t < P.L) ? (row[t] - mean) * inv : 0.f;
        const __nv_bfloat16 h = __float2bfloat16_rn(z);
        hi[t] = h;
        lo[t] = __float2bfloat16_rn(z - __bfloat162float(h));
    }
}

constexpr int kPearsonThreads = 256;                 // two threads per row: each takes 128 of the 256 columns of a step
constexpr int kColTile = 256;                        // column variates per step (one N = 256 product)
constexpr int kPearsonSmemBytes = 1024 /*barrier, row maxima, alignment*/ + 2 * kTileBytes /*row tile hi, lo*/ + 4 * kTileBytes /*column tile hi, lo*/;
constexpr uint32_t kPearsonTmemCols = 256;
constexpr int kPearsonChunks = (2 * 1024 + 2 * 2048) / kPearsonThreads;      // 16-byte chunks a thread moves per step (24)

__global__ void __launch_bounds__(kPearsonThreads, 2) pearson_max_kernel(const PearsonParams P) {
    extern __shared__ unsigned char smem_dyn[];
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_dyn);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_dyn + 8);
    float* s_best = reinterpret_cast<float*>(smem_dyn + 64);     // [128] maxima of the threads that take columns 128 .. 255
    unsigned char* sA = align_tiles(smem_dyn + 64 + kTile * sizeof(float));      // row tile: hi, then lo (16 KB each)
    unsigned char* sB = sA + 2 * kTileBytes;                                     // column tile: hi, then lo (32 KB each)
    if (sB + 4 * kTileBytes > smem_dyn + kPearsonSmemBytes) {    // dynamic shared memory base not 1024-byte aligned
        chain_wait();
        if (threadIdx.x == 0) set_status(P.status, VARDROP_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5;
    if (warp == 0) {
        tmem_alloc(tmem_slot, kPearsonTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar, 1);
        mbar_fence_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    chain_wait();
    chain_release();

    const int b = blockIdx.y, ti = blockIdx.x;
    const int n_col_tiles = P.Npad / kColTile, n_chunks = P.Lpad / 64, n_steps = n_col_tiles * n_chunks;
    const int chunks_row = P.Lpad / 8;                           // 16-byte chunks per stored row
    const uint4* zh = reinterpret_cast<const uint4*>(P.z_hi) + static_cast<size_t>(b) * P.Npad * chunks_row;
    const uint4* zl = reinterpret_cast<const uint4*>(P.z_lo) + static_cast<size_t>(b) * P.Npad * chunks_row;
    constexpr uint32_t idesc = umma_idesc_bf16(128, kColTile, 0, 0);
    const uint64_t d_ah = umma_desc_sw128(smem_u32(sA), 16, 1024);
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int row = tid & (kTile - 1), chalf = tid >> 7;         // tensor-memory lane and which 128 columns of it
    const int v = ti * kTile + row;                              // this thread's variate
    float best = -2.f;
    uint32_t phase = 0;
    bool ok = true, pending = false;

    // A step = 64 time steps of one column tile: the row tile's and the column tile's hi / lo chunks, 24 per thread.  They are
    // fetched into registers one step ahead, while the previous step's products run, and parked in shared memory (128-byte
    // swizzle) once those products are done.
    uint4 regs[kPearsonChunks];
    auto fetch = [&](int step) {
        const int tj = step / n_chunks, kc = step - tj * n_chunks;
#pragma unroll
        for (int u = 0; u < kPearsonChunks; ++u) {
            const int idx = tid + kPearsonThreads * u;           // 0 .. 6143: A hi, A lo (1024 each), B hi, B lo (2048 each)
            const bool is_a = idx < 2048;
            const int local = is_a ? (idx & 1023) : ((idx - 2048) & 2047);
            const bool lo_half = is_a ? idx >= 1024 : idx >= 4096;
            const int r = local >> 3, ch = local & 7;
            const size_t o = static_cast<size_t>((is_a ? ti * kTile : tj * kColTile) + r) * chunks_row + kc * 8 + ch;
            regs[u] = __ldg((lo_half ? zl : zh) + o);
        }
    };
    auto park = [&]() {
#pragma unroll
        for (int u = 0; u < kPearsonChunks; ++u) {
            const int idx = tid + kPearsonThreads * u;
            const bool is_a = idx < 2048;
            const int local = is_a ? (idx & 1023) : ((idx - 2048) & 2047);
            const bool lo_half = is_a ? idx >= 1024 : idx >= 4096;
            const int r = local >> 3, ch = local & 7;
            unsigned char* tile = is_a ? sA + (lo_half ? kTileBytes : 0) : sB + (lo_half ? 2 * kTileBytes : 0);
            *reinterpret_cast<uint4*>(tile + r * kRowBytes + ((ch ^ (r & 7)) << 4)) = regs[u];
        }
    };

    if (n_steps > 0) fetch(0);
    for (int step = 0; step < n_steps && ok; ++step) {
        const int tj = step / n_chunks, kc = step - tj * n_chunks;
        if (pending) {                                           // the previous step's products are done: its tiles may be overwritten
            ok &= mbar_wait(bar, phase);
            phase ^= 1u;
            pending = false;
        }
        park();
        fence_proxy_async_smem();
        tc_fence_before();
        ok = __syncthreads_and(ok);
        if (!ok) break;
        if (tid == 0) {                                          // rho += hi hi + hi lo + lo hi over these 64 time steps
            tc_fence_after();
            const uint64_t d_al = umma_desc_advance(d_ah, kTileBytes), d_bh = umma_desc_advance(d_ah, 2 * kTileBytes);
            const uint64_t d_bl = umma_desc_advance(d_ah, 4 * kTileBytes);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                tc_mma_bf16(tmem, umma_desc_advance(d_ah, ks * 32), umma_desc_advance(d_bh, ks * 32), idesc, (kc > 0 || ks > 0) ? 1u : 0u);
                tc_mma_bf16(tmem, umma_desc_advance(d_ah, ks * 32), umma_desc_advance(d_bl, ks * 32), idesc, 1u);
                tc_mma_bf16(tmem, umma_desc_advance(d_al, ks * 32), umma_desc_advance(d_bh, ks * 32), idesc, 1u);
            }
            tc_commit(bar);
        }
        pending = true;
        if (step + 1 < n_steps) fetch(step + 1);                 // in flight while the products run
        if (kc + 1 == n_chunks) {                                // the column tile is complete: this thread's row, its 128 columns
            ok &= mbar_wait(bar, phase);
            phase ^= 1u;
            pending = false;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float r[32];
                tmem_ld32(tmem + lane_sel + chalf * 128 + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int w = tj * kColTile + chalf * 128 + c * 32 + i;
                    if (w < P.N && w != v) best = fmaxf(best, r[i]);
                }
            }
            tc_fence_before();
            ok = __syncthreads_and(ok);                          // every row is read before the next column tile's products
        }
    }

    if (chalf == 1) s_best[row] = best;
    __syncthreads();
    if (chalf == 0) best = fmaxf(best, s_best[row]);
    const bool mine = chalf == 0 && ok && v < P.N;
    if (mine) P.max_rho[static_cast<size_t>(b) * P.N + v] = best;
    const unsigned above = __ballot_sync(0xffffffffu, mine && best >= P.threshold);
    if ((tid & 31) == 0 && above) atomicAdd(P.n_above + b, __popc(above));
    if (!ok) set_status(P.status, VARDROP_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kPearsonTmemCols);
}

struct PearsonWs {
    size_t z_hi, z_lo, total;
    int Npad, Lpad;
};
PearsonWs pearson_layout(const vardrop_pearson_cfg& c) {
    PearsonWs w;
    w.Npad = (c.N + kColTile - 1) / kColTile * kColTile;
    w.Lpad = (c.L + 63) / 64 * 64;
    const size_t bytes = align_up(static_cast<size_t>(c.B) * w.Npad * w.Lpad * sizeof(__nv_bfloat16), 1024);
    w.z_hi = kWsHeaderBytes;
    w.z_lo = w.z_hi + bytes;
    w.total = w.z_lo + bytes;
    return w;
}

}  // namespace

int pearson_validate(const vardrop_pearson_cfg& c) {
    if (c.B < 1 || c.N < 1 || c.L < 2) return fail(VARDROP_ERR_INVALID_ARG, "pearson: B, N >= 1 and L >= 2 required (B=%d N=%d L=%d)", c.B, c.N, c.L);
    if (c.B > 65535) return fail(VARDROP_ERR_UNSUPPORTED, "pearson: B=%d above 65535", c.B);
    if (c.L > 65536 || c.N > (1 << 22)) return fail(VARDROP_ERR_UNSUPPORTED, "pearson: L=%d or N=%d too large", c.L, c.N);
    if (!(c.threshold >= -1.f && c.threshold <= 1.f)) return fail(VARDROP_ERR_INVALID_ARG, "pearson: threshold must lie in [-1, 1]");
    return VARDROP_OK;
}

size_t pearson_workspace_bytes(const vardrop_pearson_cfg& c) { return pearson_layout(c).total; }

int pearson_launch(const float* x, const vardrop_pearson_cfg& c, float* max_rho, int32_t* n_above, void* ws, cudaStream_t stream) {
    const PearsonWs w = pearson_layout(c);
    char* base = static_cast<char*>(ws);
    PearsonParams P{};
    P.x = x; P.z_hi = reinterpret_cast<__nv_bfloat16*>(base + w.z_hi); P.z_lo = reinterpret_cast<__nv_bfloat16*>(base + w.z_lo);
    P.max_rho = max_rho; P.n_above = n_above; P.status = reinterpret_cast<int*>(base);
    P.B = c.B; P.N = c.N; P.L = c.L; P.Npad = w.Npad; P.Lpad = w.Lpad; P.threshold = c.threshold;
    cudaError_t err;
    { LaunchScope ls_(K_PEARSON_NORM, stream); err = launch_chained(pearson_normalize_kernel, dim3((w.Npad + 7) / 8, c.B), dim3(256), 0, stream, P); }
    if (int st = check_cuda(err, "pearson: normalize launch")) return st;
    static thread_local int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_dev != dev) {
        if (int st = check_cuda(cudaFuncSetAttribute(pearson_max_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPearsonSmemBytes), "pearson: smem attribute")) return st;
        attr_dev = dev;
    }
    { LaunchScope ls_(K_PEARSON_MAX, stream); err = launch_chained(pearson_max_kernel, dim3((c.N + kTile - 1) / kTile, c.B), dim3(kPearsonThreads), kPearsonSmemBytes, stream, P); }
    return check_cuda(err, "pearson: launch");
}

}  // namespace vardrop
