// Variate redundancy of a batch (Appendix A, Eq. 4): for every instance and variate, the largest Pearson correlation
// coefficient with any other variate of the same window, and how many variates exceed a threshold (Sec. 1 quotes the
// share above 0.9).  This is the O(N^2 T) similarity the paper argues against computing per batch; here it checks how
// redundant a workload is.
//
// pearson_normalize_kernel   one warp per (instance, variate): mean and centred norm in fp32, then the unit vector
//                            z = (x - mean) / |x - mean| is stored as two bf16 terms, z = hi + lo (16 mantissa bits),
//                            in [B, Npad, Lpad] arrays padded with zeros (Npad a multiple of 128, Lpad of 64).
// pearson_max_kernel         one CTA per (128-variate row tile, instance) walks over the column tiles: rho = z_v . z_w is a
//                            dense contraction, so it runs on the tcgen05 tensor cores (hi hi + hi lo + lo hi, fp32
//                            accumulator in tensor memory); one thread per row takes the maximum over the other variates.
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

constexpr int kPearsonThreads = 128;
constexpr int kPearsonSmemBytes = 1024 /*barrier, alignment*/ + 4 * kTileBytes /*row tile hi, lo; column tile hi, lo*/;
constexpr uint32_t kPearsonTmemCols = 128;

__global__ void __launch_bounds__(kPearsonThreads) pearson_max_kernel(const PearsonParams P) {
    extern __shared__ unsigned char smem_dyn[];
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_dyn);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_dyn + 8);
    unsigned char* sA_hi = align_tiles(smem_dyn + 16);
    unsigned char* sA_lo = sA_hi + kTileBytes;
    unsigned char* sB_hi = sA_lo + kTileBytes;
    unsigned char* sB_lo = sB_hi + kTileBytes;
    if (sB_lo + kTileBytes > smem_dyn + kPearsonSmemBytes) {     // dynamic shared memory base not 1024-byte aligned
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
    const int n_tiles = P.Npad / kTile, n_chunks = P.Lpad / 64;
    const int chunks_row = P.Lpad / 8;                           // 16-byte chunks per stored row
    const uint4* zh = reinterpret_cast<const uint4*>(P.z_hi) + static_cast<size_t>(b) * P.Npad * chunks_row;
    const uint4* zl = reinterpret_cast<const uint4*>(P.z_lo) + static_cast<size_t>(b) * P.Npad * chunks_row;
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128, 0, 0);
    const uint64_t d_ah = umma_desc_sw128(smem_u32(sA_hi), 16, 1024);
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
    const int v = ti * kTile + tid;                              // this thread's variate
    float best = -2.f;
    uint32_t phase = 0;
    bool ok = true;

    for (int tj = 0; tj < n_tiles && ok; ++tj) {
        for (int kc = 0; kc < n_chunks; ++kc) {
            // the four 128 x 64 tiles of this step, 16-byte chunks spread over the CTA, stored with the 128-byte swizzle
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint4 va[4], vb[4], vc[4], vd[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = tid + kPearsonThreads * (4 * half + u);
                    const int r = idx >> 3, ch = idx & 7;
                    const size_t oa = static_cast<size_t>(ti * kTile + r) * chunks_row + kc * 8 + ch;
                    const size_t ob = static_cast<size_t>(tj * kTile + r) * chunks_row + kc * 8 + ch;
                    va[u] = __ldg(zh + oa);
                    vb[u] = __ldg(zl + oa);
                    vc[u] = __ldg(zh + ob);
                    vd[u] = __ldg(zl + ob);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = tid + kPearsonThreads * (4 * half + u);
                    const int r = idx >> 3, ch = idx & 7;
                    const int off = r * kRowBytes + ((ch ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(sA_hi + off) = va[u];
                    *reinterpret_cast<uint4*>(sA_lo + off) = vb[u];
                    *reinterpret_cast<uint4*>(sB_hi + off) = vc[u];
                    *reinterpret_cast<uint4*>(sB_lo + off) = vd[u];
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {                                      // rho += hi hi + hi lo + lo hi over these 64 time steps
                tc_fence_after();
                const uint64_t d_al = umma_desc_advance(d_ah, kTileBytes), d_bh = umma_desc_advance(d_ah, 2 * kTileBytes);
                const uint64_t d_bl = umma_desc_advance(d_ah, 3 * kTileBytes);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    tc_mma_bf16(tmem, umma_desc_advance(d_ah, ks * 32), umma_desc_advance(d_bh, ks * 32), idesc, (kc > 0 || ks > 0) ? 1u : 0u);
                    tc_mma_bf16(tmem, umma_desc_advance(d_ah, ks * 32), umma_desc_advance(d_bl, ks * 32), idesc, 1u);
                    tc_mma_bf16(tmem, umma_desc_advance(d_al, ks * 32), umma_desc_advance(d_bh, ks * 32), idesc, 1u);
                }
                tc_commit(bar);
            }
            ok &= mbar_wait(bar, phase);                         // products done: the tiles may be overwritten
            phase ^= 1u;
            ok = __syncthreads_and(ok);
            if (!ok) break;
        }
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float r[32];
            tmem_ld32(tmem + lane_sel + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int w = tj * kTile + c * 32 + i;
                if (w < P.N && w != v) best = fmaxf(best, r[i]);
            }
        }
        tc_fence_before();
        __syncthreads();                                         // every row is read before the next column tile's products
    }

    if (ok && v < P.N) P.max_rho[static_cast<size_t>(b) * P.N + v] = best;
    const unsigned above = __ballot_sync(0xffffffffu, ok && v < P.N && best >= P.threshold);
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
    w.Npad = (c.N + kTile - 1) / kTile * kTile;
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
    { LaunchScope ls_(K_PEARSON_MAX, stream); err = launch_chained(pearson_max_kernel, dim3(w.Npad / kTile, c.B), dim3(kPearsonThreads), kPearsonSmemBytes, stream, P); }
    return check_cuda(err, "pearson: launch");
}

}  // namespace vardrop
