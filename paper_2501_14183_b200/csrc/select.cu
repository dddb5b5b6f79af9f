// Grouping by hash value and stratified sampling (Eq. 1, Eq. 2), without a spin-wait.
//
// Small problems (N <= 2048): one CTA per hash row does everything in shared memory (select_small_kernel).
// Larger ones take three launches:
//   select_count_kernel   every CTA compares a slice of variates against a slice of keys and adds, per variate n,
//                         lt[n] = #{m : key_m < key_n} and eq[n] = #{m < n : key_m = key_n} with integer atomics.  lt[n] is
//                         the start of n's group in (key, index) order and eq[n] is n's rank inside its group, so lt + eq
//                         is n's sorted position.
//   select_group_kernel   one CTA per hash row scatters the members, scans the group heads into dense group ids and
//                         offsets, and draws each member's Philox priority.
//   select_sample_kernel  every member counts the members of its own group with a smaller (priority, rank) pair; it is
//                         kept when that count is below the group's quota.  The CTA that finishes last for a hash row
//                         compacts the kept variates into sel_idx / inv_idx with one scan.
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace vardrop {

namespace {

constexpr int kSelThreads = 256;    // select_count_kernel
constexpr int kTailThreads = 1024;  // select_group_kernel, select_sample_kernel: one CTA walks a whole hash row, so the
                                    // round trips to memory are spread over as many threads as a CTA can have
constexpr int kTailChunks = 8;      // positions per thread in a batch of the ordered compaction (64 registers a thread)
constexpr int kKeyChunk = 128;      // keys compared per CTA by select_count_kernel
constexpr size_t kGroupMaxSmem = 216 * 1024;   // select_group_kernel keeps 12 bytes per variate in shared memory up to this

struct SelectParams {
    const uint64_t* keys;
    int32_t *group_id, *group_offsets, *members, *n_groups, *sel_idx, *n_sel, *inv_idx;
    // workspace
    int* status;
    unsigned int* done1;   // [S]
    unsigned int* done2;   // [S]
    int32_t* lt;           // [S, N]
    int32_t* eq;           // [S, N]
    uint32_t* prio;        // [S, N] priority by sorted position
    int32_t* keep;         // [S, N] by variate
    int S, N, gs;
    long long rate_ppm;
    uint32_t seed_lo, seed_hi, step;
};

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies, xors with the key, and a
// Weyl key schedule.  Returns word 0 of the output block.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

__device__ __forceinline__ int quota_of(int size, int gs, long long rate_ppm) {
    long long by_rate = (static_cast<long long>(size) * rate_ppm + 999999ll) / 1000000ll;
    if (by_rate < 1) by_rate = 1;
    long long q = size;
    if (gs > 0 && gs < q) q = gs;
    if (by_rate < q) q = by_rate;
    return static_cast<int>(q);
}

// Inclusive scan of one int per thread across the CTA (kThreads threads); returns this thread's inclusive value
// and the CTA total through `total`.
template <int kThreads>
__device__ __forceinline__ int block_scan_inclusive(int v, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += o;
    }
    __syncthreads();
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        const int s = warp_sums[w];
        if (w < warp) base += s;
        tot += s;
    }
    *total = tot;
    return v + base;
}

// True in every thread of exactly one CTA per hash row: the one whose arrival completes the count.
__device__ __forceinline__ bool last_cta_of_row(unsigned int* counter, unsigned int ctas_per_row, int* flag_smem) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int prev = atomicAdd(counter, 1u);
        *flag_smem = (prev + 1u == ctas_per_row);
    }
    __syncthreads();
    const bool last = *flag_smem != 0;
    if (last) __threadfence();
    return last;
}

// Ordered compaction by one CTA of kThreads threads: for every position p < N, in ascending order,
// `emit(p, set, before, payload)` is called with (set, payload) = flag(p) and before = number of set flags at positions
// below p; returns the number of set flags.  Positions are dealt to the threads round-robin (position = batch base +
// chunk * kThreads + thread) and a batch of kChunks chunks is handled with fully unrolled loops, so the (dependent) loads
// behind the flags of a thread are coalesced and all in flight at once instead of one memory round trip per position; a
// batch is ordered with warp ballots and one scan of the per-warp counts.
template <int kThreads, int kChunks, class FlagFn, class EmitFn>
__device__ __forceinline__ int ordered_compact(int N, FlagFn flag, EmitFn emit) {
    constexpr int kWarps = kThreads / 32;
    static_assert(kChunks <= 32 && kChunks * kWarps <= kThreads, "one ballot word per thread at most");
    __shared__ uint32_t s_mask[kChunks * kWarps];  // ballot of chunk k, warp w at [k * kWarps + w]: position order
    __shared__ int s_excl[kChunks * kWarps];       // set flags of the batch before that (chunk, warp)
    __shared__ int s_warp[kWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int done = 0;                                  // set flags of the batches before this one
    for (int base = 0; base < N; base += kChunks * kThreads) {
        uint32_t bits = 0;                         // bit k: flag of position base + k * kThreads + thread
        int payload[kChunks];
#pragma unroll
        for (int k = 0; k < kChunks; ++k) {
            const int p = base + k * kThreads + static_cast<int>(threadIdx.x);
            payload[k] = 0;
            if (p < N && flag(p, &payload[k])) bits |= 1u << k;
        }
        uint32_t mine = 0;
#pragma unroll
        for (int k = 0; k < kChunks; ++k) {
            const uint32_t m = __ballot_sync(0xffffffffu, (bits >> k) & 1u);
            if (lane == k) mine = m;
        }
        __syncthreads();                           // the tables of the previous batch are no longer read
        if (lane < kChunks) s_mask[lane * kWarps + warp] = mine;
        __syncthreads();
        int total = 0;
        const bool entry = static_cast<int>(threadIdx.x) < kChunks * kWarps;      // one (chunk, warp) ballot per thread
        const int cnt = entry ? __popc(s_mask[threadIdx.x]) : 0;
        const int incl = block_scan_inclusive<kThreads>(cnt, s_warp, &total);
        if (entry) s_excl[threadIdx.x] = incl - cnt;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kChunks; ++k) {
            const int p = base + k * kThreads + static_cast<int>(threadIdx.x);
            if (p < N) {
                const uint32_t m = s_mask[k * kWarps + warp];
                emit(p, ((bits >> k) & 1u) != 0, done + s_excl[k * kWarps + warp] + __popc(m & ((1u << lane) - 1u)), payload[k]);
            }
        }
        done += total;
    }
    return done;
}

__global__ void __launch_bounds__(kSelThreads) select_count_kernel(const SelectParams P) {
    __shared__ uint64_t skeys[kKeyChunk];
    chain_wait();
    chain_release();
    const int s = blockIdx.z, N = P.N;
    const uint64_t* keys = P.keys + static_cast<size_t>(s) * N;
    int32_t* lt = P.lt + static_cast<size_t>(s) * N;
    int32_t* eq = P.eq + static_cast<size_t>(s) * N;
    const int n = blockIdx.x * kSelThreads + threadIdx.x;
    const int m0 = blockIdx.y * kKeyChunk;
    const int mcount = min(kKeyChunk, N - m0);
    for (int i = threadIdx.x; i < mcount; i += blockDim.x) skeys[i] = keys[m0 + i];
    __syncthreads();
    if (n < N) {
        const uint64_t mine = keys[n];
        int c_lt = 0, c_eq = 0;
        const int n_first = blockIdx.x * kSelThreads;
        if (m0 >= n_first + kSelThreads) {                 // every key of the slice has a higher index than every variate here
            for (int i = 0; i < mcount; ++i) c_lt += skeys[i] < mine;
        } else if (m0 + mcount <= n_first) {               // every key of the slice has a lower index
            for (int i = 0; i < mcount; ++i) {
                const uint64_t other = skeys[i];
                c_lt += other < mine;
                c_eq += other == mine;
            }
        } else {
            for (int i = 0; i < mcount; ++i) {
                const uint64_t other = skeys[i];
                c_lt += other < mine;
                c_eq += (other == mine) & (m0 + i < n);
            }
        }
        if (c_lt) atomicAdd(lt + n, c_lt);
        if (c_eq) atomicAdd(eq + n, c_eq);
    }
}

// One CTA per hash row, after the counts are complete: members, group heads -> ids and offsets, priorities.
// The three passes reach members / eq / group ids through the sorted positions, i.e. in scattered order.  A single SM
// turns every scattered warp access to global memory into 32 separate requests, which is what this kernel's time used
// to be; with kShared the three arrays live in shared memory (12 bytes per variate) and global memory only sees
// coalesced reads and writes.  Rows too long for that work on the global arrays directly.
template <bool kShared>
__global__ void __launch_bounds__(kTailThreads) select_group_kernel(const SelectParams P) {
    extern __shared__ int32_t s_rows[];
    chain_wait();
    chain_release();
    const int s = blockIdx.x, N = P.N;
    const int32_t* lt = P.lt + static_cast<size_t>(s) * N;
    int32_t* eq = P.eq + static_cast<size_t>(s) * N;
    int32_t* members = P.members + static_cast<size_t>(s) * N;
    int32_t* gid = P.group_id + static_cast<size_t>(s) * N;
    int32_t* off = P.group_offsets + static_cast<size_t>(s) * (N + 1);
    uint32_t* prio = P.prio + static_cast<size_t>(s) * N;
    int32_t* gid_by_pos = P.lt + static_cast<size_t>(s) * N;       // lt is dead after the first pass: group id by position
    int32_t* w_eq = kShared ? s_rows : eq;                         // working copies, by variate / position / variate
    int32_t* w_members = kShared ? s_rows + N : members;
    int32_t* w_gid = kShared ? s_rows + 2 * N : gid;
    // every loop of this kernel takes several positions per thread at a time: the loads of a batch are issued together, so
    // a batch costs one or two memory round trips instead of one per position
    constexpr int U = 4;
    for (int base = 0; base < N; base += U * kTailThreads) {
        int dst[U], rank[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = base + u * kTailThreads + static_cast<int>(threadIdx.x);
            rank[u] = i < N ? __ldcg(eq + i) : 0;
            dst[u] = i < N ? __ldcg(lt + i) + rank[u] : -1;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = base + u * kTailThreads + static_cast<int>(threadIdx.x);
            if (dst[u] >= 0) {
                w_members[dst[u]] = i;
                if (kShared) w_eq[i] = rank[u];
            }
        }
    }
    __syncthreads();
    // group heads over the sorted positions: the first member of every group has no equal key before it
    const int total_groups = ordered_compact<kTailThreads, kTailChunks>(
        N, [&](int p, int* nn) { *nn = w_members[p]; return w_eq[*nn] == 0; },
        [&](int p, bool head, int before, int nn) {
            if (head) off[before] = p;
            const int g = before - (head ? 0 : 1);       // heads at or below p, minus one
            w_gid[nn] = g;
            gid_by_pos[p] = g;
            if (kShared) members[p] = nn;
        });
    for (int i = total_groups + threadIdx.x; i <= N; i += blockDim.x) off[i] = N;
    if (threadIdx.x == 0) P.n_groups[s] = total_groups;
    __syncthreads();
    for (int base = 0; base < N; base += U * kTailThreads) {
        int rank[U], g[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int p = base + u * kTailThreads + static_cast<int>(threadIdx.x);
            const int nn = p < N ? w_members[p] : 0;
            rank[u] = w_eq[nn];
            g[u] = w_gid[nn];
            if (kShared && p < N) gid[p] = w_gid[p];     // position p doubles as a variate index for the copy-out
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int p = base + u * kTailThreads + static_cast<int>(threadIdx.x);
            if (p < N)
                prio[p] = philox4x32_10_word0(static_cast<uint32_t>(rank[u]), static_cast<uint32_t>(g[u]), static_cast<uint32_t>(s), P.step,
                                              P.seed_lo, P.seed_hi);
        }
    }
}

__global__ void __launch_bounds__(kTailThreads) select_sample_kernel(const SelectParams P) {
    __shared__ int flag;
    chain_wait();
    chain_release();
    const int s = blockIdx.z, N = P.N;
    const int32_t* members = P.members + static_cast<size_t>(s) * N;
    const int32_t* gid_by_pos = P.lt + static_cast<size_t>(s) * N;      // written by select_group_kernel
    const int32_t* off = P.group_offsets + static_cast<size_t>(s) * (N + 1);
    const uint32_t* prio = P.prio + static_cast<size_t>(s) * N;
    int32_t* keep = P.keep + static_cast<size_t>(s) * N;
    const int p = blockIdx.x * kTailThreads + threadIdx.x;
    if (p < N) {
        const int nn = members[p];
        const int g = gid_by_pos[p];
        const int begin = off[g], end = off[g + 1];
        const uint32_t mine = prio[p];
        int smaller = 0;
        for (int o = begin; o < end; ++o) {
            const uint32_t other = __ldg(prio + o);
            smaller += (other < mine) | ((other == mine) & (o < p));
        }
        keep[nn] = smaller < quota_of(end - begin, P.gs, P.rate_ppm);
    }
    if (!last_cta_of_row(P.done2 + s, gridDim.x, &flag)) return;

    // ---- the last CTA of this hash row: compaction of the kept variates in ascending index order --------
    int32_t* sel = P.sel_idx + static_cast<size_t>(s) * N;
    int32_t* inv = P.inv_idx + static_cast<size_t>(s) * N;
    const int total = ordered_compact<kTailThreads, kTailChunks>(
        N, [&](int i, int*) { return __ldcg(keep + i) != 0; },
        [&](int i, bool kept, int before, int) {
            if (kept) sel[before] = i;
            inv[i] = kept ? before : -1;
        });
    for (int i = total + threadIdx.x; i < N; i += blockDim.x) sel[i] = -1;
    if (threadIdx.x == 0) P.n_sel[s] = total;
}

// ---------------------------------------------------------------------------------------------------------
// Small problems (N <= 2048): one CTA per hash row does everything in shared memory with two bitonic sorts.
//   sort 1: (key, variate)                      -> members, group heads -> ids, offsets
//   sort 2: (group id, Philox priority, rank j) -> position inside the group = sampling rank
// then the kept flags are compacted with one scan.  No scratch in global memory, no atomics.
// ---------------------------------------------------------------------------------------------------------
constexpr int kSmallMaxN = 2048;

// Bitonic sort of M (a power of two >= 64) items by M / 2 threads.  Thread t keeps items 2t and 2t + 1 in registers.
// Compare-exchange distance j = 1 stays inside the thread, j = 2 .. 32 goes through warp shuffles (the partner of item
// i is item i ^ j = slot (i & 1) of lane t ^ (j / 2)), and only j >= 64 passes through shared memory.
// Items are (key, payload) pairs ordered by key, then payload; kPayload = false sorts bare keys.
template <bool kPayload>
__device__ __forceinline__ void bitonic_sort_regs(uint64_t& k0, uint32_t& p0, uint64_t& k1, uint32_t& p1, uint64_t* sk, uint32_t* sp, int M) {
    const int t = threadIdx.x;
    auto greater = [](uint64_t ka, uint32_t pa, uint64_t kb, uint32_t pb) { return ka > kb || (kPayload && ka == kb && pa > pb); };
    // keep the smaller of (mine, other) when `want_min`, else the larger
    auto keep = [&](uint64_t& km, uint32_t& pm, uint64_t ko, uint32_t po, bool want_min) {
        const bool mine_greater = greater(km, pm, ko, po);
        if (mine_greater == want_min) { km = ko; pm = po; }
    };
    for (int k = 2; k <= M; k <<= 1) {
        const bool up = ((2 * t) & k) == 0;              // the same for both items of the thread once k >= 2
        int j = k >> 1;
        for (; j >= 64; j >>= 1) {                       // partners live in another warp
            sk[2 * t] = k0; sk[2 * t + 1] = k1;
            if (kPayload) { sp[2 * t] = p0; sp[2 * t + 1] = p1; }
            __syncthreads();
            const int l = (2 * t) ^ j;
            const uint64_t ok0 = sk[l], ok1 = sk[l + 1];
            const uint32_t op0 = kPayload ? sp[l] : 0u, op1 = kPayload ? sp[l + 1] : 0u;
            __syncthreads();
            const bool lower = ((2 * t) & j) == 0;
            keep(k0, p0, ok0, op0, lower == up);
            keep(k1, p1, ok1, op1, lower == up);
        }
        for (; j >= 2; j >>= 1) {                        // partners live in the same warp
            const int m = j >> 1;
            const uint64_t ok0 = __shfl_xor_sync(0xffffffffu, k0, m), ok1 = __shfl_xor_sync(0xffffffffu, k1, m);
            const uint32_t op0 = kPayload ? __shfl_xor_sync(0xffffffffu, p0, m) : 0u, op1 = kPayload ? __shfl_xor_sync(0xffffffffu, p1, m) : 0u;
            const bool lower = (t & m) == 0;
            keep(k0, p0, ok0, op0, lower == up);
            keep(k1, p1, ok1, op1, lower == up);
        }
        if (greater(k0, p0, k1, p1) == up) {             // distance 1: the thread's own pair (up is taken at k >= 2; k = 2 sorts pairs
            const uint64_t tk = k0; k0 = k1; k1 = tk;    //              alternately up and down by bit 1 of the item index)
            const uint32_t tp = p0; p0 = p1; p1 = tp;
        }
    }
}

// exclusive scan of two values per thread (positions 2 tid and 2 tid + 1) over the CTA; returns the exclusive prefix
// of position 2 tid and the total
__device__ __forceinline__ int block_scan_pair(int v0, int v1, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    int v = v0 + v1;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += o;
    }
    __syncthreads();
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    int base = 0, tot = 0;
    for (int w = 0; w < n_warps; ++w) {
        const int sw = warp_sums[w];
        if (w < warp) base += sw;
        tot += sw;
    }
    *total = tot;
    return v + base - v0 - v1;
}

// launched with M / 2 threads (M >= 64 a power of two, N <= M)
__global__ void __launch_bounds__(kSmallMaxN / 2) select_small_kernel(const SelectParams P, int M) {
    extern __shared__ __align__(16) unsigned char sm_raw[];
    uint64_t* a = reinterpret_cast<uint64_t*>(sm_raw);            // [M] sorted keys, later sorted (group, priority, rank) codes
    uint32_t* idx = reinterpret_cast<uint32_t*>(a + M);           // [M] variate by sorted position
    int* gpos = reinterpret_cast<int*>(idx + M);                  // [M] group id by sorted position
    int* off_s = gpos + M;                                        // [M + 1] group offsets
    int* keep_s = off_s + M + 1;                                  // [M] kept flag by variate
    __shared__ int warp_sums[kSmallMaxN / 64];
    chain_wait();
    chain_release();
    const int s = blockIdx.x, N = P.N, tid = threadIdx.x;
    const uint64_t* keys = P.keys + static_cast<size_t>(s) * N;
    int32_t* members = P.members + static_cast<size_t>(s) * N;
    int32_t* gid = P.group_id + static_cast<size_t>(s) * N;
    int32_t* off = P.group_offsets + static_cast<size_t>(s) * (N + 1);
    int32_t* sel = P.sel_idx + static_cast<size_t>(s) * N;
    int32_t* inv = P.inv_idx + static_cast<size_t>(s) * N;
    const int p0 = 2 * tid, p1 = 2 * tid + 1;                     // the two items / positions this thread owns

    uint64_t k0 = p0 < N ? keys[p0] : ~0ull, k1 = p1 < N ? keys[p1] : ~0ull;
    uint32_t n0 = p0, n1 = p1;
    // Keys of up to 53 bits (k <= 4 frequencies of 12 bits, say) leave room for the variate index below them: one 64-bit
    // word per item orders by (key, index), and the sort moves a third less data per compare-exchange.
    constexpr int kIndexBits = 11;
    static_assert((1 << kIndexBits) >= kSmallMaxN, "index field too narrow");
    const bool wide = __syncthreads_or((p0 < N && (k0 >> (64 - kIndexBits)) != 0) || (p1 < N && (k1 >> (64 - kIndexBits)) != 0));
    if (!wide) {
        if (p0 < N) k0 = (k0 << kIndexBits) | n0;
        if (p1 < N) k1 = (k1 << kIndexBits) | n1;
        bitonic_sort_regs<false>(k0, n0, k1, n1, a, idx, M);
        n0 = static_cast<uint32_t>(k0) & ((1u << kIndexBits) - 1u);       // padding items (all ones) sort last and are never read
        n1 = static_cast<uint32_t>(k1) & ((1u << kIndexBits) - 1u);
        k0 >>= kIndexBits;
        k1 >>= kIndexBits;
    } else {
        bitonic_sort_regs<true>(k0, n0, k1, n1, a, idx, M);
    }
    a[p0] = k0; a[p1] = k1; idx[p0] = n0; idx[p1] = n1;
    __syncthreads();

    // group heads -> dense ids and offsets
    const int h0 = (p0 < N) && (p0 == 0 || k0 != a[p0 - 1]);
    const int h1 = (p1 < N) && (k1 != k0);
    int G = 0;
    const int before = block_scan_pair(h0, h1, warp_sums, &G);
    const int g0 = before + h0 - 1, g1 = before + h0 + h1 - 1;
    if (p0 < N) {
        gpos[p0] = g0;
        if (h0) { off_s[g0] = p0; off[g0] = p0; }
        members[p0] = n0;
        gid[n0] = g0;
    }
    if (p1 < N) {
        gpos[p1] = g1;
        if (h1) { off_s[g1] = p1; off[g1] = p1; }
        members[p1] = n1;
        gid[n1] = g1;
    }
    if (tid == 0) { off_s[G] = N; P.n_groups[s] = G; }
    for (int i = G + tid; i <= N; i += blockDim.x) off[i] = N;
    __syncthreads();

    // sampling rank: sort (group, priority, j)
    uint64_t c0 = ~0ull, c1 = ~0ull;
    if (p0 < N) {
        const int j = p0 - off_s[g0];
        const uint32_t pri = philox4x32_10_word0(static_cast<uint32_t>(j), static_cast<uint32_t>(g0), static_cast<uint32_t>(s), P.step, P.seed_lo, P.seed_hi);
        c0 = (static_cast<uint64_t>(g0) << 43) | (static_cast<uint64_t>(pri) << 11) | static_cast<uint64_t>(j);
    }
    if (p1 < N) {
        const int j = p1 - off_s[g1];
        const uint32_t pri = philox4x32_10_word0(static_cast<uint32_t>(j), static_cast<uint32_t>(g1), static_cast<uint32_t>(s), P.step, P.seed_lo, P.seed_hi);
        c1 = (static_cast<uint64_t>(g1) << 43) | (static_cast<uint64_t>(pri) << 11) | static_cast<uint64_t>(j);
    }
    uint32_t d0 = 0, d1 = 0;
    __syncthreads();                                              // everyone is done reading the sorted keys in `a`
    // Groups are usually small: a member's sampling rank is then the number of codes of its group below its own, counted over
    // the group's few positions.  Only when some group is long does the second sort pay.
    constexpr int kCountMaxGroup = 64;
    const int size0 = p0 < N ? off_s[g0 + 1] - off_s[g0] : 0, size1 = p1 < N ? off_s[g1 + 1] - off_s[g1] : 0;
    a[p0] = c0; a[p1] = c1;
    if (!__syncthreads_or(size0 > kCountMaxGroup || size1 > kCountMaxGroup)) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int p = 2 * tid + e;
            if (p < N) {
                const uint64_t mine = e ? c1 : c0;
                const int g = e ? g1 : g0;
                const int begin = off_s[g], end = off_s[g + 1];
                int below = 0;
                for (int o = begin; o < end; ++o) below += a[o] < mine;
                keep_s[idx[p]] = below < quota_of(end - begin, P.gs, P.rate_ppm);
            }
        }
    } else {
        bitonic_sort_regs<false>(c0, d0, c1, d1, a, nullptr, M);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int q = 2 * tid + e;
            const uint64_t c = e ? c1 : c0;
            if (q < N) {
                const int g = static_cast<int>(c >> 43), j = static_cast<int>(c & 2047u);
                const int begin = off_s[g], size = off_s[g + 1] - begin;
                keep_s[idx[begin + j]] = (q - begin) < quota_of(size, P.gs, P.rate_ppm);
            }
        }
    }
    __syncthreads();

    // compaction in ascending variate order
    const int kp0 = p0 < N ? keep_s[p0] : 0, kp1 = p1 < N ? keep_s[p1] : 0;
    int total = 0;
    int pos = block_scan_pair(kp0, kp1, warp_sums, &total);
    if (p0 < N) { if (kp0) { sel[pos] = p0; inv[p0] = pos; ++pos; } else inv[p0] = -1; }
    if (p1 < N) { if (kp1) { sel[pos] = p1; inv[p1] = pos; } else inv[p1] = -1; }
    for (int i = total + tid; i < N; i += blockDim.x) sel[i] = -1;
    if (tid == 0) P.n_sel[s] = total;
}

struct SelectWs {
    size_t done1, done2, lt, eq, prio, keep, total, zero_begin, zero_bytes;
};
SelectWs select_layout(int S, int N) {
    SelectWs w;
    size_t o = kWsHeaderBytes;
    w.zero_begin = o;
    w.done1 = o; o += align_up(sizeof(unsigned int) * S, 16);
    w.done2 = o; o += align_up(sizeof(unsigned int) * S, 16);
    w.lt = o;    o += align_up(sizeof(int32_t) * S * N, 16);
    w.eq = o;    o += align_up(sizeof(int32_t) * S * N, 16);
    w.zero_bytes = o - w.zero_begin;
    w.prio = o;  o += align_up(sizeof(uint32_t) * S * N, 16);
    w.keep = o;  o += align_up(sizeof(int32_t) * S * N, 16);
    w.total = o;
    return w;
}

}  // namespace

int select_validate(const vardrop_select_cfg& c) {
    if (c.S < 1 || c.S > 65535) return fail(VARDROP_ERR_INVALID_ARG, "select: S=%d outside 1..65535", c.S);
    if (c.N < 1 || c.N > 65536) return fail(VARDROP_ERR_INVALID_ARG, "select: N=%d outside 1..65536", c.N);
    if (!(c.rate > 0.0) || c.rate > 1.0) return fail(VARDROP_ERR_INVALID_ARG, "select: rate=%g outside (0, 1]", c.rate);
    return VARDROP_OK;
}

size_t select_workspace_bytes(const vardrop_select_cfg& c) { return select_layout(c.S, c.N).total; }

int select_launch(const uint64_t* keys, const vardrop_select_cfg& c, int32_t* group_id, int32_t* group_offsets, int32_t* members,
                  int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx, void* ws, cudaStream_t stream) {
    const SelectWs w = select_layout(c.S, c.N);
    char* base = static_cast<char*>(ws);
    SelectParams P{};
    P.keys = keys; P.group_id = group_id; P.group_offsets = group_offsets; P.members = members; P.n_groups = n_groups;
    P.sel_idx = sel_idx; P.n_sel = n_sel; P.inv_idx = inv_idx;
    P.status = reinterpret_cast<int*>(base);
    P.done1 = reinterpret_cast<unsigned int*>(base + w.done1);
    P.done2 = reinterpret_cast<unsigned int*>(base + w.done2);
    P.lt = reinterpret_cast<int32_t*>(base + w.lt);
    P.eq = reinterpret_cast<int32_t*>(base + w.eq);
    P.prio = reinterpret_cast<uint32_t*>(base + w.prio);
    P.keep = reinterpret_cast<int32_t*>(base + w.keep);
    P.S = c.S; P.N = c.N; P.gs = c.gs;
    P.rate_ppm = llround(c.rate * 1.0e6);
    P.seed_lo = static_cast<uint32_t>(c.seed & 0xFFFFFFFFu);
    P.seed_hi = static_cast<uint32_t>(c.seed >> 32);
    P.step = c.step;
    if (c.N <= kSmallMaxN) {
        int M = 64;
        while (M < c.N) M <<= 1;
        const size_t smem = static_cast<size_t>(M) * (8 + 4 + 4 + 4 + 4) + 16;
        static thread_local int attr_dev = -1;
        int dev = 0;
        cudaGetDevice(&dev);
        if (attr_dev != dev) {
            if (int st = check_cuda(cudaFuncSetAttribute(select_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024), "select: smem attribute")) return st;
            attr_dev = dev;
        }
        cudaError_t err;
        { LaunchScope ls_(K_SELECT_SMALL, stream); err = launch_chained(select_small_kernel, dim3(c.S), dim3(M / 2), smem, stream, P, M); }
        return check_cuda(err, "select: launch");
    }
    if (int st = check_cuda(cudaMemsetAsync(base + w.zero_begin, 0, w.zero_bytes, stream), "select: clear counters")) return st;
    const dim3 grid1((c.N + kSelThreads - 1) / kSelThreads, (c.N + kKeyChunk - 1) / kKeyChunk, c.S);
    cudaError_t err;
    { LaunchScope ls_(K_SELECT_COUNT, stream); err = launch_chained(select_count_kernel, grid1, dim3(kSelThreads), 0, stream, P); }
    if (int st = check_cuda(err, "select: count launch")) return st;
    const size_t group_smem = 3 * sizeof(int32_t) * static_cast<size_t>(c.N);
    if (group_smem <= kGroupMaxSmem) {
        static thread_local int group_attr_dev = -1;
        int dev = 0;
        cudaGetDevice(&dev);
        if (group_attr_dev != dev) {
            if (int st = check_cuda(cudaFuncSetAttribute(select_group_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kGroupMaxSmem)),
                                    "select: smem attribute")) return st;
            group_attr_dev = dev;
        }
        LaunchScope ls_(K_SELECT_GROUP, stream);
        err = launch_chained(select_group_kernel<true>, dim3(c.S), dim3(kTailThreads), group_smem, stream, P);
    } else {
        LaunchScope ls_(K_SELECT_GROUP, stream);
        err = launch_chained(select_group_kernel<false>, dim3(c.S), dim3(kTailThreads), 0, stream, P);
    }
    if (int st = check_cuda(err, "select: group launch")) return st;
    const dim3 grid2((c.N + kTailThreads - 1) / kTailThreads, 1, c.S);
    { LaunchScope ls_(K_SELECT_SAMPLE, stream); err = launch_chained(select_sample_kernel, grid2, dim3(kTailThreads), 0, stream, P); }
    return check_cuda(err, "select: sample launch");
}

// ---- allocation-free variant ------------------------------------------------------------------------------
// Scratch for vardrop_select_static: a fixed array that is part of the loaded module, so a caller that may not
// allocate device memory still has somewhere for the counters, ranks, priorities and keep flags to live.
// Sized for S * N <= kStaticMaxRows (worst case S = kStaticMaxRows, N = 1).
static __device__ __align__(256) unsigned char g_select_static_scratch[kStaticSelectBytes];

int select_static_launch(const uint64_t* keys, const vardrop_select_cfg& c, int32_t* group_id, int32_t* group_offsets, int32_t* members,
                         int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx, cudaStream_t stream) {
    if (static_cast<long long>(c.S) * c.N > kStaticMaxRows)
        return fail(VARDROP_ERR_UNSUPPORTED, "select_static: S*N = %lld exceeds the built-in scratch limit of %d; use vardrop_select with a workspace",
                    static_cast<long long>(c.S) * c.N, kStaticMaxRows);
    if (select_workspace_bytes(c) > static_cast<size_t>(kStaticSelectBytes))
        return fail(VARDROP_ERR_UNSUPPORTED, "select_static: layout of %zu bytes exceeds the built-in scratch of %d bytes",
                    select_workspace_bytes(c), kStaticSelectBytes);
    // The array's name is only a handle on the host; the device address is looked up once per device, with that
    // device current, and remembered.
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void* dev_ptr[kMaxDevices] = {};
    int dev = -1;
    if (int st = check_cuda(cudaGetDevice(&dev), "select_static: cudaGetDevice")) return st;
    if (dev < 0 || dev >= kMaxDevices) return fail(VARDROP_ERR_UNSUPPORTED, "select_static: device ordinal %d not supported", dev);
    void* ptr = nullptr;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!dev_ptr[dev]) {
            void* p = nullptr;
            if (int st = check_cuda(cudaGetSymbolAddress(&p, g_select_static_scratch), "select_static: cudaGetSymbolAddress")) return st;
            dev_ptr[dev] = p;
        }
        ptr = dev_ptr[dev];
    }
    return select_launch(keys, c, group_id, group_offsets, members, n_groups, sel_idx, n_sel, inv_idx, ptr, stream);
}

}  // namespace vardrop
