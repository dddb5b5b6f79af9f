/*
 * CPU oracle for the VarDrop per-batch training path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of what the path computes, written from the paper
 * (Kang et al., "VarDrop", AAAI-25): Algorithm 1 (k-dominant frequency hashing), the grouping rule at the
 * end of "Procedure of k-DFH", Eq. 1 and Eq. 2 (stratified sampling), the token-reduction ratio delta,
 * Eq. 3 (scaled dot-product attention) and its derivative.  It shares no code with the CUDA library and
 * is never called by it; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * No blocking, fusion or reordering beyond what the definitions state; OpenMP only spreads independent
 * (b, n) windows and (b, h) attention problems over cores.
 *
 * Pins (see tests/test_oracle_*.py): closed-form sinusoid spectra, Parseval, numpy's rfft, the theorem of
 * Appendix C, brute-force partitions, Eq. 1 / Eq. 2 / delta identities, Philox known answers and
 * frequency statistics, brute-force attention in pure Python, finite differences.  No function here is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define VDO_PI 3.14159265358979323846264338327950288

int vdo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------------------------------------------
 * Algorithm 1, step 1 ("Fast_Fourier_Transform", real amplitudes retained) and step 2 (low-pass filter):
 * amplitude spectrum of every window by direct summation of the DFT definition,
 *   X_f = sum_t x_t exp(-2 pi i f t / L),  A_f = |X_f|   (unnormalised),
 * for the candidate bins f_lo <= f < f_hi only (bins at or above the cut-off are removed).
 * x: [B, N, L] float32 (converted exactly to double);  amp: [B, N, f_hi - f_lo] double.
 * ------------------------------------------------------------------------------------------------- */
void vdo_dft_amplitudes(const float* x, int B, int N, int L, int f_lo, int f_hi, double* amp) {
    const int nf = f_hi - f_lo;
    double* c = (double*)malloc(sizeof(double) * (size_t)L);
    double* s = (double*)malloc(sizeof(double) * (size_t)L);
    for (int m = 0; m < L; ++m) {            /* the L distinct values of cos/sin(2 pi m / L) */
        c[m] = cos(2.0 * VDO_PI * (double)m / (double)L);
        s[m] = sin(2.0 * VDO_PI * (double)m / (double)L);
    }
    const long long W = (long long)B * N;
#pragma omp parallel for schedule(static)
    for (long long w = 0; w < W; ++w) {
        const float* xw = x + w * L;
        for (int f = f_lo; f < f_hi; ++f) {
            double re = 0.0, im = 0.0;
            for (int t = 0; t < L; ++t) {
                const int m = (int)(((long long)f * t) % L);
                re += (double)xw[t] * c[m];
                im -= (double)xw[t] * s[m];
            }
            amp[w * nf + (f - f_lo)] = sqrt(re * re + im * im);
        }
    }
    free(c);
    free(s);
}

/* ---------------------------------------------------------------------------------------------------
 * Algorithm 1, steps 3-5.
 *   step 3: abar[n, f] = (1/B) sum_b amp[b, n, f]            (scope 0, the paper's batch-wise grouping)
 *           abar[b, n, f] = amp[b, n, f]                      (scope 1: the algorithm run per instance)
 *   step 4: the k candidate bins of largest abar, in descending-amplitude order (Definition 1);
 *           equal amplitudes: the lower bin ranks first.
 *   step 5: hash value = the ordered k-tuple, packed 12 bits per bin with the rank-1 bin most significant
 *           (any injective code of the ordered tuple gives the same groups).
 * amp: [B, N, nf];  abar: [S, N, nf] (may be NULL);  freqs: [S, N, k];  keys: [S, N];  S = 1 or B.
 * ------------------------------------------------------------------------------------------------- */
void vdo_rank_and_pack(const double* amp, int B, int N, int nf, int f_lo, int k, int scope,
                       double* abar_out, int32_t* freqs, uint64_t* keys) {
    const int S = scope == 0 ? 1 : B;
    double* row = (double*)malloc(sizeof(double) * (size_t)nf);
    char* used = (char*)malloc((size_t)nf);
    for (int s = 0; s < S; ++s) {
        for (int n = 0; n < N; ++n) {
            for (int j = 0; j < nf; ++j) {
                if (scope == 0) {
                    double acc = 0.0;
                    for (int b = 0; b < B; ++b) acc += amp[((size_t)b * N + n) * nf + j];
                    row[j] = acc / (double)B;
                } else {
                    row[j] = amp[((size_t)s * N + n) * nf + j];
                }
                if (abar_out) abar_out[((size_t)s * N + n) * nf + j] = row[j];
            }
            memset(used, 0, (size_t)nf);
            uint64_t key = 0;
            for (int r = 0; r < k; ++r) {
                int best = -1;
                for (int j = 0; j < nf; ++j) {          /* ascending bin; strict '>' keeps the lower bin on ties */
                    if (used[j]) continue;
                    if (best < 0 || row[j] > row[best]) best = j;
                }
                used[best] = 1;
                freqs[((size_t)s * N + n) * k + r] = f_lo + best;
                key = (key << 12) | (uint64_t)(f_lo + best);
            }
            keys[(size_t)s * N + n] = key;
        }
    }
    free(row);
    free(used);
}

/* Algorithm 1 as a whole. */
void vdo_hash(const float* x, int B, int N, int L, int k, int f_lo, int f_hi, int scope,
              uint64_t* keys, int32_t* freqs, double* abar_out) {
    const int nf = f_hi - f_lo;
    double* amp = (double*)malloc(sizeof(double) * (size_t)B * N * nf);
    vdo_dft_amplitudes(x, B, N, L, f_lo, f_hi, amp);
    vdo_rank_and_pack(amp, B, N, nf, f_lo, k, scope, abar_out, freqs, keys);
    free(amp);
}

/* ---------------------------------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11):
 * ten rounds of  (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
 * with M0 = 0xD2511F53, M1 = 0xCD9E8D57, the key bumped by (0x9E3779B9, 0xBB67AE85) between rounds.
 * ------------------------------------------------------------------------------------------------- */
void vdo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ---------------------------------------------------------------------------------------------------
 * Grouping ("variates with the same hash value form a group") and stratified sampling (Eq. 1, Eq. 2).
 *
 * Groups: classes of equal key; group ids are dense ranks of the key in ascending key order; the members
 * of a group are listed by ascending variate index n.
 *
 * Quota of group g (Eq. 1 with the cap gs, composed with a proportional sampling rate and a floor of one):
 *   quota_g = min(|G_g|, gs if gs > 0, max(1, ceil(|G_g| * rate_ppm / 10^6))),  rate_ppm = round(rate * 10^6),
 * in 64-bit integer arithmetic.  rate = 1 gives Eq. 1 exactly.
 *
 * Random sampling inside a group: member j (its rank in ascending n) gets the priority
 *   word 0 of Philox4x32-10(counter = (j, g, s, step), key = (seed low 32 bits, seed high 32 bits));
 * S_g = the quota_g members of smallest (priority, j).  Eq. 2: the kept set is the union over groups,
 * listed by ascending n.
 *
 * keys: [S, N].  Outputs per scope s: group_id[S,N], group_offsets[S,N+1] (entries past G equal N),
 * members[S,N] (variates sorted by (key, n)), n_groups[S], sel_idx[S,N] (first n_sel valid, rest -1),
 * n_sel[S], inv_idx[S,N] (position of n in sel_idx, or -1 when dropped).
 * ------------------------------------------------------------------------------------------------- */
typedef struct { uint64_t key; int32_t n; } vdo_kn;
static int vdo_cmp_kn(const void* a, const void* b) {
    const vdo_kn* x = (const vdo_kn*)a; const vdo_kn* y = (const vdo_kn*)b;
    if (x->key != y->key) return x->key < y->key ? -1 : 1;
    return (x->n > y->n) - (x->n < y->n);
}
typedef struct { uint32_t pri; int32_t j; } vdo_pj;
static int vdo_cmp_pj(const void* a, const void* b) {
    const vdo_pj* x = (const vdo_pj*)a; const vdo_pj* y = (const vdo_pj*)b;
    if (x->pri != y->pri) return x->pri < y->pri ? -1 : 1;
    return (x->j > y->j) - (x->j < y->j);
}

int64_t vdo_quota(int64_t size, int32_t gs, double rate) {
    const int64_t rate_ppm = llround(rate * 1.0e6);
    int64_t by_rate = (size * rate_ppm + 999999) / 1000000;      /* ceil(size * rate) */
    if (by_rate < 1) by_rate = 1;
    int64_t q = size;
    if (gs > 0 && gs < q) q = gs;
    if (by_rate < q) q = by_rate;
    return q;
}

void vdo_select(const uint64_t* keys, int S, int N, int32_t gs, double rate, uint64_t seed, uint32_t step,
                int32_t* group_id, int32_t* group_offsets, int32_t* members, int32_t* n_groups,
                int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx) {
    if (N <= 0 || S <= 0) return;
    vdo_kn* kn = (vdo_kn*)malloc(sizeof(vdo_kn) * (size_t)N);
    vdo_pj* pj = (vdo_pj*)malloc(sizeof(vdo_pj) * (size_t)N);
    char* keep = (char*)malloc((size_t)N);
    const uint32_t pkey[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    for (int s = 0; s < S; ++s) {
        const uint64_t* ks = keys + (size_t)s * N;
        int32_t* gid = group_id + (size_t)s * N;
        int32_t* off = group_offsets + (size_t)s * (N + 1);
        int32_t* mem = members + (size_t)s * N;
        int32_t* sel = sel_idx + (size_t)s * N;
        int32_t* inv = inv_idx + (size_t)s * N;
        for (int n = 0; n < N; ++n) { kn[n].key = ks[n]; kn[n].n = n; }
        qsort(kn, (size_t)N, sizeof(vdo_kn), vdo_cmp_kn);
        int G = 0;
        for (int p = 0; p < N; ++p) {
            if (p == 0 || kn[p].key != kn[p - 1].key) { off[G] = p; ++G; }
            gid[kn[p].n] = G - 1;
            mem[p] = kn[p].n;
        }
        for (int g = G; g <= N; ++g) off[g] = N;
        n_groups[s] = G;
        memset(keep, 0, (size_t)N);
        for (int g = 0; g < G; ++g) {
            const int begin = off[g], size = off[g + 1] - off[g];
            const int64_t quota = vdo_quota(size, gs, rate);
            for (int j = 0; j < size; ++j) {
                const uint32_t ctr[4] = { (uint32_t)j, (uint32_t)g, (uint32_t)s, step };
                uint32_t r[4];
                vdo_philox4x32_10(ctr, pkey, r);
                pj[j].pri = r[0];
                pj[j].j = j;
            }
            qsort(pj, (size_t)size, sizeof(vdo_pj), vdo_cmp_pj);
            for (int64_t q = 0; q < quota; ++q) keep[mem[begin + pj[q].j]] = 1;
        }
        int cnt = 0;
        for (int n = 0; n < N; ++n) {
            if (keep[n]) { sel[cnt] = n; inv[n] = cnt; ++cnt; } else inv[n] = -1;
        }
        for (int p = cnt; p < N; ++p) sel[p] = -1;
        n_sel[s] = cnt;
    }
    free(kn); free(pj); free(keep);
}

/* ---------------------------------------------------------------------------------------------------
 * Token gather + Eq. 3 over the kept tokens, per (batch instance b, head h):
 *   Q' = Q[b, sel, h, :] (likewise K', V');  S = Q' K'^T * scale;  P = softmax over keys;  O' = P V';
 *   LSE_i = log sum_j exp(S_ij).
 * q, k, v: [B, N, H, D] double;  sel: [Ns] variate indices (NULL: all N tokens, the VarDrop-off path).
 * o: [B, Ns, H, D];  lse: [B, H, Ns].
 * ------------------------------------------------------------------------------------------------- */
void vdo_attn_fwd(const double* q, const double* k, const double* v, int B, int N, int H, int D,
                  const int32_t* sel, int Ns, double scale, double* o, double* lse) {
    if (!sel) Ns = N;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double* p = (double*)malloc(sizeof(double) * (size_t)Ns);
            for (int i = 0; i < Ns; ++i) {
                const int ni = sel ? sel[i] : i;
                const double* qi = q + (((size_t)b * N + ni) * H + h) * D;
                double mx = -INFINITY;
                for (int j = 0; j < Ns; ++j) {
                    const int nj = sel ? sel[j] : j;
                    const double* kj = k + (((size_t)b * N + nj) * H + h) * D;
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d) acc += qi[d] * kj[d];
                    p[j] = acc * scale;
                    if (p[j] > mx) mx = p[j];
                }
                double den = 0.0;
                for (int j = 0; j < Ns; ++j) { p[j] = exp(p[j] - mx); den += p[j]; }
                double* oi = o + (((size_t)b * Ns + i) * H + h) * D;
                for (int d = 0; d < D; ++d) oi[d] = 0.0;
                for (int j = 0; j < Ns; ++j) {
                    const int nj = sel ? sel[j] : j;
                    const double* vj = v + (((size_t)b * N + nj) * H + h) * D;
                    const double pij = p[j] / den;
                    for (int d = 0; d < D; ++d) oi[d] += pij * vj[d];
                }
                lse[((size_t)b * H + h) * Ns + i] = mx + log(den);
            }
            free(p);
        }
    }
}

/* ---------------------------------------------------------------------------------------------------
 * Derivative of Eq. 3 (the paper trains through it but does not print it; this is the chain rule):
 *   dV' = P^T dO';  dP = dO' V'^T;  Delta_i = sum_j P_ij dP_ij;  dS = P o (dP - Delta);
 *   dQ' = dS K' * scale;  dK' = dS^T Q' * scale.
 * Gradients go back to the full variate layout: row sel[i] of dq/dk/dv gets row i of dQ'/dK'/dV', every
 * dropped variate's row is exactly zero.
 * d_o: [B, Ns, H, D] gradient of the reduced output;  dq, dk, dv: [B, N, H, D].
 * ------------------------------------------------------------------------------------------------- */
void vdo_attn_bwd(const double* q, const double* k, const double* v, const double* d_o, int B, int N, int H, int D,
                  const int32_t* sel, int Ns, double scale, double* dq, double* dk, double* dv) {
    if (!sel) Ns = N;
    const size_t total = (size_t)B * N * H * D;
    memset(dq, 0, sizeof(double) * total);
    memset(dk, 0, sizeof(double) * total);
    memset(dv, 0, sizeof(double) * total);
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double* P = (double*)malloc(sizeof(double) * (size_t)Ns * Ns);
            double* dS = (double*)malloc(sizeof(double) * (size_t)Ns * Ns);
#define ROW(ptr, tok) ((ptr) + (((size_t)b * N + (sel ? sel[tok] : (tok))) * H + h) * D)
#define DOROW(tok) (d_o + (((size_t)b * Ns + (tok)) * H + h) * D)
            for (int i = 0; i < Ns; ++i) {
                const double* qi = ROW(q, i);
                double mx = -INFINITY, den = 0.0;
                for (int j = 0; j < Ns; ++j) {
                    const double* kj = ROW(k, j);
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d) acc += qi[d] * kj[d];
                    P[(size_t)i * Ns + j] = acc * scale;
                    if (acc * scale > mx) mx = acc * scale;
                }
                for (int j = 0; j < Ns; ++j) { P[(size_t)i * Ns + j] = exp(P[(size_t)i * Ns + j] - mx); den += P[(size_t)i * Ns + j]; }
                for (int j = 0; j < Ns; ++j) P[(size_t)i * Ns + j] /= den;
            }
            for (int i = 0; i < Ns; ++i) {
                const double* doi = DOROW(i);
                double delta = 0.0;
                for (int j = 0; j < Ns; ++j) {
                    const double* vj = ROW(v, j);
                    double dp = 0.0;
                    for (int d = 0; d < D; ++d) dp += doi[d] * vj[d];
                    dS[(size_t)i * Ns + j] = dp;                       /* dP for now */
                    delta += P[(size_t)i * Ns + j] * dp;
                }
                for (int j = 0; j < Ns; ++j)
                    dS[(size_t)i * Ns + j] = P[(size_t)i * Ns + j] * (dS[(size_t)i * Ns + j] - delta);
            }
            for (int i = 0; i < Ns; ++i) {                              /* dQ' = dS K' * scale */
                double* dqi = (double*)ROW(dq, i);
                for (int j = 0; j < Ns; ++j) {
                    const double* kj = ROW(k, j);
                    const double w = dS[(size_t)i * Ns + j] * scale;
                    for (int d = 0; d < D; ++d) dqi[d] += w * kj[d];
                }
            }
            for (int j = 0; j < Ns; ++j) {                              /* dK' = dS^T Q' * scale;  dV' = P^T dO' */
                double* dkj = (double*)ROW(dk, j);
                double* dvj = (double*)ROW(dv, j);
                for (int i = 0; i < Ns; ++i) {
                    const double* qi = ROW(q, i);
                    const double* doi = DOROW(i);
                    const double w = dS[(size_t)i * Ns + j] * scale;
                    const double pij = P[(size_t)i * Ns + j];
                    for (int d = 0; d < D; ++d) { dkj[d] += w * qi[d]; dvj[d] += pij * doi[d]; }
                }
            }
#undef ROW
#undef DOROW
            free(P); free(dS);
        }
    }
}

/* ---------------------------------------------------------------------------------------------------
 * Variate redundancy (Appendix A, Eq. 4): Pearson correlation coefficient between two variates of one
 * window,  rho(v, w) = sum_i (v_i - mean v)(w_i - mean w) / (sqrt(sum_i (v_i - mean v)^2) sqrt(sum_i (w_i - mean w)^2)),
 * and, per variate, its largest coefficient with any OTHER variate (the quantity whose histogram the
 * appendix shows, and whose share above 0.9 Sec. 1 quotes).  The paper does not say what a constant
 * variate gets (its denominator is zero): it is given rho = 0 with everything.
 *   x        [B, N, L] float32
 *   max_rho  [B, N]    for every instance: max over w != v of rho(v, w); -2 when N = 1 (no other variate)
 * ------------------------------------------------------------------------------------------------- */
void vdo_pearson_max(const float* x, int B, int N, int L, double* max_rho) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int v = 0; v < N; ++v) {
            const float* xv = x + ((size_t)b * N + v) * L;
            double mv = 0.0;
            for (int i = 0; i < L; ++i) mv += (double)xv[i];
            mv /= L;
            double svv = 0.0;
            for (int i = 0; i < L; ++i) svv += ((double)xv[i] - mv) * ((double)xv[i] - mv);
            double best = -2.0;
            for (int w = 0; w < N; ++w) {
                if (w == v) continue;
                const float* xw = x + ((size_t)b * N + w) * L;
                double mw = 0.0;
                for (int i = 0; i < L; ++i) mw += (double)xw[i];
                mw /= L;
                double sww = 0.0, svw = 0.0;
                for (int i = 0; i < L; ++i) {
                    sww += ((double)xw[i] - mw) * ((double)xw[i] - mw);
                    svw += ((double)xv[i] - mv) * ((double)xw[i] - mw);
                }
                const double den = sqrt(svv) * sqrt(sww);
                const double rho = den > 0.0 ? svw / den : 0.0;
                if (rho > best) best = rho;
            }
            max_rho[(size_t)b * N + v] = best;
        }
    }
}

/* ---------------------------------------------------------------------------------------------------
 * Token reduction on the raw window (Sec. 3.3): the kept variates of every instance, in the order of sel.
 *   x      [B, N, L] float32
 *   sel    [S, N] int32 (S = 1: one selection for the batch; S = B: one per instance), n_sel [S]
 *   x_sel  [B, N, L] float32: rows 0 .. n_sel-1 of instance b are x[b, sel[s(b), j], :]; other rows are left alone
 * ------------------------------------------------------------------------------------------------- */
void vdo_gather_rows(const float* x, int B, int N, int L, const int32_t* sel, const int32_t* n_sel, int S, float* x_sel) {
    for (int b = 0; b < B; ++b) {
        const int s = S > 1 ? b : 0;
        for (int j = 0; j < n_sel[s]; ++j)
            for (int t = 0; t < L; ++t)
                x_sel[((size_t)b * N + j) * L + t] = x[((size_t)b * N + sel[(size_t)s * N + j]) * L + t];
    }
}
