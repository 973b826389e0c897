// One-kernel stream step for bf16 caches (main loop of Algorithm 1: UpdateSoftmaxNormalizer, UpdateMatrixProduct,
// mu update, QueryStreamAttn; window of Section 3.2).
//
// The three-kernel step (insertion, cluster scan, value scan) is a chain of dependent launches: the query must see
// the state after the insertion. With few (sequence, KV head) units each of those kernels is short and the chain
// itself is the cost. Here one grid does the whole step in one pass over the state as it was BEFORE the insertion,
// and nobody waits for anybody:
//
//   every block   loads the queries, the token e that leaves the window and W(v_e); scans its slice of the packed
//                 representative heads for the nearest representative of k_e (as insert_mma_kernel does); then its
//                 warps take items from the unit's two queues: 16 clusters (partition function), or 16 slots of M /
//                 16 window rows (numerator). A warp starts in one role: cluster warps need no numerator
//                 accumulators and spend those registers on a second tile of rows in flight (cluster_scan with two
//                 tiles); when its queue is empty a warp helps with the other one.
//   M             which slots of M the token e replaces depends only on (seed, unit, e, slot, mu, W): the warp that
//                 scans a tile of M flips the tile's 16 coins itself, scores (k_e, v_e) with weight mu/(s W_e) in place
//                 of a replaced slot and writes the slot. No other warp touches that slot in this step.
//   window        the row the new token (k, v) will take is scored from the call's input instead of from the ring
//   last block    (arrival ticket) merges the slices' nearest representatives, decides join / open, and corrects the
//                 partition function for the one cluster that changes: it scores that cluster's t sample rows (or its
//                 representative) and k_e, and adds  new contribution - old contribution  as one more partial;
//                 then it applies the cluster update, stores the new token in the window, merges all partials and
//                 writes out = z / tau.
//
// mu after the insertion (mu + W_e) is known from the start, so the scan weights M with the final mu.
#pragma once
#include "subgen_insert_mma.cuh"

namespace sgk {

constexpr int kFsThreads = 256;
constexpr int kFsWarps = kFsThreads / 32;

// Scores of one 16-row tile against q without the softmax bookkeeping: sc = (row g, head 2tq), (g, 2tq+1),
// (g+8, 2tq), (g+8, 2tq+1).
template <int D>
__device__ __forceinline__ void tile_raw_scores(const uint4 (&ka)[D / 32], const uint4 (&kb)[D / 32], const uint32_t (&qb)[D / 32][4],
                                                float (&sc)[4]) {
    sc[0] = sc[1] = sc[2] = sc[3] = 0.f;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        mma_bf16_16816(sc, ka[c].x, kb[c].x, ka[c].y, kb[c].y, qb[c][0], qb[c][1]);
        mma_bf16_16816(sc, ka[c].z, kb[c].z, ka[c].w, kb[c].w, qb[c][2], qb[c][3]);
    }
}

// What a step knows about its two tokens once the unit's counters are read: the new token (k, v) of the call and the
// token e that leaves the window and is inserted into D and M (the new token itself when there is no window).
struct StepToken {
    int n;                            // tokens seen before this step
    int e;                            // index of the token that leaves the window (n - window)
    int slot;                         // window row both tokens use: e leaves it, the new token takes it
    bool has_ins;                     // a token leaves the window in this step
    unsigned long long W;             // W(v_e), 0 without insertion
    unsigned long long tot;           // mu after the insertion
    const __nv_bfloat16 *kE, *vE;     // rows of token e (in the window ring, or the call's input when window = 0)
    const __nv_bfloat16 *knew, *vnew; // rows of the new token (the call's input)
};

// Nearest representative of the key in krow over rows [c0, c1) of the unit's packed heads (Xu, Xhu, xhnu: the unit's
// representatives, their packed heads and the heads' squared norms): the tensor-core filter
// and exact follow-up of insert_mma_kernel. Warps take KT tiles of 16 heads per turn; every thread ends with the
// best (D2, index) its warp has seen (bst is updated, not reset).
template <int D, int KT>
__device__ __forceinline__ void head_scan_slice(const __nv_bfloat16* Xu, const __nv_bfloat16* Xhu, const float* xhnu,
                                                unsigned long long delta2_fx, int c0, int c1, const uint4* krow, int nwarps,
                                                Best& bst) {
    typedef __nv_bfloat16 T;
    constexpr int LPR = D / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, tq = lane & 3;
    uint32_t kb0[4];
    float kn = 0.f;
    {
        const uint4 r = krow[tq];
        float f[8];
        Elem<T>::unpack(r, f);
#pragma unroll
        for (int j = 0; j < 8; ++j) kn = fmaf(f[j], f[j], kn);
        kb0[0] = g == 0 ? r.x : 0u; kb0[1] = g == 0 ? r.y : 0u;
        kb0[2] = g == 0 ? r.z : 0u; kb0[3] = g == 0 ? r.w : 0u;
    }
    kn += __shfl_xor_sync(0xffffffffu, kn, 1);
    kn += __shfl_xor_sync(0xffffffffu, kn, 2);
    const float d2f = (float)((double)delta2_fx * (1.0 / 4294967296.0));
    auto exact_row = [&](int row) {                                  // exact D2 of one flagged row, by the warp
        unsigned long long acc = 0;
        if (lane < LPR) {
            float xf[8], kf[8];
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(Xu + (size_t)row * D + lane * 8), xf);
            Elem<T>::unpack(krow[lane], kf);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc += fx_sqdiff(xf[j], kf[j]);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (better(acc, row, bst)) { bst.d2 = acc; bst.idx = row; }
    };
    for (int base = c0 + warp * 16 * KT; base < c1; base += nwarps * 16 * KT) {
        uint4 ha[KT], hc[KT];
        float xa[KT], xb[KT];
#pragma unroll
        for (int i = 0; i < KT; ++i) {
            const int ra = base + i * 16 + g, rb = ra + 8;
            const bool va = ra < c1, vb = rb < c1;
            ha[i] = ldg16(Xhu + (size_t)(va ? ra : c1 - 1) * kHeadDims + tq * 8);
            hc[i] = ldg16(Xhu + (size_t)(vb ? rb : c1 - 1) * kHeadDims + tq * 8);
            xa[i] = va ? xhnu[ra] : 0.f;
            xb[i] = vb ? xhnu[rb] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < KT; ++i) {
            const int ra = base + i * 16 + g, rb = ra + 8;
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            mma_bf16_16816(sc, ha[i].x, hc[i].x, ha[i].y, hc[i].y, kb0[0], kb0[1]);
            mma_bf16_16816(sc, ha[i].z, hc[i].z, ha[i].w, hc[i].w, kb0[2], kb0[3]);
            const float na = xa[i] + kn, nb = xb[i] + kn;
            const bool fa = ra < c1 && tq == 0 && (na - 2.f * sc[0]) <= d2f + 1.220703125e-4f * na;
            const bool fb = rb < c1 && tq == 0 && (nb - 2.f * sc[2]) <= d2f + 1.220703125e-4f * nb;
            unsigned ma = __ballot_sync(0xffffffffu, fa), mb = __ballot_sync(0xffffffffu, fb);
            while (ma) { exact_row(base + i * 16 + ((__ffs(ma) - 1) >> 2)); ma &= ma - 1; }
            while (mb) { exact_row(base + i * 16 + 8 + ((__ffs(mb) - 1) >> 2)); mb &= mb - 1; }
        }
    }
}

// One warp's share of the numerator: items of 16 slots of M (weight mu/(s W), numerator only), then items of 16
// window rows (weight 1, numerator and partition function), on the state as it stands BEFORE the step's insertion,
// with the step's two changes made on the fly:
//   UpdateMatrixProduct  the warp flips the 16 value coins of its tile of M (four Philox blocks, while the rows are on
//                        their way), scores (k_e, v_e) with weight mu/(s W_e) in place of a slot that takes token e
//                        and writes that slot; no other warp touches the slot in this step;
//   window               the row the new token will take is scored from the call's input.
// first: the warp's first item; later ones are base + atomicAdd(counter, 1). krow / vrow: token e in shared memory.
template <int D>
__device__ __forceinline__ void value_scan(MmaState<D>& S, const uint32_t (&qb)[D / 32][4], const Cache<__nv_bfloat16>& C, int u,
                                           const StepToken& tk, const uint4* krow, const uint4* vrow, int first, unsigned* counter,
                                           int base_ticket) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, LPR = D / 8;
    const int lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
    const int w = C.w, s = C.s;
    const T* Mku = C.Mk + (size_t)u * s * D;
    const T* Mvu = C.Mv + (size_t)u * s * D;
    const float* MiWu = C.MinvW + (size_t)u * s;
    const T* Rk = C.ringK + (size_t)u * w * D;
    const T* Rv = C.ringV + (size_t)u * w * D;
    const unsigned long long W = tk.W, tot = tk.tot;
    const float mu_over_s = (float)tot / (float)s;
    const float inv_we = W ? 1.f / (float)W : 0.f;
    const int wn = min(tk.n + 1, w), slot = tk.slot;
    const int n_b = (s + 15) >> 4, n_v = n_b + ((wn + 15) >> 4);
    int item = first;
    while (item < n_v) {
        int next = 0;
        if (lane == 0) next = base_ticket + (int)atomicAdd(counter, 1u);     // asked for early, needed late
        const bool isM = item < n_b;
        const int base = (isM ? item : item - n_b) * 16;
        const int lim = isM ? s : wn;
        const T* Kb = isM ? Mku : Rk;
        const T* Vb = isM ? Mvu : Rv;
        const int ia = min(base + g, lim - 1), ib = min(base + g + 8, lim - 1);
        bool va = base + g < lim, vb = base + g + 8 < lim;
        const int iv[4] = {min(base + 2 * tq, lim - 1), min(base + 2 * tq + 1, lim - 1), min(base + 2 * tq + 8, lim - 1),
                           min(base + 2 * tq + 9, lim - 1)};
        const T* pka = Kb + (size_t)ia * D;
        const T* pkb = Kb + (size_t)ib * D;
        const T* pv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) pv[i] = Vb + (size_t)iv[i] * D;
        float wa_in = 1.f, wb_in = 1.f;
        unsigned sub = 0;                     // slots of this tile that take token e
        if (isM) {
            wa_in = MiWu[ia];                 // 1/W, 0 for a null slot
            wb_in = MiWu[ib];
        } else if (w && slot >= base && slot < base + 16) {
            // the new token's row: not in the ring yet, read from the call's input
            if (ia == slot) pka = tk.knew;
            if (ib == slot) pkb = tk.knew;
#pragma unroll
            for (int i = 0; i < 4; ++i) if (iv[i] == slot) pv[i] = tk.vnew;
        }
        uint4 ka[NC], kb[NC], v[4][D / 64];
        load_keys_stream<D>(pka, pkb, tq, ka, kb);           // keys and values in flight together
        load_values_stream<D>(pv, g, v);
        if (isM && W > 0) {
            unsigned nib = 0;
            if (lane < 4) {
                const int blk = (base >> 2) + lane;
                if (blk * 4 < s) {
                    const uint4 r = philox4x32_10(make_uint4((uint32_t)tk.e, unit_id(C, u), (uint32_t)blk, 1u), C.key0, C.key1);
                    const uint32_t words[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int qq = 0; qq < 4; ++qq)
                        if (blk * 4 + qq < s && coin_value(words[qq], tot, W)) nib |= 1u << qq;
                }
            }
            sub = __shfl_sync(0xffffffffu, nib, 0) | (__shfl_sync(0xffffffffu, nib, 1) << 4) |
                  (__shfl_sync(0xffffffffu, nib, 2) << 8) | (__shfl_sync(0xffffffffu, nib, 3) << 12);
            if (sub) {                        // rare: about s / (tokens inserted) slots per step
                if ((sub >> g) & 1u) { wa_in = inv_we; for (int c = 0; c < NC; ++c) ka[c] = ldg16(tk.kE + c * 32 + tq * 8); }
                if ((sub >> (g + 8)) & 1u) { wb_in = inv_we; for (int c = 0; c < NC; ++c) kb[c] = ldg16(tk.kE + c * 32 + tq * 8); }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = 2 * tq + (i & 1) + (i >> 1) * 8;
                    if ((sub >> r) & 1u)
                        for (int cc = 0; cc < D / 64; ++cc) v[i][cc] = ldg16(tk.vE + cc * 64 + g * 8);
                }
            }
        }
        float wza = 1.f, wzb = 1.f;
        if (isM) {
            va = va && wa_in != 0.f;
            vb = vb && wb_in != 0.f;
            wza = va ? mu_over_s * wa_in : 0.f;
            wzb = vb ? mu_over_s * wb_in : 0.f;
        }
        float p[4];
        tile_scores<D, D>(S, ka, kb, va, vb, qb, p);
        if (!isM) {
            S.tau0 += p[0] + p[2];
            S.tau1 += p[1] + p[3];
        }
        const float pz[4] = {wza * p[0], wza * p[1], wzb * p[2], wzb * p[3]};
        tile_values<D>(S, pz, v, g, tq);
        while (sub) {                         // the replaced slots take (k_e, v_e): half a warp per row
            const int i = base + __ffs(sub) - 1;
            sub &= sub - 1;
            if (lane < LPR) reinterpret_cast<uint4*>(C.Mk + ((size_t)u * s + i) * D)[lane] = krow[lane];
            else if (lane < 2 * LPR) reinterpret_cast<uint4*>(C.Mv + ((size_t)u * s + i) * D)[lane - LPR] = vrow[lane - LPR];
            if (lane == 31) {
                C.MW[(size_t)u * s + i] = W;
                C.MinvW[(size_t)u * s + i] = inv_we;
                C.Mtok[(size_t)u * s + i] = tk.e;
            }
        }
        item = __shfl_sync(0xffffffffu, next, 0);
    }
}

// The partition function changes in one cluster per step: token e joins cluster c (count + 1, some of its t slots
// take k_e) or opens a new one (weight 1). The scan saw the cluster as it was; this computes, per head,
//   pdl = new contribution - old contribution,  relative to the maximum pmx of the scores involved,
// from the scores of the cluster's sample rows (its representative while it is a singleton) and of k_e. The coins
// are the draws apply_cluster takes. Called by ONE warp; psc: shared [65][8]; pmx, pdl: shared [G]. Must run before
// apply_cluster overwrites the sample rows.
template <int D, int G>
__device__ __forceinline__ void tau_correction(const Cache<__nv_bfloat16>& C, int u, const StepToken& tk,
                                               const uint32_t (&qb)[D / 32][4], bool patched, bool joins, int c_join,
                                               float (*psc)[8], float* pmx, float* pdl) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32;
    const int lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
    const int t = C.t;
    if (!patched) {
        if (lane < G) { pmx[lane] = -INFINITY; pdl[lane] = 0.f; }
        return;
    }
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const T* Su = C.S + (size_t)u * C.m_max * t * D;
    const int c = joins ? c_join : 0;
    const int n_old = joins ? C.cnt[(size_t)u * C.m_max + c] : 0;
    const int nrow_old = !joins ? 0 : (n_old >= 2 ? t : 1);
    const int R = nrow_old + 1;
    auto rowptr = [&](int r) -> const T* {
        if (r >= nrow_old) return tk.kE;
        return n_old >= 2 ? Su + ((size_t)c * t + r) * D : Xu + (size_t)c * D;
    };
    for (int r0 = 0; r0 < R; r0 += 16) {
        const int ra = r0 + g, rb = r0 + g + 8;
        uint4 ka[NC], kb[NC];
        load_keys<D>(rowptr(min(ra, R - 1)), rowptr(min(rb, R - 1)), tq, ka, kb);
        float sc[4];
        tile_raw_scores<D>(ka, kb, qb, sc);
        if (ra < R) { psc[ra][2 * tq] = sc[0]; psc[ra][2 * tq + 1] = sc[1]; }
        if (rb < R) { psc[rb][2 * tq] = sc[2]; psc[rb][2 * tq + 1] = sc[3]; }
    }
    unsigned long long coins = 0;
    if (joins) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int j = half * 32 + lane;
            bool hit = false;
            if (j < t) {
                const uint4 r = philox4x32_10(make_uint4((uint32_t)tk.e, unit_id(C, u), (uint32_t)(j >> 2), 0u), C.key0, C.key1);
                const uint32_t word = (j & 3) == 0 ? r.x : (j & 3) == 1 ? r.y : (j & 3) == 2 ? r.z : r.w;
                hit = coin_cluster(word, (uint32_t)n_old + 1u);
            }
            coins |= (unsigned long long)__ballot_sync(0xffffffffu, hit) << (32 * half);
        }
    }
    __syncwarp();
    if (lane < G) {
        const float se = psc[nrow_old][lane];
        float mx = se;
        for (int r = 0; r < nrow_old; ++r) mx = fmaxf(mx, psc[r][lane]);
        const float ee = __expf(se - mx);
        float delta;
        if (!joins) {
            delta = ee;                                   // a new singleton cluster: weight 1
        } else if (n_old >= 2) {
            float so = 0.f, sn = 0.f;
            for (int j = 0; j < t; ++j) {
                const float ej = __expf(psc[j][lane] - mx);
                so += ej;
                sn += ((coins >> j) & 1ull) ? ee : ej;
            }
            delta = ((float)(n_old + 1) * sn - (float)n_old * so) / (float)t;
        } else {
            const float ex = __expf(psc[0][lane] - mx);
            const int ne = __popcll(coins);
            delta = 2.f * ((float)ne * ee + (float)(t - ne) * ex) / (float)t - ex;
        }
        pmx[lane] = mx;
        pdl[lane] = delta;
    }
}

// The token that leaves the window (kE, vE: its rows; has_ins = false: none leaves yet): its rows into krow / vrow,
// its weights into sm_w (range check reported through sm_bad), and the nearest representative of its key over this
// block's slice of the unit's representatives [0, m_scan) into sm_best. Called by the whole block; ends with a
// barrier. Kept out of line, with plain pointers as arguments, so that the kernel's two call sites share one copy
// and its registers do not weigh on the scans.
template <int D>
__device__ __noinline__ void leaving_token(const __nv_bfloat16* Xu, const __nv_bfloat16* Xhu, const float* xhnu,
                                           unsigned long long delta2_fx, const __nv_bfloat16* kE, const __nv_bfloat16* vE,
                                           bool has_ins, int m_scan, uint4* krow, uint4* vrow, unsigned long long* sm_w,
                                           int* sm_bad, Best* smb, Best* sm_best) {
    typedef __nv_bfloat16 T;
    constexpr int LPR = D / 8;
    const int tid = threadIdx.x, warp = tid >> 5, splits = gridDim.x;
    if (tid == 0) *sm_bad = 0;
    if (has_ins) {
        // past the L1: before the kernel's dependency wait nothing has refreshed this SM's view of the ring
        if (tid < LPR) krow[tid] = __ldcg(reinterpret_cast<const uint4*>(kE) + tid);
        else if (tid < 2 * LPR) vrow[tid - LPR] = __ldcg(reinterpret_cast<const uint4*>(vE) + (tid - LPR));
    }
    __syncthreads();
    if (has_ins && warp == 0) token_weights_rows<T, D>(krow, vrow, sm_w, sm_bad);
    __syncthreads();
    Best bst;
    bst.d2 = ~0ull; bst.idx = INT_MAX; bst.pad = 0;
    if (has_ins) {
        if (m_scan > 0) {
            const int per = (((m_scan + splits - 1) / splits) + 15) & ~15;       // slices are whole tiles
            const int c0 = blockIdx.x * per;
            head_scan_slice<D, 2>(Xu, Xhu, xhnu, delta2_fx, c0, min(m_scan, c0 + per), krow, kFsWarps, bst);
        }
        bst = block_best(bst, smb);
        if (tid == 0) *sm_best = bst;
    }
    __syncthreads();
}

template <int D, int G>
__global__ void __launch_bounds__(kFsThreads, 2) step_fused_kernel(Cache<__nv_bfloat16> C, const __nv_bfloat16* __restrict__ q,
                                                                  const __nv_bfloat16* __restrict__ k_new,
                                                                  const __nv_bfloat16* __restrict__ v_new,
                                                                  __nv_bfloat16* __restrict__ out, int step_k) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, LPR = D / 8, STR = D + 2, NW = kFsWarps;
    // During the scan every warp keeps the row list of its item here; afterwards the same bytes hold the warps'
    // partials [warp][G][D+2].
    constexpr int kListBytes = NW * (16 * 64 + 2 * kTauRows * 4);
    constexpr int kPartBytes = NW * G * STR * 4;
    constexpr int kScratchBytes = kListBytes > kPartBytes ? kListBytes : kPartBytes;
    __shared__ __align__(16) unsigned char scratch[kScratchBytes];
    __shared__ uint4 krow[LPR], vrow[LPR];
    __shared__ Best smb[32];
    __shared__ unsigned long long sm_w[2];
    __shared__ float psc[65][8];          // last block: raw scores of the changing cluster's rows and of k_e
    __shared__ float sred[16];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, tq = lane & 3;
    const int b = u / C.Hkv, kvh = u % C.Hkv;
    const size_t qrow0 = (size_t)b * C.H + (size_t)kvh * G;
    const int w = C.w, s = C.s, t = C.t, U = C.B * C.Hkv;
    const T* knew_u = k_new + (size_t)u * D;
    const T* vnew_u = v_new + (size_t)u * D;
    __shared__ int sm_bad;
    __shared__ Best sm_best;

    // ---- the token that leaves the window: its rows, its weights, its nearest representative ----
    // With a window of two rows or more none of this depends on the call's inputs or on the previous step: the
    // leaving token has been in the ring since an earlier step, the previous step writes another ring row, and
    // representatives never change once written. So it runs BEFORE the dependency wait, while the previous step's
    // last blocks finish: on the token count epoch + step_k (the epochs were set by a kernel that completed before
    // this one was launched) and on the representatives [0, m_hist): the cluster count left by the step before
    // the previous one, which has completed (the previous step passed its own wait before it let this kernel be
    // scheduled). The previous step can have opened at most one cluster beyond that; it is looked at after the wait.
    // Shorter windows (the leaving token is the previous step's, or the call's own) do all of it after the wait.
    const bool early = w >= 2;
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const T* Xhu = C.Xh + (size_t)u * C.m_max * kHeadDims;
    const float* xhnu = C.xhn + (size_t)u * C.m_max;
    int n_pre = -1, m_scan = 0;
    if (early) {
        n_pre = __ldcg(C.epoch + u) + step_k;
        m_scan = __ldcg(C.m_hist + (size_t)(step_k & 1) * U + u);
        const int slot_pre = n_pre % w;
        leaving_token<D>(Xu, Xhu, xhnu, C.delta2_fx, C.ringK + ((size_t)u * w + slot_pre) * D, C.ringV + ((size_t)u * w + slot_pre) * D,
                         n_pre >= w, m_scan, krow, vrow, sm_w, &sm_bad, smb, &sm_best);
    }
    // The call's inputs may come from the kernel that precedes this one in the stream: the rest waits for it.
    pdl_wait();
    pdl_trigger();

    uint32_t qb[NC][4];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        uint4 r = make_uint4(0, 0, 0, 0);
        if (g < G) r = ldg16(q + (qrow0 + g) * D + c * 32 + tq * 8);
        qb[c][0] = r.x; qb[c][1] = r.y; qb[c][2] = r.z; qb[c][3] = r.w;
    }
    const int n = C.n_unit[u], m = C.m_unit[u];
    const unsigned long long mu_old = C.mu[u];
    const bool has_ins = n >= w;                     // a token leaves the window (w = 0: the new token itself)
    const int e = n - w;
    const int slot = w ? n % w : 0;
    const T* kE = w ? C.ringK + ((size_t)u * w + slot) * D : knew_u;      // rows of the token that leaves
    const T* vE = w ? C.ringV + ((size_t)u * w + slot) * D : vnew_u;
    if (n != n_pre) {                                 // short window, or nothing prepared for this count
        m_scan = m;
        leaving_token<D>(Xu, Xhu, xhnu, C.delta2_fx, kE, vE, has_ins, m, krow, vrow, sm_w, &sm_bad, smb, &sm_best);
    }
    const unsigned long long W = has_ins ? sm_w[0] : 0ull;
    const unsigned long long tot = mu_old + W;       // mu after this step's insertion
    StepToken tk;
    tk.n = n; tk.e = e; tk.slot = slot; tk.has_ins = has_ins; tk.W = W; tk.tot = tot;
    tk.kE = kE; tk.vE = vE; tk.knew = knew_u; tk.vnew = vnew_u;
    if (has_ins && tid < 32) {
        Best bst = sm_best;
        // the cluster the previous step may have opened since the early scan: exact distance, read past the L1
        if (blockIdx.x == 0) {
            for (int row = m_scan; row < m; ++row) {
                unsigned long long acc = 0;
                if (lane < LPR) {
                    float xf[8], kf[8];
                    Elem<T>::unpack(__ldcg(reinterpret_cast<const uint4*>(Xu + (size_t)row * D + lane * 8)), xf);
                    Elem<T>::unpack(krow[lane], kf);
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc += fx_sqdiff(xf[j], kf[j]);
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (better(acc, row, bst)) { bst.d2 = acc; bst.idx = row; }
            }
        }
        if (tid == 0) {
            C.part1[(size_t)u * splits + blockIdx.x] = bst;
            if (sm_bad && blockIdx.x == 0) atomicOr(&C.status[u], 2);
        }
    }

    // ---- scan of the state as it stands before the insertion ----
    unsigned* als = reinterpret_cast<unsigned*>(scratch) + warp * (16 * 64 / 4);
    int* rix = reinterpret_cast<int*>(scratch + NW * 16 * 64) + warp * kTauRows;
    float* rwt = reinterpret_cast<float*>(scratch + NW * (16 * 64 + kTauRows * 4)) + warp * kTauRows;
    const int wn = min(n + 1, w);
    const int n_a = (m + 15) >> 4;
    // Roles. The unit's TW warps are dealt to the two queues in proportion to the rows behind them (cluster rows
    // are not counted anywhere: at most t per cluster and at most one per inserted token, at least one per cluster).
    const int TW = splits * NW, gw = blockIdx.x * NW + warp;
    int VW;
    {
        long long ec = min((long long)m * t, (long long)max(n - w, 0));
        ec = max(ec, (long long)m);
        const long long ev = 2ll * (s + wn);
        VW = (int)(((long long)TW * ev + (ev + ec) / 2) / (ev + ec));
        if (n_a == 0) VW = TW;
        else VW = TW == 1 ? 0 : max(1, min(VW, TW - 1));
    }
    const int CW = TW - VW;
    const int vi = (int)((long long)gw * VW / TW), ci = gw - vi;
    const bool is_v = (int)((long long)(gw + 1) * VW / TW) > vi;
    // the first ticket(s) of the queue this warp will help with later: asked for now, needed then
    int t1 = 0, t2 = 0;
    if (lane == 0) {
        if (is_v) {
            t1 = 2 * CW + (int)atomicAdd(&C.qnext[u], 1u);
            t2 = 2 * CW + (int)atomicAdd(&C.qnext[u], 1u);
        } else {
            t1 = VW + (int)atomicAdd(&C.qnext2[u], 1u);
        }
    }
    MmaState<D> S;
    {
        MmaState<16> SA;                  // cluster warps: running maxima and partition sums only
        SA.m0 = SA.m1 = -INFINITY;
        SA.tau0 = SA.tau1 = 0.f;
        SA.acc[0][0] = SA.acc[0][1] = SA.acc[0][2] = SA.acc[0][3] = 0.f;
        if (!is_v) cluster_scan<D, 16, 2>(SA, qb, C, u, m, ci, CW + ci, &C.qnext[u], 2 * CW, als, rix, rwt);
        S.m0 = SA.m0; S.m1 = SA.m1; S.tau0 = SA.tau0; S.tau1 = SA.tau1;
    }
#pragma unroll
    for (int j = 0; j < D / 16; ++j) S.acc[j][0] = S.acc[j][1] = S.acc[j][2] = S.acc[j][3] = 0.f;
    value_scan<D>(S, qb, C, u, tk, krow, vrow, is_v ? vi : __shfl_sync(0xffffffffu, t1, 0), &C.qnext2[u], VW);
    // value warps that are done help with whatever clusters are left (one tile in flight: the accumulators are live)
    if (is_v) cluster_scan<D, D, 1>(S, qb, C, u, m, __shfl_sync(0xffffffffu, t1, 0), __shfl_sync(0xffffffffu, t2, 0), &C.qnext[u],
                                    2 * CW, als, rix, rwt);
    __syncthreads();                                  // the row lists are dead: their bytes take the partials

    // ---- warp partial -> shared [warp][G][D+2] -> block partial in global memory ----
    float* smp = reinterpret_cast<float*>(scratch);
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        S.tau0 += __shfl_xor_sync(0xffffffffu, S.tau0, off);
        S.tau1 += __shfl_xor_sync(0xffffffffu, S.tau1, off);
    }
    {
        const int h0 = 2 * tq, h1 = 2 * tq + 1;
        float* w0 = smp + ((size_t)warp * G + (h0 < G ? h0 : 0)) * STR;
        float* w1 = smp + ((size_t)warp * G + (h1 < G ? h1 : 0)) * STR;
        if (g == 0) {
            if (h0 < G) { w0[0] = S.m0; w0[1] = S.tau0; }
            if (h1 < G) { w1[0] = S.m1; w1[1] = S.tau1; }
        }
#pragma unroll
        for (int j = 0; j < D / 16; ++j) {
            const int col = (j >> 2) * 64 + g * 8 + 2 * (j & 3);
            if (h0 < G) { w0[2 + col] = S.acc[j][0]; w0[2 + col + 1] = S.acc[j][2]; }
            if (h1 < G) { w1[2 + col] = S.acc[j][1]; w1[2 + col + 1] = S.acc[j][3]; }
        }
    }
    float* part_u = C.part2 + (size_t)u * splits * G * STR;
    block_combine<D, G>(smp, part_u + (size_t)blockIdx.x * G * STR);
    __syncthreads();
    if (splits > 1) {
        // arrival ticket: the release half of the atomic publishes this block's partials (ordered before it by the
        // barrier), the acquire half lets the last block read everybody else's
        if (tid == 0) {
            unsigned old;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(&C.ticket2[u]) : "memory");
            sm_last = (old == (unsigned)splits - 1u);
        }
        __syncthreads();
        if (!sm_last) return;
    }

    // ---- last block of the unit ----
    // Nearest representative over all slices, then two things side by side: warp 0 scores the one cluster that
    // changes (its sample rows, or its representative while it is a singleton, and k_e) and forms the correction
    // new contribution - old contribution of the partition function; the other warps merge the blocks' partials.
    Best bb;
    bb.d2 = ~0ull; bb.idx = INT_MAX; bb.pad = 0;
    bool joins = false, is_full = false;
    if (has_ins) {
        for (int i = tid; i < splits; i += kFsThreads) {
            const ulonglong2 raw = __ldcg(reinterpret_cast<const ulonglong2*>(C.part1 + (size_t)u * splits + i));
            const int idx = (int)(raw.y & 0xffffffffull);
            if (better(raw.x, idx, bb)) { bb.d2 = raw.x; bb.idx = idx; }
        }
        bb = block_best(bb, smb);
        joins = (m > 0) && (bb.d2 <= C.delta2_fx);
        is_full = !joins && (m >= C.m_max);
    }
    const bool patched = has_ins && !is_full;
    float* pmx = sred;                                // [G] maximum the correction is relative to
    float* pdl = sred + 8;                            // [G] the correction
    if (warp == 0) tau_correction<D, G>(C, u, tk, qb, patched, joins, bb.idx, psc, pmx, pdl);
    // Merge of the blocks' partials {max, tau, z[D]}, first half: per head the maximum over the partials, the
    // partition sum under it and every partial's factor exp(max_i - max) (warps 1.. while warp 0 is busy above).
    float* fac = smp;                                 // [splits][8]
    float* hmx = smp + 128 * 8;                       // [G] maximum over the partials
    float* htau = hmx + 8;                            // [G] partition sum relative to it
    float4* zsum = reinterpret_cast<float4*>(smp + 128 * 8 + 16);    // [kFsThreads] column quads per group of partials
    if (warp > 0) {
        for (int hh = warp - 1; hh < G; hh += NW - 1) {
            float mx = -INFINITY;
            float2 ph[4];                             // splits <= 128: four partials per lane
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = lane + 32 * k;
                ph[k] = make_float2(-INFINITY, 0.f);
                if (i < splits) ph[k] = __ldcg(reinterpret_cast<const float2*>(part_u + ((size_t)i * G + hh) * STR));
                mx = fmaxf(mx, ph[k].x);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            float tau = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = lane + 32 * k;
                const float f = ph[k].x == -INFINITY ? 0.f : __expf(ph[k].x - mx);
                if (i < splits) fac[i * 8 + hh] = f;
                tau = fmaf(ph[k].y, f, tau);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) tau += __shfl_xor_sync(0xffffffffu, tau, off);
            if (lane == 0) { hmx[hh] = mx; htau[hh] = tau; }
        }
    }
    __syncthreads();                                  // the correction is in shared memory; the old sample rows were read
    int m_after = m;
    if (has_ins) {
        bool join2, full2;
        int m_ref = m;
        const int m_new = apply_cluster<T, D, false>(C, u, e, bb, m_ref, krow, sm_w, join2, full2);
        m_after = m_new;
        if (tid == 0) {
            C.mu[u] = tot;
            C.m_unit[u] = m_new;
            C.last_cid[u] = join2 ? bb.idx : (full2 ? -1 : m);
            C.last_open[u] = join2 ? 0 : 1;
            C.last_d2[u] = bb.d2;
        }
    }
    if (w) {                                          // the new token takes the window row the leaving one had
        uint4* ringk = reinterpret_cast<uint4*>(C.ringK + ((size_t)u * w + slot) * D);
        uint4* ringv = reinterpret_cast<uint4*>(C.ringV + ((size_t)u * w + slot) * D);
        if (tid < LPR) ringk[tid] = reinterpret_cast<const uint4*>(knew_u)[tid];
        else if (tid < 2 * LPR) ringv[tid - LPR] = reinterpret_cast<const uint4*>(vnew_u)[tid - LPR];
    }
    __syncthreads();                                  // status bits of this step are set
    const bool poisoned = C.status[u] != 0;
    // second half: the numerators. A thread takes one quad of neighbouring columns and every P-th partial, so that
    // all its loads are independent; the P groups meet in shared memory.
    constexpr int NQ = G * D / 4, P = kFsThreads / NQ;
    {
        const int qd = tid % NQ, pg = tid / NQ;
        const int hh = (4 * qd) / D, cc = (4 * qd) % D;
        float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i0 = pg; i0 < splits; i0 += 8 * P) {
            float4 pz[8];
            float f[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = i0 + k * P;
                f[k] = i < splits ? fac[i * 8 + hh] : 0.f;
                // rows of a partial start 8 bytes into a 16-byte slot pattern (D + 2 floats): two 8-byte loads
                const float* pp = part_u + ((size_t)min(i, splits - 1) * G + hh) * STR + 2 + cc;
                const float2 lo = __ldcg(reinterpret_cast<const float2*>(pp)), hi = __ldcg(reinterpret_cast<const float2*>(pp + 2));
                pz[k] = make_float4(lo.x, lo.y, hi.x, hi.y);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                acc4.x = fmaf(pz[k].x, f[k], acc4.x); acc4.y = fmaf(pz[k].y, f[k], acc4.y);
                acc4.z = fmaf(pz[k].z, f[k], acc4.z); acc4.w = fmaf(pz[k].w, f[k], acc4.w);
            }
        }
        zsum[tid] = acc4;
    }
    __syncthreads();
    if (tid < NQ) {
        const int hh = (4 * tid) / D, cc = (4 * tid) % D;
        float4 z = zsum[tid];
#pragma unroll
        for (int pg = 1; pg < P; ++pg) {
            const float4 o = zsum[pg * NQ + tid];
            z.x += o.x; z.y += o.y; z.z += o.z; z.w += o.w;
        }
        const float mf = fmaxf(hmx[hh], pmx[hh]);
        const float fa = hmx[hh] == -INFINITY ? 0.f : __expf(hmx[hh] - mf);
        const float fb = pmx[hh] == -INFINITY ? 0.f : __expf(pmx[hh] - mf);
        const float tau = htau[hh] * fa + pdl[hh] * fb;
        const float sc = tau > 0.f ? fa / tau : 0.f;
        float r0 = z.x * sc, r1 = z.y * sc, r2 = z.z * sc, r3 = z.w * sc;
        if (poisoned) r0 = r1 = r2 = r3 = __int_as_float(0x7fc00000);
        __nv_bfloat162* dst = reinterpret_cast<__nv_bfloat162*>(out + qrow0 * D + (size_t)hh * D + cc);
        dst[0] = __floats2bfloat162_rn(r0, r1);
        dst[1] = __floats2bfloat162_rn(r2, r3);
    }
    if (tid == 0) {
        C.n_unit[u] = n + 1;
        C.m_hist[(size_t)(step_k & 1) * U + u] = m_after;     // read by the step after the next one, before its wait
        C.ticket2[u] = 0;
        C.qnext[u] = 0;
        C.qnext2[u] = 0;
    }
}

}  // namespace sgk
