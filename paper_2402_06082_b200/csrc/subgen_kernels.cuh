// Kernels of the SubGen stream step, the token-by-token prefill and the exact comparison path.
#pragma once
#include <limits.h>

#include "subgen_device.cuh"

namespace sgk {

constexpr int kInsertThreads = 256;
constexpr int kQueryThreads = 256;
constexpr int kPrefillThreads = 512;

// ---------------------------------------------------------------------------------------------
// Step kernel 1: window push + insertion of the token that leaves the window.
// grid (splits, U). Each block scans a slice of the unit's representatives for the nearest one
// (procedure UpdateSoftmaxNormalizer, argmin), the block that finishes last merges the slices and
// applies the update (join/open, coins, UpdateMatrixProduct, mu) and then stores the new token in
// the window row the old one occupied. Nothing waits on another block.
template <typename T, int D, bool BND>
__global__ void __launch_bounds__(kInsertThreads) insert_kernel(Cache<T> C, const T* __restrict__ k_new,
                                                                const T* __restrict__ v_new) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR;
    __shared__ uint4 krow[LPR], vrow[LPR];
    __shared__ Best smb[32];
    __shared__ unsigned long long sm_w[2];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, lr = lane % LPR, sub = lane / LPR;
    // first kernel of a step: everything earlier in the stream has completed before it reads anything; the query
    // kernel may be scheduled at once (it loads its queries and then waits for this kernel)
    pdl_wait();
    pdl_trigger();
    const int n = C.n_unit[u], w = C.w;
    const uint4* knew_u = reinterpret_cast<const uint4*>(k_new + (size_t)u * D);
    const uint4* vnew_u = reinterpret_cast<const uint4*>(v_new + (size_t)u * D);
    const int slot = w ? n % w : 0;
    uint4* ringk = w ? reinterpret_cast<uint4*>(C.ringK + ((size_t)u * w + slot) * D) : nullptr;
    uint4* ringv = w ? reinterpret_cast<uint4*>(C.ringV + ((size_t)u * w + slot) * D) : nullptr;
    if (w && n < w) {                       // window not full yet: nothing leaves it
        if (blockIdx.x == 0) {
            if (tid < LPR) ringk[tid] = knew_u[tid];
            else if (tid < 2 * LPR) ringv[tid - LPR] = vnew_u[tid - LPR];
        }
        return;
    }
    const int e = n - w;                    // the token that leaves (the new token itself when w = 0)
    if (tid < LPR) krow[tid] = w ? ringk[tid] : knew_u[tid];
    __syncthreads();
    const int m = C.m_unit[u];
    float kf[EPL];
    Elem<T>::unpack(krow[lr], kf);
    const int per = (m + splits - 1) / splits;
    const int c0 = blockIdx.x * per, c1 = min(m, c0 + per);
    Best b;
    b.d2 = ~0ull; b.idx = INT_MAX; b.pad = 0;
    scan_centres<T, D>(C.X + (size_t)u * C.m_max * D, c0, c1, kf, warp * RPW + sub, (nt >> 5) * RPW, lr, b);
    b = block_best(b, smb);
    if (splits > 1) {
        if (tid == 0) {
            C.part1[(size_t)u * splits + blockIdx.x] = b;
            __threadfence();
            sm_last = (atomicAdd(&C.ticket1[u], 1u) == (unsigned)splits - 1u);
        }
        __syncthreads();
        if (!sm_last) return;
        __threadfence();
        Best bb;
        bb.d2 = ~0ull; bb.idx = INT_MAX; bb.pad = 0;
        for (int i = tid; i < splits; i += nt) {
            const ulonglong2 raw = __ldcg(reinterpret_cast<const ulonglong2*>(C.part1 + (size_t)u * splits + i));
            const int idx = (int)(raw.y & 0xffffffffull);
            if (better(raw.x, idx, bb)) { bb.d2 = raw.x; bb.idx = idx; }
        }
        b = block_best(bb, smb);
        if (tid == 0) C.ticket1[u] = 0;
    }
    if (tid < LPR) vrow[tid] = w ? ringv[tid] : vnew_u[tid];
    __syncthreads();
    apply_insert<T, D, BND>(C, u, e, b, m, krow, vrow, sm_w);
    if (w) {
        if (tid < LPR) ringk[tid] = knew_u[tid];
        else if (tid < 2 * LPR) ringv[tid - LPR] = vnew_u[tid - LPR];
    }
}

// ---------------------------------------------------------------------------------------------
// Step kernel 2: procedure QueryStreamAttn over the updated state plus the window terms.
// grid (splits, U). Row groups stride over (a) clusters: t sample rows weighted n'/t, or the
// representative alone with weight 1 while n' = 1; (b) M slots: key and value row, weight
// mu/(s W); (c) window rows, weight 1 in both sums. The G query heads of a KV head share every
// load. Blocks write (max, tau, z) partials; the block that finishes last merges them, divides,
// writes out and advances the unit's token count.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kQueryThreads) query_kernel(Cache<T> C, const T* __restrict__ q, T* __restrict__ out, int advance) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR, STR = D + 2;
    __shared__ float sm[(kQueryThreads / 32) * G * STR];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, lr = lane % LPR, sub = lane / LPR;
    const int b = u / C.Hkv, kvh = u % C.Hkv;
    const size_t qrow0 = (size_t)b * C.H + (size_t)kvh * G;

    // the queries are an input of the call (complete before its first kernel ran); the state is the insertion's
    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint4 r = *reinterpret_cast<const uint4*>(q + (qrow0 + g) * D + lr * EPL);
        Elem<T>::unpack(r, qf[g]);
    }
    pdl_wait();
    pdl_trigger();
    // advance = 1: the query of a stream step (its token is in the ring, not counted yet); 0: read-only query
    const int n = C.n_unit[u] - (advance ? 0 : 1), w = C.w, t = C.t, s = C.s;
    const int wn = min(n + 1, w), m = C.m_unit[u];
    Acc<G, EPL> A;
    A.init();
    const int gg = (blockIdx.x * (kQueryThreads / 32) + warp) * RPW + sub;
    const int GG = splits * (kQueryThreads / 32) * RPW;

    {   // (a) clusters
        constexpr int UN = 4;
        const T* Xu = C.X + (size_t)u * C.m_max * D;
        const T* Su = C.S + (size_t)u * C.m_max * t * D;
        const int* cntu = C.cnt + (size_t)u * C.m_max;
        const float inv_t = 1.f / (float)t;
        for (int cb = 0; cb < m; cb += GG) {
            const int c = cb + gg;
            const int cn = c < m ? cntu[c] : 0;
            const int rows = cn == 1 ? 1 : (cn > 1 ? t : 0);
            const T* src = cn == 1 ? Xu + (size_t)c * D : Su + (size_t)c * t * D;
            const float wt = cn == 1 ? 1.f : (float)cn * inv_t;
            const int rmax = __reduce_max_sync(0xffffffffu, rows);
            for (int j0 = 0; j0 < rmax; j0 += UN) {
                uint4 kraw[UN], vdummy[UN];
                bool valid[UN];
                float wt_tau[UN], wt_z[UN];
#pragma unroll
                for (int i = 0; i < UN; ++i) {
                    valid[i] = j0 + i < rows;
                    wt_tau[i] = wt; wt_z[i] = 0.f;
                    kraw[i] = make_uint4(0, 0, 0, 0);
                    vdummy[i] = kraw[i];
                    if (valid[i]) kraw[i] = *reinterpret_cast<const uint4*>(src + (size_t)(j0 + i) * D + lr * EPL);
                }
                float sc[UN][G];
                scores<T, D, G, UN>(kraw, qf, sc);
                fold<T, D, G, UN, false>(A, sc, valid, wt_tau, wt_z, vdummy);
            }
        }
    }
    {   // (b) value samples M
        constexpr int UN = 2;
        const T* Mku = C.Mk + (size_t)u * s * D;
        const T* Mvu = C.Mv + (size_t)u * s * D;
        const unsigned long long* MWu = C.MW + (size_t)u * s;
        const float mu_over_s = (float)C.mu[u] / (float)s;
        for (int ib = 0; ib < s; ib += GG * UN) {
            uint4 kraw[UN], vraw[UN];
            bool valid[UN];
            float wt_tau[UN], wt_z[UN];
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int idx = ib + i * GG + gg;
                const unsigned long long Wi = idx < s ? MWu[idx] : 0ull;
                valid[i] = Wi != 0ull;
                wt_tau[i] = 0.f;
                wt_z[i] = valid[i] ? mu_over_s / (float)Wi : 0.f;
                kraw[i] = make_uint4(0, 0, 0, 0);
                vraw[i] = kraw[i];
                if (valid[i]) {
                    kraw[i] = *reinterpret_cast<const uint4*>(Mku + (size_t)idx * D + lr * EPL);
                    vraw[i] = *reinterpret_cast<const uint4*>(Mvu + (size_t)idx * D + lr * EPL);
                }
            }
            float sc[UN][G];
            scores<T, D, G, UN>(kraw, qf, sc);
            fold<T, D, G, UN, true>(A, sc, valid, wt_tau, wt_z, vraw);
        }
    }
    {   // (c) window
        constexpr int UN = 2;
        const T* Rk = C.ringK + (size_t)u * w * D;
        const T* Rv = C.ringV + (size_t)u * w * D;
        for (int jb = 0; jb < wn; jb += GG * UN) {
            uint4 kraw[UN], vraw[UN];
            bool valid[UN];
            float wt_tau[UN], wt_z[UN];
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int idx = jb + i * GG + gg;
                valid[i] = idx < wn;
                wt_tau[i] = 1.f; wt_z[i] = 1.f;
                kraw[i] = make_uint4(0, 0, 0, 0);
                vraw[i] = kraw[i];
                if (valid[i]) {
                    kraw[i] = *reinterpret_cast<const uint4*>(Rk + (size_t)idx * D + lr * EPL);
                    vraw[i] = *reinterpret_cast<const uint4*>(Rv + (size_t)idx * D + lr * EPL);
                }
            }
            float sc[UN][G];
            scores<T, D, G, UN>(kraw, qf, sc);
            fold<T, D, G, UN, true>(A, sc, valid, wt_tau, wt_z, vraw);
        }
    }

    float* part_u = C.part2 + (size_t)u * splits * G * STR;
    block_partial<T, D, G>(A, sm, part_u + (size_t)blockIdx.x * G * STR);
    __threadfence();
    __syncthreads();
    if (splits > 1) {
        if (tid == 0) {
            __threadfence();
            sm_last = (atomicAdd(&C.ticket2[u], 1u) == (unsigned)splits - 1u);
        }
        __syncthreads();
        if (!sm_last) return;
        __threadfence();
    }
    final_merge<T, D, G>(part_u, splits, out + qrow0 * D, C.status[u] != 0);
    if (tid == 0) {
        if (advance) C.n_unit[u] = n + 1;
        C.ticket2[u] = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// Token-by-token prefill: one block per unit replays the insertion of every token that leaves the
// window, in stream order, then stores the tokens that stay in the window. By construction the state
// equals that of the same number of stream steps.
// Rows of unit (b, h): K + (row0 + i) * D, row0 = (b*Hkv + h) * n_add (dense [B,Hkv,n,D]) or
// h * total + cu[b] (packed [Hkv,total,D]).
template <typename T, int D, bool BND>
__global__ void __launch_bounds__(kPrefillThreads) prefill_seq_kernel(Cache<T> C, const T* __restrict__ K,
                                                                      const T* __restrict__ V, int n_uniform,
                                                                      const int* __restrict__ cu, int total) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR;
    __shared__ uint4 krow[LPR], vrow[LPR];
    __shared__ Best smb[32];
    __shared__ unsigned long long sm_w[2];
    const int u = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, lr = lane % LPR, sub = lane / LPR;
    const int b = u / C.Hkv, h = u % C.Hkv, w = C.w;
    const int n_add = cu ? cu[b + 1] - cu[b] : n_uniform;
    const size_t row0 = cu ? (size_t)h * total + cu[b] : (size_t)u * n_uniform;
    const int n_prev = C.n_unit[u], n_tot = n_prev + n_add;
    const int ins_lo = max(0, n_prev - w), ins_hi = max(0, n_tot - w);
    int m = C.m_unit[u];
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    for (int e = ins_lo; e < ins_hi; ++e) {
        const T* ks = e < n_prev ? C.ringK + ((size_t)u * w + e % w) * D : K + (row0 + (e - n_prev)) * D;
        const T* vs = e < n_prev ? C.ringV + ((size_t)u * w + e % w) * D : V + (row0 + (e - n_prev)) * D;
        if (tid < LPR) krow[tid] = reinterpret_cast<const uint4*>(ks)[tid];
        else if (tid < 2 * LPR) vrow[tid - LPR] = reinterpret_cast<const uint4*>(vs)[tid - LPR];
        __syncthreads();
        float kf[EPL];
        Elem<T>::unpack(krow[lr], kf);
        Best bst;
        bst.d2 = ~0ull; bst.idx = INT_MAX; bst.pad = 0;
        scan_centres<T, D>(Xu, 0, m, kf, warp * RPW + sub, (nt >> 5) * RPW, lr, bst);
        bst = block_best(bst, smb);
        m = apply_insert<T, D, BND>(C, u, e, bst, m, krow, vrow, sm_w);
    }
    if (w) {
        const int lo = max(n_prev, n_tot - w);
        for (int p = tid; p < (n_tot - lo) * LPR; p += nt) {
            const int tok = lo + p / LPR, part = p % LPR;
            reinterpret_cast<uint4*>(C.ringK + ((size_t)u * w + tok % w) * D)[part] =
                reinterpret_cast<const uint4*>(K + (row0 + (tok - n_prev)) * D)[part];
            reinterpret_cast<uint4*>(C.ringV + ((size_t)u * w + tok % w) * D)[part] =
                reinterpret_cast<const uint4*>(V + (row0 + (tok - n_prev)) * D)[part];
        }
    }
    if (tid == 0) C.n_unit[u] = n_tot;
}

// ---------------------------------------------------------------------------------------------
// Sums for subgen_cache_stats: out[0..6] = clusters, singleton clusters, filled M slots, window rows,
// tokens, pairs scored by the prefill, distinct sample rows of the clusters with more than one member.
template <typename T>
__global__ void stats_kernel(Cache<T> C, int U, unsigned long long* out) {
    const int u = blockIdx.x;
    if (u >= U) return;
    const int m = C.m_unit[u], n = C.n_unit[u];
    unsigned long long single = 0, filled = 0;
    unsigned long long distinct = 0;
    for (int c = threadIdx.x; c < m; c += blockDim.x) {
        const bool one = C.cnt[(size_t)u * C.m_max + c] == 1;
        single += one;
        if (!one) distinct += C.ndist[(size_t)u * C.m_max + c];
    }
    atomicAdd(&out[6], distinct);
    for (int i = threadIdx.x; i < C.s; i += blockDim.x) filled += C.MW[(size_t)u * C.s + i] != 0ull;
    atomicAdd(&out[1], single);
    atomicAdd(&out[2], filled);
    if (threadIdx.x == 0) {
        atomicAdd(&out[0], (unsigned long long)m);
        atomicAdd(&out[3], (unsigned long long)min(n, C.w));
        atomicAdd(&out[4], (unsigned long long)n);
        atomicAdd(&out[5], C.pairs[u]);
    }
}

// ---------------------------------------------------------------------------------------------
// Exact comparison path (Eq. 1): full per-unit KV cache.
template <typename T> struct ExactCache {
    int B, H, Hkv, G, n_max;
    T* Kc;           // [U, n_max, D]
    T* Vc;
    int* n_unit;     // [U]
    float* part;     // [U, splits, G, D + 2]
    unsigned* ticket;
    unsigned* qnext; // [U] work queue of the tensor-core kernel
    int* tok;        // [U, n_max] stream position of the token in each cache row
    int* pos;        // [U] tokens ever appended (differs from n_unit after a compression)
};

template <typename T, int D>
__global__ void exact_append_kernel(ExactCache<T> E, const T* __restrict__ K, const T* __restrict__ V, int n_uniform,
                                    const int* __restrict__ cu, int total) {
    constexpr int LPR = D / Elem<T>::EPL;
    const int u = blockIdx.y, b = u / E.Hkv, h = u % E.Hkv;
    const int n_add = cu ? cu[b + 1] - cu[b] : n_uniform;
    const size_t row0 = cu ? (size_t)h * total + cu[b] : (size_t)u * n_uniform;
    const int n_prev = E.n_unit[u];
    const uint4* ks = reinterpret_cast<const uint4*>(K + row0 * D);
    const uint4* vs = reinterpret_cast<const uint4*>(V + row0 * D);
    uint4* kd = reinterpret_cast<uint4*>(E.Kc + ((size_t)u * E.n_max + n_prev) * D);
    uint4* vd = reinterpret_cast<uint4*>(E.Vc + ((size_t)u * E.n_max + n_prev) * D);
    const size_t cnt = (size_t)n_add * LPR;
    for (size_t p = (size_t)blockIdx.x * blockDim.x + threadIdx.x; p < cnt; p += (size_t)gridDim.x * blockDim.x) {
        kd[p] = ks[p];
        vd[p] = vs[p];
        if (p % LPR == 0) E.tok[(size_t)u * E.n_max + n_prev + p / LPR] = E.pos[u] + (int)(p / LPR);
    }
}

template <typename T>
__global__ void exact_advance_kernel(ExactCache<T> E, int U, int n_uniform, const int* __restrict__ cu) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const int b = u / E.Hkv;
    const int add = cu ? cu[b + 1] - cu[b] : n_uniform;
    E.n_unit[u] += add;
    E.pos[u] += add;
}

// grid (splits, U): append (k, v) as row n, then softmax(K q)^T V over rows 0..n. The new row is
// scored from the inputs, so no block reads a row another block writes in the same launch.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kQueryThreads) exact_step_kernel(ExactCache<T> E, const T* __restrict__ q,
                                                                   const T* __restrict__ k_new,
                                                                   const T* __restrict__ v_new, T* __restrict__ out) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR, STR = D + 2, UN = 2;
    __shared__ float sm[(kQueryThreads / 32) * G * STR];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, lr = lane % LPR, sub = lane / LPR;
    const int b = u / E.Hkv, kvh = u % E.Hkv;
    const int n = E.n_unit[u];
    const size_t qrow0 = (size_t)b * E.H + (size_t)kvh * G;
    const T* Ku = E.Kc + (size_t)u * E.n_max * D;
    const T* Vu = E.Vc + (size_t)u * E.n_max * D;
    const T* kn = k_new + (size_t)u * D;
    const T* vn = v_new + (size_t)u * D;
    if (blockIdx.x == 0 && n < E.n_max) {
        if (tid < LPR) reinterpret_cast<uint4*>(E.Kc + ((size_t)u * E.n_max + n) * D)[tid] = reinterpret_cast<const uint4*>(kn)[tid];
        else if (tid < 2 * LPR)
            reinterpret_cast<uint4*>(E.Vc + ((size_t)u * E.n_max + n) * D)[tid - LPR] = reinterpret_cast<const uint4*>(vn)[tid - LPR];
        if (tid == 0) E.tok[(size_t)u * E.n_max + n] = E.pos[u];
    }
    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint4 r = *reinterpret_cast<const uint4*>(q + (qrow0 + g) * D + lr * EPL);
        Elem<T>::unpack(r, qf[g]);
    }
    Acc<G, EPL> A;
    A.init();
    const int gg = (blockIdx.x * (kQueryThreads / 32) + warp) * RPW + sub;
    const int GG = splits * (kQueryThreads / 32) * RPW;
    for (int jb = 0; jb <= n; jb += GG * UN) {
        uint4 kraw[UN], vraw[UN];
        bool valid[UN];
        float wt_tau[UN], wt_z[UN];
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            const int idx = jb + i * GG + gg;
            valid[i] = idx <= n;
            wt_tau[i] = 1.f; wt_z[i] = 1.f;
            kraw[i] = make_uint4(0, 0, 0, 0);
            vraw[i] = kraw[i];
            if (valid[i]) {
                const T* kp = idx == n ? kn : Ku + (size_t)idx * D;
                const T* vp = idx == n ? vn : Vu + (size_t)idx * D;
                kraw[i] = *reinterpret_cast<const uint4*>(kp + lr * EPL);
                vraw[i] = *reinterpret_cast<const uint4*>(vp + lr * EPL);
            }
        }
        float sc[UN][G];
        scores<T, D, G, UN>(kraw, qf, sc);
        fold<T, D, G, UN, true>(A, sc, valid, wt_tau, wt_z, vraw);
    }
    float* part_u = E.part + (size_t)u * splits * G * STR;
    block_partial<T, D, G>(A, sm, part_u + (size_t)blockIdx.x * G * STR);
    __threadfence();
    __syncthreads();
    if (splits > 1) {
        if (tid == 0) {
            __threadfence();
            sm_last = (atomicAdd(&E.ticket[u], 1u) == (unsigned)splits - 1u);
        }
        __syncthreads();
        if (!sm_last) return;
        __threadfence();
    }
    final_merge<T, D, G>(part_u, splits, out + qrow0 * D, false);
    if (tid == 0) {
        E.n_unit[u] = n + 1;
        E.pos[u] = E.pos[u] + 1;
        E.ticket[u] = 0;
    }
}

}  // namespace sgk
