// Device-side building blocks of the SubGen kernels (sm_100a).
//
// Row geometry: every cached vector is one row of D elements (D*sizeof(T) = 128..512 bytes). A row is
// read by LPR = D/EPL consecutive lanes with one 16-byte load each (EPL = elements per 16 bytes), so a
// warp covers RPW = 32/LPR rows per load instruction ("row groups").
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sgk {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;
constexpr float kMaxAbsInput = 32768.0f;

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies, key bumped by the
// Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(kPhiloxM0, c.x), lo0 = kPhiloxM0 * c.x;
        const uint32_t hi1 = __umulhi(kPhiloxM1, c.z), lo1 = kPhiloxM1 * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += kPhiloxW0;
        k1 += kPhiloxW1;
    }
    return c;
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while
// its predecessor in the stream is still running; pdl_wait() returns once that predecessor has completed and
// its writes are visible (at once when the kernel was launched the ordinary way), pdl_trigger() lets the
// successor start being scheduled. Everything a kernel reads that an earlier kernel wrote comes after pdl_wait().
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

constexpr int kHeadDims = 32;   // coordinates of a representative kept in the packed head array

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int EPL = 4;
    static __device__ __forceinline__ void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ float to_out(float x) { return x; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int EPL = 8;
    // bf16 -> fp32 is a 16-bit shift of the pattern
    static __device__ __forceinline__ void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
        f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
        f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
        f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    static __device__ __forceinline__ __nv_bfloat16 to_out(float x) { return __float2bfloat16_rn(x); }
};

// Fixed-point terms: single binary32 operations, never contracted, truncated to integers.
__device__ __forceinline__ uint64_t fx_sqdiff(float a, float b) {
    const float df = __fsub_rn(a, b);
    return __float2ull_rz(__fmul_rn(__fmul_rn(df, df), 4294967296.0f));
}
__device__ __forceinline__ uint64_t fx_sq(float a) {
    return __float2ull_rz(__fmul_rn(__fmul_rn(a, a), 16777216.0f));
}

// Cluster coin: probability 1/n.
__device__ __forceinline__ bool coin_cluster(uint32_t u, uint32_t n) {
    return (uint64_t)u * (uint64_t)n < 4294967296ull;
}
// Value coin: u * tot < W * 2^32 in 128-bit integers, tot = mu_old + W.
__device__ __forceinline__ bool coin_value(uint32_t u, uint64_t tot, uint64_t W) {
    const uint64_t lhs_lo = (uint64_t)u * tot, lhs_hi = __umul64hi((uint64_t)u, tot);
    const uint64_t rhs_lo = W << 32, rhs_hi = W >> 32;
    return lhs_hi < rhs_hi || (lhs_hi == rhs_hi && lhs_lo < rhs_lo);
}

struct Best {          // (D2, index) ordered lexicographically: nearest, then lowest index
    unsigned long long d2;
    int idx;
    int pad;
};
__device__ __forceinline__ bool better(unsigned long long d2, int idx, const Best& b) {
    return d2 < b.d2 || (d2 == b.d2 && idx < b.idx);
}

// Pointers into the per-unit cache arrays (all device memory). Unit u = seq * Hkv + kvhead.
template <typename T> struct Cache {
    int B, H, Hkv, G, t, s, w, m_max;
    unsigned long long delta2_fx;
    uint32_t key0, key1;
    T* X;            // [U, m_max, D]     representatives x_i
    T* S;            // [U, m_max, t, D]  cluster samples S_i (materialised once n_i >= 2)
    float* xn;       // [U, m_max]        ||x_i||^2 in fp32, used only to pre-filter distance candidates
    T* Xh;           // [U, m_max, kHeadDims]  the first kHeadDims coordinates of x_i, packed: the step's insertion
                     //                   reads these instead of the full rows to rule out far representatives
    float* xhn;      // [U, m_max]        squared norm of that head in fp32
    int* cnt;        // [U, m_max]        n_i
    int* ctok;       // [U, m_max]        token index of x_i
    int* stok;       // [U, m_max, t]     token index in S_i(j)
    unsigned char* alias;   // [U, m_max, t]  the cluster's distinct sampled tokens. The t reservoirs sample with
                     //                   replacement, so slots often repeat a token; entry k < ndist[c] names the
                     //                   first slot holding the k-th distinct token and how many slots hold it:
                     //                   slot | (copies - 1) << 4 for t <= 16, else the slot itself (no merging).
                     //                   The query reads each distinct row once, weighted by its copies.
    unsigned char* ndist;   // [U, m_max]     number of valid entries in the alias row (clusters with n_i > 1)
    T* Mk;           // [U, s, D]
    T* Mv;           // [U, s, D]
    unsigned long long* MW;    // [U, s]  W of the sampled token, 0 = null
    int* Mtok;       // [U, s]
    float* MinvW;    // [U, s]            1/W in fp32 (0 = null), the query's estimator weight is mu/s times this
    T* ringK;        // [U, w, D]         token j in row j % w
    T* ringV;
    int* n_unit;     // [U] tokens seen
    int* m_unit;     // [U] clusters
    unsigned long long* mu;    // [U]
    int* status;     // [U]
    int* last_cid;   // [U]
    int* last_open;  // [U]
    unsigned long long* last_d2;   // [U]
    // scratch of the step kernels
    Best* part1;     // [U, splits]
    float* part2;    // [U, splits, G, D + 2]
    unsigned* ticket1;   // [U]
    unsigned* ticket2;   // [U]
    float* part_tau;     // [U, splits, G, 2] cluster partials {max, tau} of the query
    unsigned* qnext;     // [U] next work item of the cluster scan's per-unit queue
    unsigned* qnext2;    // [U] same for the scan of M and the window
    unsigned long long* pairs;   // [U] (key, representative) pairs scored by the chunked prefill so far
    int* epoch;                  // [U] tokens seen, as released by the step's insertion kernel (see acquire_unit)
    Best* next_best;             // [U] nearest representative found ahead of the next step (insert_mma_kernel, MODE 1)
    int* m_hist;                 // [2][U] one-kernel step: cluster count left by the step before the previous one (see step_fused_kernel)
    const int* order;            // [U] or NULL: the unit that the blocks with blockIdx.y = i serve, units with many
                                 //     clusters first (handles whose per-unit grids need several waves of blocks)
    int uid_stride, uid_off;     // numbering of the units in the Philox counter, see unit_id()
    // bounded-m variant: m_max is a budget, the threshold doubles and clusters merge when it is exhausted
    int bounded;
    unsigned long long* thr2;    // [U] threshold in force (fixed point), starts as delta2_fx
    int* level;                  // [U] doublings so far
};

// The unit index that keys the Philox draws of unit u = seq * Hkv + kvhead of this handle. A handle that serves a
// shard of a larger job (some of its KV heads, or some of its sequences) numbers its units as the whole job would,
// seq * uid_stride + uid_off + kvhead, so that sharding does not change a single draw.
template <typename T>
__device__ __forceinline__ uint32_t unit_id(const Cache<T>& C, int u) {
    return (uint32_t)((u / C.Hkv) * C.uid_stride + C.uid_off + (u % C.Hkv));
}

// The squared threshold a key of unit u is tested against. BND: the handle runs the bounded-m variant; it is a
// template parameter of the insertion kernels so that the plain path carries none of the variant's code.
template <bool BND, typename T>
__device__ __forceinline__ unsigned long long threshold2(const Cache<T>& C, int u) {
    return BND ? C.thr2[u] : C.delta2_fx;
}

// ---------------------------------------------------------------------------------------------
// Nearest representative: scan rows [c0, c1) of X_u with `ngroups` row groups, every group keeps its
// best (D2, idx). kf = this lane's EPL elements of the key. All lanes of a warp must call together.
template <typename T, int D>
__device__ __forceinline__ void scan_centres(const T* Xu, int c0, int c1, const float* kf,
                                             int group, int ngroups, int lr, Best& best) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL;
    constexpr int UN = 4;
    for (int base = c0; base < c1; base += ngroups * UN) {
        uint4 raw[UN];
        int row[UN];
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            row[i] = base + i * ngroups + group;
            raw[i] = make_uint4(0, 0, 0, 0);
            if (row[i] < c1) raw[i] = *reinterpret_cast<const uint4*>(Xu + (size_t)row[i] * D + lr * EPL);
        }
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            float xf[EPL];
            Elem<T>::unpack(raw[i], xf);
            unsigned long long acc = 0;
#pragma unroll
            for (int j = 0; j < EPL; ++j) acc += fx_sqdiff(xf[j], kf[j]);
#pragma unroll
            for (int off = 1; off < LPR; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (row[i] < c1 && better(acc, row[i], best)) { best.d2 = acc; best.idx = row[i]; }
        }
    }
}

// Block-wide lexicographic minimum. sm: shared array of at least 32 Best. Result valid in all threads.
__device__ __forceinline__ Best block_best(Best b, Best* sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long od = __shfl_xor_sync(0xffffffffu, b.d2, off);
        const int oi = __shfl_xor_sync(0xffffffffu, b.idx, off);
        if (better(od, oi, b)) { b.d2 = od; b.idx = oi; }
    }
    __syncthreads();
    if (lane == 0) sm[warp] = b;
    __syncthreads();
    Best r = sm[0];
    for (int i = 1; i < nw; ++i) if (better(sm[i].d2, sm[i].idx, r)) r = sm[i];
    return r;
}

// The distinct tokens among t slot tokens st[0..t), in slot order, in the encoding of Cache::alias. One thread.
__device__ __forceinline__ int distinct_slots(const int* st, int t, unsigned char* al) {
    if (t > 16) {
        for (int j = 0; j < t; ++j) al[j] = (unsigned char)j;
        return t;
    }
    int k = 0;
    for (int j = 0; j < t; ++j) {
        const int tok = st[j];
        int hit = -1;
        for (int i = 0; i < k; ++i) if (st[al[i] & 15] == tok) hit = i;
        if (hit >= 0) al[hit] = (unsigned char)(al[hit] + 16);
        else al[k++] = (unsigned char)j;
    }
    return k;
}

// Rebuild the alias row of cluster c of unit u from its slot tokens. Called by a whole block after the writes to
// stok are visible (a __syncthreads() since them); the first warp does the work, one slot per lane.
template <typename T>
__device__ __forceinline__ void rebuild_alias(const Cache<T>& C, int u, int c) {
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x, t = C.t;
    const size_t cc = (size_t)u * C.m_max + c;
    const int* st = C.stok + cc * t;
    unsigned char* al = C.alias + cc * t;
    if (t > 16) {                                   // no merging: every slot stands for itself
        for (int j = lane; j < t; j += 32) al[j] = (unsigned char)j;
        if (lane == 0) C.ndist[cc] = (unsigned char)t;
        return;
    }
    const int tok = lane < t ? st[lane] : -2 - lane;          // lanes beyond t hold tokens nobody shares
    bool first = lane < t;
    int copies = 0;
    for (int i = 0; i < t; ++i) {
        const int other = __shfl_sync(0xffffffffu, tok, i);
        if (other == tok) { copies += 1; if (i < lane) first = false; }
    }
    const unsigned firsts = __ballot_sync(0xffffffffu, first);
    if (first) al[__popc(firsts & ((1u << lane) - 1u))] = (unsigned char)(lane | ((copies - 1) << 4));
    if (lane == 0) C.ndist[cc] = (unsigned char)__popc(firsts);
}

// ---------------------------------------------------------------------------------------------
// Bounded-m variant: token e has no representative within the threshold and all m_max clusters are in use.
// The paper fixes no rule for this; the one taken here follows the doubling idea of the incremental clustering
// it cites: double the threshold (thr2 <- max(4 thr2, 1), capped at 2^62), sweep the clusters in index order,
// keep cluster i if no kept representative lies within the new threshold of x_i, otherwise merge it into the
// nearest kept one (ties: lowest kept index); kept clusters move to the front in order. Merging i (n_i members)
// into j (n_j): count n_j + n_i, and slot q of j takes slot q of i with probability n_i / (n_j + n_i), coin
//   u * (n_j + n_i) < n_i * 2^32,  u = word q % 4 of Philox(counter = (e, unit, q / 4 + 256 * i, 2 + 4 * level)),
// which keeps every slot uniform over the union (property 5 of Lemma 2). Then e is placed against the kept
// representatives; if it still must open a cluster and there is still no room, the threshold doubles again.
// Executed by a whole block; on return best and m describe the placement of e under the new threshold.
template <typename T, int D>
__device__ void make_room(const Cache<T>& C, int u, int e, const uint4* krow, Best& best, int& m) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR;
    __shared__ Best smb[32];
    __shared__ uint4 xrow[LPR];
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, lr = lane % LPR, sub = lane / LPR;
    const int group = warp * RPW + sub, ngroups = (nt >> 5) * RPW, t = C.t;
    T* Xu = C.X + (size_t)u * C.m_max * D;
    T* Su = C.S + (size_t)u * C.m_max * t * D;
    int* cntu = C.cnt + (size_t)u * C.m_max;
    int* ctoku = C.ctok + (size_t)u * C.m_max;
    int* stoku = C.stok + (size_t)u * C.m_max * t;
    float* xnu = C.xn + (size_t)u * C.m_max;
    unsigned long long thr = C.thr2[u];
    int level = C.level[u];
    for (int round = 0; round < 40; ++round) {
        ++level;
        thr = thr >= (1ull << 60) ? (1ull << 62) : (thr ? 4ull * thr : 1ull);
        int kept = 0;
        for (int i = 0; i < m; ++i) {
            __syncthreads();                       // rows and counts written for cluster i-1 are visible
            if (tid < LPR) xrow[tid] = reinterpret_cast<const uint4*>(Xu + (size_t)i * D)[tid];
            __syncthreads();
            float xf[EPL];
            Elem<T>::unpack(xrow[lr], xf);
            Best b;
            b.d2 = ~0ull; b.idx = INT_MAX; b.pad = 0;
            scan_centres<T, D>(Xu, 0, kept, xf, group, ngroups, lr, b);
            b = block_best(b, smb);
            const int n_i = cntu[i];
            if (kept > 0 && b.d2 <= thr) {
                const int j = b.idx, n_j = cntu[j];
                const unsigned long long n_new = (unsigned long long)n_i + (unsigned long long)n_j;
                for (int p = tid; p < t * LPR; p += nt) {
                    const int q = p / LPR, part = p % LPR;
                    const uint4 r = philox4x32_10(make_uint4((uint32_t)e, unit_id(C, u), (uint32_t)(q >> 2) + 256u * (uint32_t)i,
                                                             2u + 4u * (uint32_t)level), C.key0, C.key1);
                    const uint32_t word = (q & 3) == 0 ? r.x : (q & 3) == 1 ? r.y : (q & 3) == 2 ? r.z : r.w;
                    uint4* dst = reinterpret_cast<uint4*>(Su + ((size_t)j * t + q) * D) + part;
                    if ((unsigned long long)word * n_new < ((unsigned long long)n_i << 32)) {
                        *dst = n_i == 1 ? xrow[part] : reinterpret_cast<const uint4*>(Su + ((size_t)i * t + q) * D)[part];
                        if (part == 0) stoku[(size_t)j * t + q] = stoku[(size_t)i * t + q];
                    } else if (n_j == 1) {
                        *dst = reinterpret_cast<const uint4*>(Xu + (size_t)j * D)[part];   // write out the implied copy
                    }
                }
                __syncthreads();                   // n_j was read by everyone before it changes
                if (tid == 0) cntu[j] = (int)n_new;
                rebuild_alias(C, u, j);
            } else {
                if (kept != i) {
                    if (tid < LPR) reinterpret_cast<uint4*>(Xu + (size_t)kept * D)[tid] = xrow[tid];
                    if (tid < kHeadDims / EPL) reinterpret_cast<uint4*>(C.Xh + ((size_t)u * C.m_max + kept) * kHeadDims)[tid] = xrow[tid];
                    if (n_i >= 2)
                        for (int p = tid; p < t * LPR; p += nt)
                            reinterpret_cast<uint4*>(Su + (size_t)kept * t * D)[p] = reinterpret_cast<const uint4*>(Su + (size_t)i * t * D)[p];
                    for (int q = tid; q < t; q += nt) {
                        stoku[(size_t)kept * t + q] = stoku[(size_t)i * t + q];
                        C.alias[((size_t)u * C.m_max + kept) * t + q] = C.alias[((size_t)u * C.m_max + i) * t + q];
                    }
                    if (tid == 0) C.ndist[(size_t)u * C.m_max + kept] = C.ndist[(size_t)u * C.m_max + i];
                    if (tid == 0) {
                        cntu[kept] = n_i; ctoku[kept] = ctoku[i]; xnu[kept] = xnu[i];
                        C.xhn[(size_t)u * C.m_max + kept] = C.xhn[(size_t)u * C.m_max + i];
                    }
                }
                ++kept;
            }
        }
        __syncthreads();
        m = kept;
        float kf[EPL];
        Elem<T>::unpack(krow[lr], kf);
        Best b;
        b.d2 = ~0ull; b.idx = INT_MAX; b.pad = 0;
        scan_centres<T, D>(Xu, 0, m, kf, group, ngroups, lr, b);
        best = block_best(b, smb);
        if ((m > 0 && best.d2 <= thr) || m < C.m_max) break;
    }
    if (tid == 0) { C.thr2[u] = thr; C.level[u] = level; }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Insertion of token e (key/value rows already in shared memory) into D and M of unit u, in three parts that the
// step's insertion kernel runs one after the other in one block (apply_insert) and that the fused step kernel
// spreads over its blocks.

// W(v_e), ||k_e||^2 (whole row and packed head, fp32) and the input range check. Called by ONE warp; leaves
// sm_w[0] = W and sm_w[1] = {||k||^2, ||k head||^2} in shared memory (visible to the block after a barrier).
// token_weights_rows reports a failed range check through bad_out (written by lane 0); token_weights sets the unit's
// status bit 2 itself.
template <typename T, int D>
__device__ __forceinline__ void token_weights_rows(const uint4* krow, const uint4* vrow, unsigned long long* sm_w, int* bad_out) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL;
    const int lane = threadIdx.x & 31;
    unsigned long long acc = 0;
    float kk = 0.f, kh = 0.f;
    bool bad = false;
    for (int p = lane; p < LPR; p += 32) {
        float vf[EPL], kf[EPL];
        Elem<T>::unpack(vrow[p], vf);
        Elem<T>::unpack(krow[p], kf);
        float part = 0.f;
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
            acc += fx_sq(vf[j]);
            part = fmaf(kf[j], kf[j], part);
            bad |= !(fabsf(vf[j]) <= kMaxAbsInput) || !(fabsf(kf[j]) <= kMaxAbsInput);
        }
        kk += part;
        if (p < kHeadDims / EPL) kh += part;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc += __shfl_xor_sync(0xffffffffu, acc, off);
        kk += __shfl_xor_sync(0xffffffffu, kk, off);
        kh += __shfl_xor_sync(0xffffffffu, kh, off);
    }
    bad = __any_sync(0xffffffffu, bad);
    if (lane == 0) {
        sm_w[0] = acc;
        sm_w[1] = (unsigned long long)__float_as_uint(kk) | ((unsigned long long)__float_as_uint(kh) << 32);
        *bad_out = bad ? 1 : 0;
    }
}
template <typename T, int D>
__device__ __forceinline__ void token_weights(const Cache<T>& C, int u, const uint4* krow, const uint4* vrow,
                                              unsigned long long* sm_w) {
    int bad = 0;                                       // lane 0's copy is the one that is written
    token_weights_rows<T, D>(krow, vrow, sm_w, &bad);
    if ((threadIdx.x & 31) == 0 && bad) atomicOr(&C.status[u], 2);
}

// UpdateSoftmaxNormalizer for token e given its nearest representative: join (count, t coins) or open
// (representative, count 1; the t copies are implied while n_i = 1 and written out when the second member
// arrives). Executed by a whole block after token_weights and a barrier. Returns the new m; join / full report
// what happened (full: the key needed a new cluster and none was free). On bounded handles best and m are
// replaced by the placement under the threshold in force after make_room.
template <typename T, int D, bool BND = false>
__device__ int apply_cluster(const Cache<T>& C, int u, int e, Best& best, int& m, const uint4* krow,
                             const unsigned long long* sm_w, bool& join, bool& full) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int t = C.t;
    if constexpr (BND) {
        if (!((m > 0) && (best.d2 <= C.thr2[u])) && m >= C.m_max) make_room<T, D>(C, u, e, krow, best, m);
    }
    join = (m > 0) && (best.d2 <= threshold2<BND>(C, u));
    full = !join && (m >= C.m_max);
    T* Xu = C.X + (size_t)u * C.m_max * D;
    T* Su = C.S + (size_t)u * C.m_max * t * D;
    int* cntu = C.cnt + (size_t)u * C.m_max;
    int* stoku = C.stok + (size_t)u * C.m_max * t;
    int m_new = m;
    if (join) {
        const int c = best.idx;
        const int n_old = cntu[c];
        const uint32_t n_new = (uint32_t)n_old + 1u;
        // slot j is written by LPR threads, one 16-byte piece each
        for (int p = tid; p < t * LPR; p += nt) {
            const int j = p / LPR, part = p % LPR;
            const uint4 r = philox4x32_10(make_uint4((uint32_t)e, unit_id(C, u), (uint32_t)(j >> 2), 0u), C.key0, C.key1);
            const uint32_t word = (j & 3) == 0 ? r.x : (j & 3) == 1 ? r.y : (j & 3) == 2 ? r.z : r.w;
            uint4* dst = reinterpret_cast<uint4*>(Su + ((size_t)c * t + j) * D) + part;
            if (coin_cluster(word, n_new)) {
                *dst = krow[part];
                if (part == 0) stoku[(size_t)c * t + j] = e;
            } else if (n_old == 1) {
                *dst = reinterpret_cast<const uint4*>(Xu + (size_t)c * D)[part];   // write out the implied copy
            }
        }
        __syncthreads();            // n_old was read by everyone before it changes
        if (tid == 0) cntu[c] = (int)n_new;
        rebuild_alias(C, u, c);
    } else if (!full) {
        const int c = m;
        if (tid < LPR) reinterpret_cast<uint4*>(Xu + (size_t)c * D)[tid] = krow[tid];
        if (tid < kHeadDims / EPL) reinterpret_cast<uint4*>(C.Xh + ((size_t)u * C.m_max + c) * kHeadDims)[tid] = krow[tid];
        for (int j = tid; j < t; j += nt) stoku[(size_t)c * t + j] = e;
        if (tid == 0) {
            cntu[c] = 1;
            C.ctok[(size_t)u * C.m_max + c] = e;
            C.xn[(size_t)u * C.m_max + c] = __uint_as_float((unsigned)sm_w[1]);
            C.xhn[(size_t)u * C.m_max + c] = __uint_as_float((unsigned)(sm_w[1] >> 32));
        }
        m_new = m + 1;
    } else if (tid == 0) {
        atomicOr(&C.status[u], 1);
    }
    return m_new;
}

// M slot i takes (k_e, v_e) with weight W. One thread.
template <typename T, int D>
__device__ __forceinline__ void store_value_sample(const Cache<T>& C, int u, int i, int e, unsigned long long W,
                                                   const uint4* krow, const uint4* vrow) {
    constexpr int LPR = D / Elem<T>::EPL;
    uint4* dk = reinterpret_cast<uint4*>(C.Mk + ((size_t)u * C.s + i) * D);
    uint4* dv = reinterpret_cast<uint4*>(C.Mv + ((size_t)u * C.s + i) * D);
    for (int p = 0; p < LPR; ++p) { dk[p] = krow[p]; dv[p] = vrow[p]; }
    C.MW[(size_t)u * C.s + i] = W;
    C.MinvW[(size_t)u * C.s + i] = 1.f / (float)W;
    C.Mtok[(size_t)u * C.s + i] = e;
}

// Insert token e into D and M of unit u, given the nearest representative. Executed by a whole block; ends with
// a __syncthreads(). Returns the new m.
//   UpdateSoftmaxNormalizer: apply_cluster;
//   UpdateMatrixProduct: s coins with the OLD mu; then mu += W.
template <typename T, int D, bool BND = false>
__device__ int apply_insert(const Cache<T>& C, int u, int e, Best best, int m, const uint4* krow, const uint4* vrow,
                            unsigned long long* sm_w /* shared, 2 elements */) {
    const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5;
    const int s = C.s;
    if (warp == 0) token_weights<T, D>(C, u, krow, vrow, sm_w);
    __syncthreads();
    const unsigned long long W = sm_w[0];
    const unsigned long long mu_old = C.mu[u];
    bool join, full;
    const int m_new = apply_cluster<T, D, BND>(C, u, e, best, m, krow, sm_w, join, full);

    // UpdateMatrixProduct: slot i flips its own coin; winners copy (k_e, v_e)
    if (W > 0) {
        const unsigned long long tot = mu_old + W;
        for (int blk = tid; blk * 4 < s; blk += nt) {
            const uint4 r = philox4x32_10(make_uint4((uint32_t)e, unit_id(C, u), (uint32_t)blk, 1u), C.key0, C.key1);
            const uint32_t words[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = blk * 4 + q;
                if (i < s && coin_value(words[q], tot, W)) store_value_sample<T, D>(C, u, i, e, W, krow, vrow);
            }
        }
    }
    __syncthreads();                // every thread has read mu_old
    if (tid == 0) {
        C.mu[u] = mu_old + W;
        C.m_unit[u] = m_new;
        C.last_cid[u] = join ? best.idx : (full ? -1 : m);
        C.last_open[u] = join ? 0 : 1;
        C.last_d2[u] = best.d2;
    }
    __syncthreads();
    return m_new;
}

// ---------------------------------------------------------------------------------------------
// Online-softmax accumulators of one row group for G query heads. The d components of z are spread
// over the group's LPR lanes, EPL each; mx and tau are replicated in the group's lanes.
template <int G, int EPL> struct Acc {
    float mx[G], tau[G], z[G][EPL];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            mx[g] = -INFINITY; tau[g] = 0.f;
#pragma unroll
            for (int j = 0; j < EPL; ++j) z[g][j] = 0.f;
        }
    }
};

// Scores of UN rows for G heads: dot products reduced over the LPR lanes of the row group.
template <typename T, int D, int G, int UN>
__device__ __forceinline__ void scores(const uint4 (&kraw)[UN], const float (&qf)[G][Elem<T>::EPL], float (&sc)[UN][G]) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL;
#pragma unroll
    for (int i = 0; i < UN; ++i) {
        float kf[EPL];
        Elem<T>::unpack(kraw[i], kf);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float a = 0.f;
#pragma unroll
            for (int j = 0; j < EPL; ++j) a = fmaf(qf[g][j], kf[j], a);
            sc[i][g] = a;
        }
    }
#pragma unroll
    for (int off = 1; off < LPR; off <<= 1)
#pragma unroll
        for (int i = 0; i < UN; ++i)
#pragma unroll
            for (int g = 0; g < G; ++g) sc[i][g] += __shfl_xor_sync(0xffffffffu, sc[i][g], off);
}

// Fold UN scored rows into the accumulators. wt_tau / wt_z: the estimator weights of each row
// (n'/t and 0 for a cluster sample; 0 and mu/(s W) for a value sample; 1 and 1 for a window token).
template <typename T, int D, int G, int UN, bool HASV>
__device__ __forceinline__ void fold(Acc<G, Elem<T>::EPL>& A, const float (&sc)[UN][G], const bool (&valid)[UN],
                                     const float (&wt_tau)[UN], const float (&wt_z)[UN], const uint4 (&vraw)[UN]) {
    constexpr int EPL = Elem<T>::EPL;
    bool any = false;
#pragma unroll
    for (int i = 0; i < UN; ++i) any |= valid[i];
    if (!any) return;
    float p[UN][G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float mnew = A.mx[g];
#pragma unroll
        for (int i = 0; i < UN; ++i) if (valid[i]) mnew = fmaxf(mnew, sc[i][g]);
        const float scale = __expf(A.mx[g] - mnew);     // exp(-inf) = 0 on the first rows
        A.mx[g] = mnew;
        float tau = A.tau[g] * scale;
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            p[i][g] = valid[i] ? __expf(sc[i][g] - mnew) : 0.f;
            tau = fmaf(wt_tau[i], p[i][g], tau);
        }
        A.tau[g] = tau;
#pragma unroll
        for (int j = 0; j < EPL; ++j) A.z[g][j] *= scale;
    }
    if (HASV) {
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            float vf[EPL];
            Elem<T>::unpack(vraw[i], vf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float c = wt_z[i] * p[i][g];
#pragma unroll
                for (int j = 0; j < EPL; ++j) A.z[g][j] = fmaf(c, vf[j], A.z[g][j]);
            }
        }
    }
}

// Merge two accumulator states (mx, tau) -> first; sa, sb are the factors for the two z vectors.
__device__ __forceinline__ void merge_scalar(float& mx, float& tau, float omx, float otau, float& sa, float& sb) {
    const float m = fmaxf(mx, omx);
    sa = (mx == -INFINITY) ? 0.f : __expf(mx - m);
    sb = (omx == -INFINITY) ? 0.f : __expf(omx - m);
    tau = tau * sa + otau * sb;
    mx = m;
}

// Combine the per-warp partials [warp][G][D+2] = {mx, tau, z[D]} in shared memory into the block's
// partial at dst (global). Starts with a __syncthreads().
template <int D, int G>
__device__ __forceinline__ void block_combine(const float* sm, float* dst) {
    constexpr int STR = D + 2;
    const int tid = threadIdx.x, nw = blockDim.x >> 5;
    __syncthreads();
    for (int o = tid; o < G * STR; o += blockDim.x) {
        const int g = o / STR, c = o % STR;
        float m = -INFINITY;
        for (int w = 0; w < nw; ++w) m = fmaxf(m, sm[((size_t)w * G + g) * STR]);
        float r;
        if (c == 0) r = m;
        else {
            r = 0.f;
            for (int w = 0; w < nw; ++w) {
                const float wm = sm[((size_t)w * G + g) * STR];
                if (wm != -INFINITY) r += sm[((size_t)w * G + g) * STR + c] * __expf(wm - m);
            }
        }
        dst[(size_t)g * STR + c] = r;
    }
}

// Block-level reduction of the row groups' accumulators and store of the block's partial
// [G][D+2] = {mx, tau, z[D]} to dst. sm: shared floats, at least (blockDim/32) * G * (D+2).
template <typename T, int D, int G>
__device__ __forceinline__ void block_partial(Acc<G, Elem<T>::EPL>& A, float* sm, float* dst) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, STR = D + 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, lr = lane % LPR;
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float omx = __shfl_xor_sync(0xffffffffu, A.mx[g], off);
            const float otau = __shfl_xor_sync(0xffffffffu, A.tau[g], off);
            float sa, sb;
            merge_scalar(A.mx[g], A.tau[g], omx, otau, sa, sb);
#pragma unroll
            for (int j = 0; j < EPL; ++j) {
                const float oz = __shfl_xor_sync(0xffffffffu, A.z[g][j], off);
                A.z[g][j] = A.z[g][j] * sa + oz * sb;
            }
        }
    }
    if (lane < LPR) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float* w = sm + ((size_t)warp * G + g) * STR;
            if (lr == 0) { w[0] = A.mx[g]; w[1] = A.tau[g]; }
#pragma unroll
            for (int j = 0; j < EPL; ++j) w[2 + lr * EPL + j] = A.z[g][j];
        }
    }
    block_combine<D, G>(sm, dst);
}

// Final merge of block partials and the division z / tau, by a whole block (all threads must call).
// part: [np][G][D+2] = {max, tau, z[D]}; part_t (may be NULL): [np_t][G][2] = {max, tau} partials that carry no
// numerator; out rows: out + g * D for g < G. poisoned -> NaN. sred: 16 floats of shared memory.
// The loads of different partials are independent (no branches, unrolled), so their latencies overlap.
template <typename T, int D, int G>
__device__ __forceinline__ void merge_partials(const float* part, int np, const float* part_t, int np_t, T* out,
                                               bool poisoned, float* sred) {
    constexpr int STR = D + 2;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int g = warp; g < G; g += nw) {            // per head: global maximum, then the partition function
        float m = -INFINITY;
        for (int i = lane; i < np; i += 32) m = fmaxf(m, __ldcg(part + ((size_t)i * G + g) * STR));
        for (int i = lane; i < np_t; i += 32) m = fmaxf(m, __ldcg(part_t + ((size_t)i * G + g) * 2));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        float tau = 0.f;
        for (int i = lane; i < np; i += 32) {
            const float* pp = part + ((size_t)i * G + g) * STR;
            const float pm = __ldcg(pp), pt = __ldcg(pp + 1);
            tau += pm == -INFINITY ? 0.f : pt * __expf(pm - m);
        }
        for (int i = lane; i < np_t; i += 32) {
            const float* pp = part_t + ((size_t)i * G + g) * 2;
            const float pm = __ldcg(pp), pt = __ldcg(pp + 1);
            tau += pm == -INFINITY ? 0.f : pt * __expf(pm - m);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tau += __shfl_xor_sync(0xffffffffu, tau, off);
        if (lane == 0) { sred[g] = m; sred[8 + g] = tau; }
    }
    __syncthreads();
    for (int o = threadIdx.x; o < G * D / 2; o += blockDim.x) {       // two neighbouring columns per thread
        const int g = (2 * o) / D, c = (2 * o) % D;
        const float m = sred[g], tau = sred[8 + g];
        float z0 = 0.f, z1 = 0.f;
#pragma unroll 16
        for (int i = 0; i < np; ++i) {
            const float* pp = part + ((size_t)i * G + g) * STR;
            const float pm = __ldcg(pp);
            const float2 pz = __ldcg(reinterpret_cast<const float2*>(pp + 2 + c));     // rows are 8-byte aligned
            const float sc = pm == -INFINITY ? 0.f : __expf(pm - m);
            z0 = fmaf(pz.x, sc, z0);
            z1 = fmaf(pz.y, sc, z1);
        }
        float r0 = tau > 0.f ? z0 / tau : 0.f, r1 = tau > 0.f ? z1 / tau : 0.f;
        if (poisoned) r0 = r1 = __int_as_float(0x7fc00000);
        out[(size_t)g * D + c] = Elem<T>::to_out(r0);
        out[(size_t)g * D + c + 1] = Elem<T>::to_out(r1);
    }
}

template <typename T, int D, int G>
__device__ __forceinline__ void final_merge(const float* part, int np, T* out, bool poisoned) {
    __shared__ float sred[16];
    merge_partials<T, D, G>(part, np, nullptr, 0, out, poisoned, sred);
}

}  // namespace sgk
