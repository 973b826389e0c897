// Query kernel for bf16 caches with the dot products on the tensor cores.
//
// The stream step is bound by HBM: every cached row is read once and used for one dot product with q
// (and one axpy into z). On CUDA cores the bf16->fp32 conversions, FMAs and lane reductions of those
// dot products cost more issue slots per byte than the memory system needs time to deliver it, so here
// both contractions run as warp-level m16n8k16 MMAs fed straight from 16-byte global loads:
//
//   scores S[16 rows][8 heads] = K_tile[16 x D] . q^T[D x 8]          (A = keys,   B = q)
//   z^T   [16 cols][8 heads]  += V_tile^T[16 cols x 16 rows] . P[16 rows x 8 heads]   (A = values^T, B = P)
//
// The G <= 8 query heads of a KV head sit in the N dimension, so grouped-query attention costs no extra
// instructions. A dot product does not depend on the order of its terms, which lets every lane take the
// 8 consecutive elements of one 16-byte load as its k-slices (q is loaded with the same pattern); the
// value tile needs rows paired inside a register, done with two byte permutes per register pair.
// P (estimator weight times exp(score - max)) is rounded to bf16 for the second MMA; the partition
// function tau is accumulated from the unrounded fp32 values; accumulation is fp32 throughout.
//
// The query runs as two kernels so that each keeps only the registers it needs and many warps stay
// resident: query_tau_kernel scans the clusters (keys only, partition function), query_z_kernel scans the
// value samples M and the window (keys and values, numerator and the window's share of tau) and its last
// block merges everything into out = z / tau.
//
// Work of one unit is cut into items (16 clusters; 16 M slots; 16 window rows) handed out through a
// per-unit atomic counter, so warps of all blocks of the unit stay busy until the unit is done. Nothing
// spins: the counter only hands out indices.
#pragma once
#include "subgen_device.cuh"

namespace sgk {

constexpr int kQmThreads = 128;

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint4 ldg16(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }

// 16-byte load of a row that is read once per step: first in line for eviction from L2. A step
// streams hundreds of megabytes of sampled rows; loaded the ordinary way they push out of the L2 everything that
// IS read again in the next step or by the next kernel (counts, alias rows, packed heads, partials, the kernels'
// own instructions), which then comes from DRAM at the head of every dependent chain.
__device__ __forceinline__ uint4 ldg16_stream(const void* p) {
    uint64_t pol;
    asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    uint4 r;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p), "l"(pol));
    return r;
}

// Per-warp running state. Lane = 4*g + tq. The lane keeps the running maxima and partial partition
// sums of heads 2tq and 2tq+1, and z^T accumulators acc[cc*4+j] = {z[2tq][c], z[2tq+1][c], z[2tq][c+1],
// z[2tq+1][c+1]} with c = cc*64 + g*8 + 2j.
template <int D> struct MmaState {
    float m0, m1, tau0, tau1;
    float acc[D / 16][4];
};

// Scores of one 16-row tile against q, then the online-softmax update of the running maxima.
// ka / kb: this lane's pieces of key rows g and g+8 (load_keys; valid memory even when the row is masked).
// Returns p[4] = exp(score - max) for (row g, head 2tq), (g, 2tq+1), (g+8, 2tq), (g+8, 2tq+1); 0 if masked.
template <int D>
__device__ __forceinline__ void load_keys(const __nv_bfloat16* pa, const __nv_bfloat16* pb, int tq, uint4 (&ka)[D / 32],
                                          uint4 (&kb)[D / 32]) {
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        ka[c] = ldg16(pa + c * 32 + tq * 8);
        kb[c] = ldg16(pb + c * 32 + tq * 8);
    }
}
// the same for rows that are read once per step (see ldg16_stream)
template <int D>
__device__ __forceinline__ void load_keys_stream(const __nv_bfloat16* pa, const __nv_bfloat16* pb, int tq, uint4 (&ka)[D / 32],
                                                 uint4 (&kb)[D / 32]) {
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        ka[c] = ldg16_stream(pa + c * 32 + tq * 8);
        kb[c] = ldg16_stream(pb + c * 32 + tq * 8);
    }
}

template <int D, int DA>
__device__ __forceinline__ void tile_scores(MmaState<DA>& S, const uint4 (&ka)[D / 32], const uint4 (&kb)[D / 32], bool va,
                                            bool vb, const uint32_t (&qb)[D / 32][4], float (&p)[4]) {
    constexpr int NC = D / 32;
    float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        mma_bf16_16816(sc, ka[c].x, kb[c].x, ka[c].y, kb[c].y, qb[c][0], qb[c][1]);
        mma_bf16_16816(sc, ka[c].z, kb[c].z, ka[c].w, kb[c].w, qb[c][2], qb[c][3]);
    }
    const float s0 = va ? sc[0] : -INFINITY, s1 = va ? sc[1] : -INFINITY;
    const float s2 = vb ? sc[2] : -INFINITY, s3 = vb ? sc[3] : -INFINITY;
    float t0 = fmaxf(s0, s2), t1 = fmaxf(s1, s3);
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, off));
        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, off));
    }
    const float n0 = fmaxf(S.m0, t0), n1 = fmaxf(S.m1, t1);
    if (__any_sync(0xffffffffu, n0 != S.m0 || n1 != S.m1)) {
        const float f0 = (S.m0 == -INFINITY) ? 0.f : __expf(S.m0 - n0);
        const float f1 = (S.m1 == -INFINITY) ? 0.f : __expf(S.m1 - n1);
        S.tau0 *= f0;
        S.tau1 *= f1;
        if (DA == D) {                 // DA != D: caller keeps no numerator accumulators
#pragma unroll
            for (int j = 0; j < DA / 16; ++j) {
                S.acc[j][0] *= f0; S.acc[j][2] *= f0;
                S.acc[j][1] *= f1; S.acc[j][3] *= f1;
            }
        }
        S.m0 = n0;
        S.m1 = n1;
    }
    const float r0 = (n0 == -INFINITY) ? 0.f : n0, r1 = (n1 == -INFINITY) ? 0.f : n1;
    p[0] = __expf(s0 - r0);
    p[1] = __expf(s1 - r1);
    p[2] = __expf(s2 - r0);
    p[3] = __expf(s3 - r1);
}

// z^T += V_tile^T . P for one 16-row tile. pz[4]: weighted p in the layout tile_scores returns.
// v: this lane's pieces of value rows 2tq, 2tq+1, 2tq+8, 2tq+9 of the tile (load_values; finite contents).
template <int D>
__device__ __forceinline__ void load_values(const __nv_bfloat16* const (&pv)[4], int g, uint4 (&v)[4][D / 64]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) v[i][cc] = ldg16(pv[i] + cc * 64 + g * 8);
}
template <int D>
__device__ __forceinline__ void load_values_stream(const __nv_bfloat16* const (&pv)[4], int g, uint4 (&v)[4][D / 64]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) v[i][cc] = ldg16_stream(pv[i] + cc * 64 + g * 8);
}

template <int D>
__device__ __forceinline__ void tile_values(MmaState<D>& S, const float (&pz)[4], const uint4 (&v)[4][D / 64], int g, int tq) {
    constexpr int NV = D / 64;
    // B operand: P[rows 2tq, 2tq+1 | 2tq+8, 2tq+9][head g], gathered from the lanes that own those rows
    const uint32_t p01 = pack_bf16x2(pz[0], pz[1]), p23 = pack_bf16x2(pz[2], pz[3]);
    const int la = 8 * tq + (g >> 1), lb = la + 4;
    const uint32_t a01 = __shfl_sync(0xffffffffu, p01, la), b01 = __shfl_sync(0xffffffffu, p01, lb);
    const uint32_t a23 = __shfl_sync(0xffffffffu, p23, la), b23 = __shfl_sync(0xffffffffu, p23, lb);
    const uint32_t sel = (g & 1) ? 0x7632u : 0x5410u;
    const uint32_t B0 = __byte_perm(a01, b01, sel), B1 = __byte_perm(a23, b23, sel);
#pragma unroll
    for (int cc = 0; cc < NV; ++cc) {
        const uint32_t r0[4] = {v[0][cc].x, v[0][cc].y, v[0][cc].z, v[0][cc].w};
        const uint32_t r1[4] = {v[1][cc].x, v[1][cc].y, v[1][cc].z, v[1][cc].w};
        const uint32_t r2[4] = {v[2][cc].x, v[2][cc].y, v[2][cc].z, v[2][cc].w};
        const uint32_t r3[4] = {v[3][cc].x, v[3][cc].y, v[3][cc].z, v[3][cc].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            mma_bf16_16816(S.acc[cc * 4 + j], __byte_perm(r0[j], r1[j], 0x5410u), __byte_perm(r0[j], r1[j], 0x7632u),
                           __byte_perm(r2[j], r3[j], 0x5410u), __byte_perm(r2[j], r3[j], 0x7632u), B0, B1);
        }
    }
}

// What the insertion of a step wrote (M, the window row, mu) made visible to a block of the value scan, which does
// not wait for the whole stream (see query_z_kernel): the insertion kernel ends a unit's update with a release store
// of the unit's epoch, the value scan begins the unit with an acquire load of it. Called by a whole block; ends with
// a __syncthreads().
template <typename T>
__device__ __forceinline__ void acquire_unit(const Cache<T>& C, int u) {
    if (threadIdx.x == 0) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(C.epoch + u) : "memory");
        (void)v;
    }
    __syncthreads();
}
template <typename T>
__device__ __forceinline__ void release_unit(const Cache<T>& C, int u, int value) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(C.epoch + u), "r"(value) : "memory");
}

constexpr int kTauRows = 256 + 16;   // rows of one pass of the cluster scan: at most 256 sample rows and 16 singletons

// floor(r / t) for small r by one multiply-high (t = 1 handled by the caller's magic = 0)
__device__ __forceinline__ int div_small(int r, unsigned magic) { return magic ? (int)__umulhi((unsigned)r, magic) : r; }

// ---------------------------------------------------------------------------------------------
// The cluster part of the partition function for one warp, as a software pipeline over items of 16 clusters:
//   tau_D += sum over the item's clusters of n'/t sum over the t samples of exp<q,k>
// (a cluster with n' = 1 is read as its representative with weight 1; slots that hold the same token are read once
// and weighted by their number). While the rows of item i are scored, the counts and alias rows of item i+1 are
// already on their way and the ticket for item i+2 has been asked for, so the only memory round trip a warp waits
// for per item is that of the rows themselves. UN tiles of 16 rows are requested together.
//   first, second  the warp's first two items (known without a memory access)
//   counter, base  later items are base + atomicAdd(counter, 1)
//   als, rix, rwt  this warp's shared-memory scratch: 16 * 64 bytes, kTauRows ints, kTauRows floats
template <int D, int DA, int UN>
__device__ __forceinline__ void cluster_scan(MmaState<DA>& S, const uint32_t (&qb)[D / 32][4], const Cache<__nv_bfloat16>& C, int u,
                                             int m, int first, int second, unsigned* counter, int base, unsigned* als, int* rix,
                                             float* rwt) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32;
    const int lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
    const int t = C.t;
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const T* Su = C.S + (size_t)u * C.m_max * t * D;
    const int* cntu = C.cnt + (size_t)u * C.m_max;
    const unsigned char* ndu = C.ndist + (size_t)u * C.m_max;
    const unsigned char* alias_bytes = C.alias + (size_t)u * C.m_max * t;
    // alias rows of an item are 16 t contiguous bytes (the array is padded by one item); they travel through two
    // registers per lane when t <= 16 and the unit's rows start on a 4-byte boundary, else they are read in place
    const bool fast = t <= 16 && !(reinterpret_cast<uintptr_t>(alias_bytes) & 3);
    const unsigned* alias_words = reinterpret_cast<const unsigned*>(alias_bytes);
    const float inv_t = 1.f / (float)t;
    const int total = (m + 15) >> 4;
    const int gsz = t <= 16 ? 16 : 256 / t;          // clusters whose rows fit one list of kTauRows entries (t <= 64)
    const int nwords = 4 * t;                        // alias words per item (fast path: <= 64)
    int item = first, next = second;
    int cn = 0, nd = 0;
    unsigned aw0 = 0, aw1 = 0;
    auto fetch = [&](int it, int& cn_, int& nd_, unsigned& a0, unsigned& a1) {
        cn_ = 0; nd_ = 0; a0 = 0; a1 = 0;
        if (it < total) {
            const int c = it * 16 + lane;
            if (lane < 16 && c < m) { cn_ = cntu[c]; nd_ = (int)ndu[c]; }
            if (fast) {
                if (lane < nwords) a0 = alias_words[(size_t)it * nwords + lane];
                if (lane + 32 < nwords) a1 = alias_words[(size_t)it * nwords + lane + 32];
            }
        }
    };
    fetch(item, cn, nd, aw0, aw1);
    while (item < total) {
        int next2 = 0;
        if (lane == 0) next2 = base + (int)atomicAdd(counter, 1u);       // asked for now, needed two items later
        int cn_n, nd_n;
        unsigned aw0_n, aw1_n;
        fetch(next, cn_n, nd_n, aw0_n, aw1_n);
        const int c = item * 16 + lane;
        if (fast) {
            if (lane < nwords) als[lane] = aw0;
            if (lane + 32 < nwords) als[lane + 32] = aw1;
        } else {
            unsigned char* dst = reinterpret_cast<unsigned char*>(als);
            for (int i = lane; i < 16 * t; i += 32) dst[i] = alias_bytes[(size_t)item * 16 * t + i];
        }
        for (int p0 = 0; p0 < 16; p0 += gsz) {
            const bool act = lane >= p0 && lane < p0 + gsz;
            const int ndl = (act && cn > 1) ? nd : 0;
            int incl = ndl;
#pragma unroll
            for (int off = 1; off < 16; off <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += v;
            }
            const int rows_m = __shfl_sync(0xffffffffu, incl, 15);
            const unsigned ms = __ballot_sync(0xffffffffu, act && cn == 1);
            const int rows = rows_m + __popc(ms);
            __syncwarp();
            if (ndl) {
                const unsigned char* al = reinterpret_cast<const unsigned char*>(als) + lane * t;
                const float wc = (float)cn * inv_t;
                for (int k = 0; k < ndl; ++k) {
                    const int e = al[k];
                    const int slot = t <= 16 ? (e & 15) : e, copies = t <= 16 ? (e >> 4) + 1 : 1;
                    rix[incl - ndl + k] = c * t + slot;
                    rwt[incl - ndl + k] = wc * (float)copies;
                }
            }
            if (act && cn == 1) {
                const int r = rows_m + __popc(ms & ((1u << lane) - 1u));
                rix[r] = c | (int)0x80000000;
                rwt[r] = 1.f;
            }
            __syncwarp();
            // row r of the list -> pointer, weight, validity
            auto resolve = [&](int r, const T*& ptr, float& wgt) -> bool {
                ptr = Xu;
                wgt = 1.f;
                if (r < rows) {
                    const int ix = rix[r];
                    ptr = ix < 0 ? Xu + (size_t)(ix & 0x7fffffff) * D : Su + (size_t)ix * D;
                    wgt = rwt[r];
                }
                return r < rows;
            };
            for (int r0 = 0; r0 < rows; r0 += 16 * UN) {
                const T *pa[UN], *pb[UN];
                float wa[UN], wb[UN];
                bool va[UN], vb[UN];
                uint4 ka[UN][NC], kb[UN][NC];
#pragma unroll
                for (int i = 0; i < UN; ++i) {
                    va[i] = resolve(r0 + 16 * i + g, pa[i], wa[i]);
                    vb[i] = resolve(r0 + 16 * i + g + 8, pb[i], wb[i]);
                }
#pragma unroll
                for (int i = 0; i < UN; ++i)
                    if (i == 0 || r0 + 16 * i < rows) load_keys_stream<D>(pa[i], pb[i], tq, ka[i], kb[i]);
#pragma unroll
                for (int i = 0; i < UN; ++i) {
                    if (i == 0 || r0 + 16 * i < rows) {
                        float p[4];
                        tile_scores<D, DA>(S, ka[i], kb[i], va[i], vb[i], qb, p);
                        S.tau0 += wa[i] * p[0] + wb[i] * p[2];
                        S.tau1 += wa[i] * p[1] + wb[i] * p[3];
                    }
                }
            }
            __syncwarp();
        }
        item = next;
        next = __shfl_sync(0xffffffffu, next2, 0);
        cn = cn_n; nd = nd_n; aw0 = aw0_n; aw1 = aw1_n;
    }
}

// The cluster part of the partition function for one warp, items of 16 clusters taken from the unit's counter one
// at a time (the plain loop; cluster_scan above is the pipelined one). als, rix, rwt: this warp's shared-memory
// scratch as for cluster_scan.
template <int D>
__device__ __forceinline__ void cluster_scan_queue(MmaState<16>& S, const uint32_t (&qb)[D / 32][4], const Cache<__nv_bfloat16>& C,
                                                   int u, int m, unsigned* als, int* rix, float* rwt) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32;
    const int lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
    const int t = C.t;
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const T* Su = C.S + (size_t)u * C.m_max * t * D;
    const int* cntu = C.cnt + (size_t)u * C.m_max;
    const unsigned char* ndu = C.ndist + (size_t)u * C.m_max;
    const unsigned char* alias_bytes = C.alias + (size_t)u * C.m_max * t;
    const unsigned* alias_words = (reinterpret_cast<uintptr_t>(alias_bytes) & 3) ? nullptr : reinterpret_cast<const unsigned*>(alias_bytes);
    const float inv_t = 1.f / (float)t;
    const int total = (m + 15) >> 4;
    const int gsz = t <= 16 ? 16 : 256 / t;          // clusters whose rows fit one list of kTauRows entries (t <= 64)
    int item = 0;
    if (lane == 0) item = (int)atomicAdd(&C.qnext[u], 1u);
    item = __shfl_sync(0xffffffffu, item, 0);
    while (item < total) {
        int next = 0;
        if (lane == 0) next = (int)atomicAdd(&C.qnext[u], 1u);     // asked for early, needed late
        // 16 clusters -> one list of rows: first the distinct samples of every cluster with n' > 1, each weighted
        // n'/t times the number of slots that hold it, then the representatives of the singletons
        const int c = item * 16 + lane;
        const int cn = (lane < 16 && c < m) ? cntu[c] : 0;
        const int nd = (lane < 16 && c < m) ? (int)ndu[c] : 0;
        // the 16 alias rows are contiguous (16 t bytes; the array is padded by one item): word loads when the
        // unit's rows start on a 4-byte boundary (m_max t a multiple of 4, or unit 0), else byte by byte
        if (alias_words) {
            for (int i = lane; i < 4 * t; i += 32) als[i] = alias_words[(size_t)item * 4 * t + i];
        } else {
            unsigned char* dst = reinterpret_cast<unsigned char*>(als);
            for (int i = lane; i < 16 * t; i += 32) dst[i] = alias_bytes[(size_t)item * 16 * t + i];
        }
        for (int p0 = 0; p0 < 16; p0 += gsz) {
            const bool act = lane >= p0 && lane < p0 + gsz;
            const int ndl = (act && cn > 1) ? nd : 0;
            int incl = ndl;
#pragma unroll
            for (int off = 1; off < 16; off <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += v;
            }
            const int rows_m = __shfl_sync(0xffffffffu, incl, 15);
            const unsigned ms = __ballot_sync(0xffffffffu, act && cn == 1);
            const int rows = rows_m + __popc(ms);
            __syncwarp();
            if (ndl) {
                const unsigned char* al = reinterpret_cast<const unsigned char*>(als) + lane * t;
                const float wc = (float)cn * inv_t;
                for (int k = 0; k < ndl; ++k) {
                    const int e = al[k];
                    const int slot = t <= 16 ? (e & 15) : e, copies = t <= 16 ? (e >> 4) + 1 : 1;
                    rix[incl - ndl + k] = c * t + slot;
                    rwt[incl - ndl + k] = wc * (float)copies;
                }
            }
            if (act && cn == 1) {
                const int r = rows_m + __popc(ms & ((1u << lane) - 1u));
                rix[r] = c | (int)0x80000000;
                rwt[r] = 1.f;
            }
            __syncwarp();
            // row r of the list -> pointer, weight, validity
            auto resolve = [&](int r, const T*& ptr, float& wgt) -> bool {
                ptr = Xu;
                wgt = 1.f;
                if (r < rows) {
                    const int ix = rix[r];
                    ptr = ix < 0 ? Xu + (size_t)(ix & 0x7fffffff) * D : Su + (size_t)ix * D;
                    wgt = rwt[r];
                }
                return r < rows;
            };
            for (int r0 = 0; r0 < rows; r0 += 16) {
                const T *pa, *pb;
                float wa, wb;
                const bool va = resolve(r0 + g, pa, wa), vb = resolve(r0 + g + 8, pb, wb);
                uint4 ka[NC], kb[NC];
                load_keys_stream<D>(pa, pb, tq, ka, kb);
                float p[4];
                tile_scores<D, 16>(S, ka, kb, va, vb, qb, p);
                S.tau0 += wa * p[0] + wb * p[2];
                S.tau1 += wa * p[1] + wb * p[3];
            }
            __syncwarp();
        }
        item = __shfl_sync(0xffffffffu, next, 0);
    }
}

// ---------------------------------------------------------------------------------------------
// Clusters: tau_D = sum over clusters of n'/t sum over the t samples of exp<q,k>; a cluster with n' = 1
// is read as its representative with weight 1. Writes per block {max, tau} per head to part_tau.
template <int D, int G>
__global__ void __launch_bounds__(kQmThreads, 6) query_tau_kernel(Cache<__nv_bfloat16> C, const __nv_bfloat16* __restrict__ q) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, NW = kQmThreads / 32;
    __shared__ float sm[NW][G][2];
    __shared__ unsigned als[NW][16 * 64 / 4];          // alias rows of the item's 16 clusters, t <= 64 bytes each
    __shared__ int rix[NW][kTauRows];                  // row list of a pass: sample row index, or representative | 2^31
    __shared__ float rwt[NW][kTauRows];
    const int u = C.order ? C.order[blockIdx.y] : (int)blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, tq = lane & 3;
    const int b = u / C.Hkv, kvh = u % C.Hkv;
    const size_t qrow0 = (size_t)b * C.H + (size_t)kvh * G;

    uint32_t qb[NC][4];                   // the queries are an input of the call, not a predecessor's output
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        uint4 r = make_uint4(0, 0, 0, 0);
        if (g < G) r = ldg16(q + (qrow0 + g) * D + c * 32 + tq * 8);
        qb[c][0] = r.x; qb[c][1] = r.y; qb[c][2] = r.z; qb[c][3] = r.w;
    }
    pdl_wait();
    // The value scan may be scheduled from here on: it starts without waiting for this kernel, so the insertion (this
    // kernel's predecessor) must be complete before it is let go.
    pdl_trigger();
    const int m = C.m_unit[u];
    MmaState<16> S;                       // the accumulators stay untouched here and cost no registers
    S.m0 = S.m1 = -INFINITY;
    S.tau0 = S.tau1 = 0.f;
    S.acc[0][0] = S.acc[0][1] = S.acc[0][2] = S.acc[0][3] = 0.f;

    cluster_scan_queue<D>(S, qb, C, u, m, als[warp], rix[warp], rwt[warp]);
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        S.tau0 += __shfl_xor_sync(0xffffffffu, S.tau0, off);
        S.tau1 += __shfl_xor_sync(0xffffffffu, S.tau1, off);
    }
    if (g == 0) {
        if (2 * tq < G) { sm[warp][2 * tq][0] = S.m0; sm[warp][2 * tq][1] = S.tau0; }
        if (2 * tq + 1 < G) { sm[warp][2 * tq + 1][0] = S.m1; sm[warp][2 * tq + 1][1] = S.tau1; }
    }
    __syncthreads();
    if (tid < G) {
        float mx = -INFINITY, tau = 0.f;
        for (int wv = 0; wv < NW; ++wv) mx = fmaxf(mx, sm[wv][tid][0]);
        for (int wv = 0; wv < NW; ++wv)
            if (sm[wv][tid][0] != -INFINITY) tau += sm[wv][tid][1] * __expf(sm[wv][tid][0] - mx);
        float* dst = C.part_tau + (((size_t)u * splits + blockIdx.x) * G + tid) * 2;
        dst[0] = mx;
        dst[1] = tau;
    }
}

// ---------------------------------------------------------------------------------------------
// Value samples and window: z = sum_M mu/(s W) exp<q,k> v + sum_window exp<q,k> v, tau_window. The block
// that finishes last merges its siblings' partials with the cluster partials of query_tau_kernel, writes
// out = z / tau and advances the unit's token count.
template <int D, int G>
__global__ void __launch_bounds__(kQmThreads, 4) query_z_kernel(Cache<__nv_bfloat16> C, const __nv_bfloat16* __restrict__ q,
                                                                __nv_bfloat16* __restrict__ out, int splits_tau, int advance) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, STR = D + 2, NW = kQmThreads / 32;
    __shared__ float sm[NW * G * STR];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, tq = lane & 3;
    const int b = u / C.Hkv, kvh = u % C.Hkv;
    const size_t qrow0 = (size_t)b * C.H + (size_t)kvh * G;
    pdl_trigger();

    uint32_t qb[NC][4];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        uint4 r = make_uint4(0, 0, 0, 0);
        if (g < G) r = ldg16(q + (qrow0 + g) * D + c * 32 + tq * 8);
        qb[c][0] = r.x; qb[c][1] = r.y; qb[c][2] = r.z; qb[c][3] = r.w;
    }
    // No wait for the cluster scan here. This kernel is scheduled once every block of the cluster scan has passed ITS
    // wait for the insertion, so what the scan below reads (M, the window, mu, n: left by the insertion and by earlier
    // steps) is complete; the acquire makes it visible. The cluster scan's partials are needed only by the final merge,
    // and the wait stands before this block delivers its partial.
    acquire_unit(C, u);
    // advance = 1: the query of a stream step, the step's token is in the ring but not counted yet;
    // advance = 0: a read-only query of the state as it stands
    const int n = C.n_unit[u] - (advance ? 0 : 1), w = C.w, s = C.s;
    const int wn = min(n + 1, w);
    MmaState<D> S;
    S.m0 = S.m1 = -INFINITY;
    S.tau0 = S.tau1 = 0.f;
#pragma unroll
    for (int j = 0; j < D / 16; ++j) S.acc[j][0] = S.acc[j][1] = S.acc[j][2] = S.acc[j][3] = 0.f;

    const T* Mku = C.Mk + (size_t)u * s * D;
    const T* Mvu = C.Mv + (size_t)u * s * D;
    const float* MiWu = C.MinvW + (size_t)u * s;
    const T* Rk = C.ringK + (size_t)u * w * D;
    const T* Rv = C.ringV + (size_t)u * w * D;
    const float mu_over_s = (float)C.mu[u] / (float)s;
    const int n_b = (s + 15) >> 4, n_c = (wn + 15) >> 4, total = n_b + n_c;
    int item = 0;
    if (lane == 0) item = (int)atomicAdd(&C.qnext2[u], 1u);
    item = __shfl_sync(0xffffffffu, item, 0);
    while (item < total) {
        int next = 0;
        if (lane == 0) next = (int)atomicAdd(&C.qnext2[u], 1u);
        // 16 value samples (weight mu/(s W), numerator only) or 16 window rows (weight 1, both sums)
        const bool isM = item < n_b;
        const int base = (isM ? item : item - n_b) * 16;
        const int lim = isM ? s : wn;
        const T* Kb = isM ? Mku : Rk;
        const T* Vb = isM ? Mvu : Rv;
        const int ia = min(base + g, lim - 1), ib = min(base + g + 8, lim - 1);
        bool va = base + g < lim, vb = base + g + 8 < lim;
        float wza = 1.f, wzb = 1.f;
        if (isM) {
            const float ia_w = MiWu[ia], ib_w = MiWu[ib];          // 1/W, 0 for a null slot
            va = va && ia_w != 0.f;
            vb = vb && ib_w != 0.f;
            wza = va ? mu_over_s * ia_w : 0.f;
            wzb = vb ? mu_over_s * ib_w : 0.f;
        }
        const T* pv[4];
        pv[0] = Vb + (size_t)min(base + 2 * tq, lim - 1) * D;
        pv[1] = Vb + (size_t)min(base + 2 * tq + 1, lim - 1) * D;
        pv[2] = Vb + (size_t)min(base + 2 * tq + 8, lim - 1) * D;
        pv[3] = Vb + (size_t)min(base + 2 * tq + 9, lim - 1) * D;
        uint4 ka[NC], kb[NC], v[4][D / 64];
        load_keys_stream<D>(Kb + (size_t)ia * D, Kb + (size_t)ib * D, tq, ka, kb);      // keys and values in flight together
        load_values_stream<D>(pv, g, v);
        float p[4];
        tile_scores<D, D>(S, ka, kb, va, vb, qb, p);
        if (!isM) {
            S.tau0 += p[0] + p[2];
            S.tau1 += p[1] + p[3];
        }
        const float pz[4] = {wza * p[0], wza * p[1], wzb * p[2], wzb * p[3]};
        tile_values<D>(S, pz, v, g, tq);
        item = __shfl_sync(0xffffffffu, next, 0);
    }

    // warp partial -> shared [warp][G][D+2]
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        S.tau0 += __shfl_xor_sync(0xffffffffu, S.tau0, off);
        S.tau1 += __shfl_xor_sync(0xffffffffu, S.tau1, off);
    }
    {
        const int h0 = 2 * tq, h1 = 2 * tq + 1;
        float* w0 = sm + ((size_t)warp * G + (h0 < G ? h0 : 0)) * STR;
        float* w1 = sm + ((size_t)warp * G + (h1 < G ? h1 : 0)) * STR;
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
    block_combine<D, G>(sm, part_u + (size_t)blockIdx.x * G * STR);
    pdl_wait();                     // the cluster scan is complete: its partials, its work queue
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
    // final merge: z partials of this kernel and the cluster partials {max, tau} of query_tau_kernel
    __shared__ float sred[16];
    merge_partials<T, D, G>(part_u, splits, C.part_tau + (size_t)u * splits_tau * G * 2, splits_tau, out + qrow0 * D,
                            C.status[u] != 0, sred);
    if (tid == 0) {
        if (advance) C.n_unit[u] = n + 1;
        C.ticket2[u] = 0;
        C.qnext[u] = 0;
        C.qnext2[u] = 0;
    }
}

// The same scan with the work cut evenly over the whole grid instead of per unit: all units have the same number
// of 16-row items (ipu), block b takes the global items [b T / NB, (b+1) T / NB), T = U * ipu, which belong to one
// unit or to a few consecutive ones. With NB equal to the number of resident blocks every block slot of the GPU
// has the same share, whatever the ratio of slots to units. A unit's partials come from the blocks whose ranges
// meet it; the block that delivers the last one merges. slots: partials a unit has room for in part2.
template <int D, int G>
__global__ void __launch_bounds__(kQmThreads, 4) query_z_flat_kernel(Cache<__nv_bfloat16> C, const __nv_bfloat16* __restrict__ q,
                                                                     __nv_bfloat16* __restrict__ out, int splits_tau, int advance,
                                                                     int ipu, int slots) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, STR = D + 2, NW = kQmThreads / 32;
    __shared__ float sm[NW * G * STR];
    __shared__ int sm_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, tq = lane & 3;
    const long long NB = gridDim.x, Ttot = (long long)C.B * C.Hkv * ipu;
    const long long i0 = (long long)blockIdx.x * Ttot / NB, i1 = ((long long)blockIdx.x + 1) * Ttot / NB;
    pdl_trigger();
    if (i0 >= i1) return;
    const int w = C.w, s = C.s;
    const int u_first = (int)(i0 / ipu), u_last = (int)((i1 - 1) / ipu);
    for (int u = u_first; u <= u_last; ++u) {
        const long long ulo = (long long)u * ipu;
        const int lo = (int)(max(i0, ulo) - ulo), hi = (int)(min(i1, ulo + ipu) - ulo);
        const int b = u / C.Hkv, kvh = u % C.Hkv;
        const size_t qrow0 = (size_t)b * C.H + (size_t)kvh * G;
        acquire_unit(C, u);         // no wait for the cluster scan before the scan of M and the window (see query_z_kernel)
        uint32_t qb[NC][4];
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            uint4 r = make_uint4(0, 0, 0, 0);
            if (g < G) r = ldg16(q + (qrow0 + g) * D + c * 32 + tq * 8);
            qb[c][0] = r.x; qb[c][1] = r.y; qb[c][2] = r.z; qb[c][3] = r.w;
        }
        const int n = C.n_unit[u] - (advance ? 0 : 1);
        const int wn = min(n + 1, w);
        MmaState<D> S;
        S.m0 = S.m1 = -INFINITY;
        S.tau0 = S.tau1 = 0.f;
#pragma unroll
        for (int j = 0; j < D / 16; ++j) S.acc[j][0] = S.acc[j][1] = S.acc[j][2] = S.acc[j][3] = 0.f;
        const T* Mku = C.Mk + (size_t)u * s * D;
        const T* Mvu = C.Mv + (size_t)u * s * D;
        const float* MiWu = C.MinvW + (size_t)u * s;
        const T* Rk = C.ringK + (size_t)u * w * D;
        const T* Rv = C.ringV + (size_t)u * w * D;
        const float mu_over_s = (float)C.mu[u] / (float)s;
        const int n_b = (s + 15) >> 4;
        for (int item = lo + warp; item < hi; item += NW) {
            // 16 value samples (weight mu/(s W), numerator only) or 16 window rows (weight 1, both sums)
            const bool isM = item < n_b;
            const int base = (isM ? item : item - n_b) * 16;
            const int lim = isM ? s : wn;
            const T* Kb = isM ? Mku : Rk;
            const T* Vb = isM ? Mvu : Rv;
            const int ia = min(base + g, lim - 1), ib = min(base + g + 8, lim - 1);
            bool va = base + g < lim, vb = base + g + 8 < lim;
            float wza = 1.f, wzb = 1.f;
            if (isM) {
                const float ia_w = MiWu[ia], ib_w = MiWu[ib];          // 1/W, 0 for a null slot
                va = va && ia_w != 0.f;
                vb = vb && ib_w != 0.f;
                wza = va ? mu_over_s * ia_w : 0.f;
                wzb = vb ? mu_over_s * ib_w : 0.f;
            }
            const T* pv[4];
            pv[0] = Vb + (size_t)min(base + 2 * tq, lim - 1) * D;
            pv[1] = Vb + (size_t)min(base + 2 * tq + 1, lim - 1) * D;
            pv[2] = Vb + (size_t)min(base + 2 * tq + 8, lim - 1) * D;
            pv[3] = Vb + (size_t)min(base + 2 * tq + 9, lim - 1) * D;
            uint4 ka[NC], kb[NC], v[4][D / 64];
            load_keys_stream<D>(Kb + (size_t)ia * D, Kb + (size_t)ib * D, tq, ka, kb);      // keys and values in flight together
            load_values_stream<D>(pv, g, v);
            float p[4];
            tile_scores<D, D>(S, ka, kb, va, vb, qb, p);
            if (!isM) {
                S.tau0 += p[0] + p[2];
                S.tau1 += p[1] + p[3];
            }
            const float pz[4] = {wza * p[0], wza * p[1], wzb * p[2], wzb * p[3]};
            tile_values<D>(S, pz, v, g, tq);
        }
        // warp partial -> shared [warp][G][D+2]
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            S.tau0 += __shfl_xor_sync(0xffffffffu, S.tau0, off);
            S.tau1 += __shfl_xor_sync(0xffffffffu, S.tau1, off);
        }
        {
            const int h0 = 2 * tq, h1 = 2 * tq + 1;
            float* w0 = sm + ((size_t)warp * G + (h0 < G ? h0 : 0)) * STR;
            float* w1 = sm + ((size_t)warp * G + (h1 < G ? h1 : 0)) * STR;
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
        // which blocks meet this unit: the largest b with b T / NB <= x is ((x + 1) NB - 1) / T
        const int b_first = (int)(((ulo + 1) * NB - 1) / Ttot), b_last = (int)(((ulo + ipu) * NB - 1) / Ttot);
        const int np = b_last - b_first + 1;
        float* part_u = C.part2 + (size_t)u * slots * G * STR;
        block_combine<D, G>(sm, part_u + (size_t)((int)blockIdx.x - b_first) * G * STR);
        pdl_wait();                 // the cluster scan is complete (returns at once after the first time)
        __threadfence();
        __syncthreads();
        bool last = true;
        if (np > 1) {
            if (tid == 0) {
                __threadfence();
                sm_last = (atomicAdd(&C.ticket2[u], 1u) == (unsigned)np - 1u);
            }
            __syncthreads();
            last = sm_last != 0;
            if (last) __threadfence();
        }
        if (last) {
            __shared__ float sred[16];
            merge_partials<T, D, G>(part_u, np, C.part_tau + (size_t)u * splits_tau * G * 2, splits_tau, out + qrow0 * D,
                                    C.status[u] != 0, sred);
            if (tid == 0) {
                if (advance) C.n_unit[u] = n + 1;
                C.ticket2[u] = 0;
                C.qnext[u] = 0;
            }
        }
        __syncthreads();            // sm and sm_last are reused by the next unit
    }
}

}  // namespace sgk
