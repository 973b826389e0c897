// Offline greedy k-center compression of a full KV cache with a recent-token window (the variant of the
// paper's end-to-end experiment, Section 3.2): keep the r most recent tokens and k centres chosen among the
// older ones by farthest-point traversal; afterwards the kept tokens are attended exactly.
//
// One launch per centre: every block first finds the newest centre (argmax of the running distance array from
// the partials the previous launch left; the first centre is the oldest token), then folds the fixed-point
// distance to it into the distance array of its slice of tokens and leaves its own partial argmax. Distances
// are the order-independent integers D2 used everywhere else, ties go to the lowest token index, so the
// selection is unique.
//
// A token's running distance can only change if D2(token, new centre) is below it. D2 is a sum of non-negative
// terms, so the terms of the first kKcHead coordinates alone are a lower bound, and a binary32 sum of squares
// shrunk by its rounding slack is a lower bound of those. Each pass therefore reads, per token, a 16-coordinate
// head (kept in planes of one uint4 per token so that the loads coalesce) and the running distance, and goes
// to the full row only where that bound does not settle the comparison; there a binary32 bound over all
// coordinates is tried before the integer sum. Skipping never changes a result: a skipped token's running
// distance is exactly what the full evaluation would have left.
#pragma once
#include "subgen_kernels.cuh"

namespace sgk {

constexpr int kKcThreads = 128;
constexpr int kKcSliceMax = 16384;                // tokens per block: the survivor list holds 16-bit offsets
constexpr int kKcHead = 16;                       // coordinates in the head
constexpr int kKcRows = 4;                        // full rows in flight per lane group

__device__ __forceinline__ bool farther(unsigned long long d2, int idx, const Best& b) {
    return d2 > b.d2 || (d2 == b.d2 && idx < b.idx);
}

// Lower bound of the fixed-point sum of `terms` (<= 160) squared differences, given their binary32 sum of
// squares s (differences rounded once, then fused multiply-adds and adds in any order). Rounding of the
// float sum is below 2^-17 relative, each fixed-point term is within 2^-22 relative of the real square and
// loses less than one unit to truncation.
__device__ __forceinline__ unsigned long long fx_lower_bound(float s, int terms) {
    s = fminf(s, 1073741824.0f);
    const unsigned long long v = __float2ull_rz(__fmul_rn(__fmul_rn(s, 0.999969482421875f), 4294967296.0f));
    return v > (unsigned long long)terms ? v - (unsigned long long)terms : 0ull;
}

// Head planes and the running distances. grid (blocks, U). head: [U, HP, n_max] uint4, HP = kKcHead / EPL.
template <typename T, int D>
__global__ void kcenter_init_kernel(ExactCache<T> E, int r, uint4* head, unsigned long long* dist) {
    constexpr int HP = kKcHead / Elem<T>::EPL;
    const int u = blockIdx.y;
    const int n_old = max(0, E.n_unit[u] - r);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_old; i += gridDim.x * blockDim.x) {
        const uint4* row = reinterpret_cast<const uint4*>(E.Kc + ((size_t)u * E.n_max + i) * D);
#pragma unroll
        for (int p = 0; p < HP; ++p) head[((size_t)u * HP + p) * E.n_max + i] = row[p];
        dist[(size_t)u * E.n_max + i] = ~0ull;
    }
}

// grid (S, U). t: index of the centre being added. part_prev / part_cur: [U, S] partial argmax of the running
// distances after centre t-1 / after centre t. counters[0] += tokens looked at, counters[1] += full rows read.
template <typename T, int D>
__global__ void __launch_bounds__(kKcThreads) kcenter_iter_kernel(ExactCache<T> E, int t, int k, int r, const uint4* head,
                                                                  unsigned long long* dist, int* centres, const Best* part_prev,
                                                                  Best* part_cur, unsigned long long* counters) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR, HP = kKcHead / EPL;
    __shared__ uint4 crow[LPR];
    __shared__ Best smb[32];
    extern __shared__ unsigned short surv[];   // offsets into the slice of the tokens that need their full row
    __shared__ int nsurv;
    const int u = blockIdx.y, S = gridDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = kKcThreads >> 5;
    const int lr = lane % LPR, sub = lane / LPR;
    pdl_trigger();                       // the next pass may be scheduled; it waits for this one right here
    pdl_wait();
    const int n = E.n_unit[u], n_old = max(0, n - r);
    if (t >= min(k, n_old)) return;
    // the newest centre
    Best b;
    b.d2 = 0ull; b.idx = INT_MAX; b.pad = 0;
    if (t > 0) {
        for (int i = tid; i < S; i += kKcThreads) {
            const Best p = part_prev[(size_t)u * S + i];
            if (farther(p.d2, p.idx, b)) b = p;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long od = __shfl_xor_sync(0xffffffffu, b.d2, off);
            const int oi = __shfl_xor_sync(0xffffffffu, b.idx, off);
            if (farther(od, oi, b)) { b.d2 = od; b.idx = oi; }
        }
        if (lane == 0) smb[warp] = b;
        __syncthreads();
        b = smb[0];
        for (int i = 1; i < nw; ++i) if (farther(smb[i].d2, smb[i].idx, b)) b = smb[i];
        __syncthreads();
    }
    const int c = t == 0 ? 0 : b.idx;
    if (blockIdx.x == 0 && tid == 0) centres[(size_t)u * k + t] = c;
    const T* Ku = E.Kc + (size_t)u * E.n_max * D;
    if (tid < LPR) crow[tid] = reinterpret_cast<const uint4*>(Ku + (size_t)c * D)[tid];
    __syncthreads();
    float cf[EPL], ch[kKcHead];
    Elem<T>::unpack(crow[lr], cf);
#pragma unroll
    for (int p = 0; p < HP; ++p) Elem<T>::unpack(crow[p], ch + p * EPL);

    const int per = (n_old + S - 1) / S, p0 = blockIdx.x * per, p1 = min(n_old, p0 + per);
    unsigned long long* du = dist + (size_t)u * E.n_max;
    const uint4* hu = head + (size_t)u * HP * E.n_max;
    Best far;
    far.d2 = 0ull; far.idx = INT_MAX; far.pad = 0;
    const int group = warp * RPW + sub, ngroups = nw * RPW;
    if (tid == 0) nsurv = 0;
    __syncthreads();
    // head filter over the whole slice, one token per thread and turn
    for (int i0 = p0; i0 < p1; i0 += kKcThreads * 4) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = i0 + q * kKcThreads + tid;
            if (i < p1) {
                const unsigned long long di = du[i];
                float s = 0.0f;
#pragma unroll
                for (int p = 0; p < HP; ++p) {
                    float xf[EPL];
                    Elem<T>::unpack(hu[(size_t)p * E.n_max + i], xf);
#pragma unroll
                    for (int j = 0; j < EPL; ++j) {
                        const float df = xf[j] - ch[p * EPL + j];
                        s = fmaf(df, df, s);
                    }
                }
                if (fx_lower_bound(s, kKcHead) >= di) {
                    if (farther(di, i, far)) { far.d2 = di; far.idx = i; }
                } else {
                    surv[atomicAdd(&nsurv, 1)] = (unsigned short)(i - p0);
                }
            }
        }
    }
    __syncthreads();
    const int ns = nsurv;
    {
        // full rows of the tokens the head did not settle: LPR lanes per row, kKcRows rows per group and turn
        for (int base = 0; base < ns; base += ngroups * kKcRows) {
            int ri[kKcRows];
            uint4 raw[kKcRows];
            unsigned long long dq[kKcRows];
#pragma unroll
            for (int q = 0; q < kKcRows; ++q) {
                const int j = base + q * ngroups + group;
                ri[q] = j < ns ? p0 + (int)surv[j] : -1;
            }
#pragma unroll
            for (int q = 0; q < kKcRows; ++q) {
                if (ri[q] >= 0) {
                    raw[q] = *reinterpret_cast<const uint4*>(Ku + (size_t)ri[q] * D + lr * EPL);
                    dq[q] = du[ri[q]];
                } else {
                    raw[q] = crow[lr];
                    dq[q] = 0ull;
                }
            }
#pragma unroll
            for (int q = 0; q < kKcRows; ++q) {
                float xf[EPL];
                Elem<T>::unpack(raw[q], xf);
                float s = 0.0f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) {
                    const float df = xf[e] - cf[e];
                    s = fmaf(df, df, s);
                }
#pragma unroll
                for (int off = 1; off < LPR; off <<= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
                const bool need = fx_lower_bound(s, D) < dq[q];
                unsigned long long acc = 0;
                if (need) {
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc += fx_sqdiff(cf[e], xf[e]);
                }
#pragma unroll
                for (int off = 1; off < LPR; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (ri[q] >= 0) {
                    unsigned long long nd = dq[q];
                    if (need && acc < nd) {
                        nd = acc;
                        if (lr == 0) du[ri[q]] = nd;
                    }
                    if (farther(nd, ri[q], far)) { far.d2 = nd; far.idx = ri[q]; }
                }
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long od = __shfl_xor_sync(0xffffffffu, far.d2, off);
        const int oi = __shfl_xor_sync(0xffffffffu, far.idx, off);
        if (farther(od, oi, far)) { far.d2 = od; far.idx = oi; }
    }
    if (lane == 0) smb[warp] = far;
    __syncthreads();
    if (tid == 0) {
        Best f = smb[0];
        for (int i = 1; i < nw; ++i) if (farther(smb[i].d2, smb[i].idx, f)) f = smb[i];
        part_cur[(size_t)u * S + blockIdx.x] = f;
        atomicAdd(counters, (unsigned long long)max(0, p1 - p0));
        atomicAdd(counters + 1, (unsigned long long)ns);
    }
}

// Gathers the kept rows (centres in selection order, then the window) into scratch. grid (blocks, U).
template <typename T, int D>
__global__ void kcenter_gather_kernel(ExactCache<T> E, int k, int r, const int* centres, T* Kt, T* Vt, int* tokt, int keep_max) {
    constexpr int LPR = D / Elem<T>::EPL;
    const int u = blockIdx.y;
    const int n = E.n_unit[u], n_old = max(0, n - r), kk = min(k, n_old), nn = kk + (n - n_old);
    for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < nn * LPR; p += gridDim.x * blockDim.x) {
        const int j = p / LPR, part = p % LPR;
        const int src = j < kk ? centres[(size_t)u * k + j] : n_old + (j - kk);
        reinterpret_cast<uint4*>(Kt + ((size_t)u * keep_max + j) * D)[part] =
            reinterpret_cast<const uint4*>(E.Kc + ((size_t)u * E.n_max + src) * D)[part];
        reinterpret_cast<uint4*>(Vt + ((size_t)u * keep_max + j) * D)[part] =
            reinterpret_cast<const uint4*>(E.Vc + ((size_t)u * E.n_max + src) * D)[part];
        if (part == 0) tokt[(size_t)u * keep_max + j] = E.tok[(size_t)u * E.n_max + src];
    }
}

// Writes the kept rows back to the front of the cache. grid (blocks, U). The lengths change in the commit kernel.
template <typename T, int D>
__global__ void kcenter_scatter_kernel(ExactCache<T> E, int k, int r, const T* Kt, const T* Vt, const int* tokt, int keep_max) {
    constexpr int LPR = D / Elem<T>::EPL;
    const int u = blockIdx.y;
    const int n = E.n_unit[u], n_old = max(0, n - r), kk = min(k, n_old), nn = kk + (n - n_old);
    for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < nn * LPR; p += gridDim.x * blockDim.x) {
        const int j = p / LPR, part = p % LPR;
        reinterpret_cast<uint4*>(E.Kc + ((size_t)u * E.n_max + j) * D)[part] =
            reinterpret_cast<const uint4*>(Kt + ((size_t)u * keep_max + j) * D)[part];
        reinterpret_cast<uint4*>(E.Vc + ((size_t)u * E.n_max + j) * D)[part] =
            reinterpret_cast<const uint4*>(Vt + ((size_t)u * keep_max + j) * D)[part];
        if (part == 0) E.tok[(size_t)u * E.n_max + j] = tokt[(size_t)u * keep_max + j];
    }
}

template <typename T>
__global__ void kcenter_commit_kernel(ExactCache<T> E, int U, int k, int r) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const int n = E.n_unit[u], n_old = max(0, n - r);
    E.n_unit[u] = min(k, n_old) + (n - n_old);
}

}  // namespace sgk
