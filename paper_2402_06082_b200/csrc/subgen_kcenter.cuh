// Offline greedy k-center compression of a full KV cache with a recent-token window (the variant of the
// paper's end-to-end experiment, Section 3.2): keep the r most recent tokens and k centres chosen among the
// older ones by farthest-point traversal; afterwards the kept tokens are attended exactly.
//
// One launch per centre: every block first finds the newest centre (argmax of the running distance array from
// the partials the previous launch left; the first centre is the oldest token), then folds the fixed-point
// distance to it into the distance array of its slice of tokens and leaves its own partial argmax. Distances
// are the order-independent integers D2 used everywhere else, ties go to the lowest token index, so the
// selection is unique.
#pragma once
#include "subgen_kernels.cuh"

namespace sgk {

constexpr int kKcThreads = 256;

__device__ __forceinline__ bool farther(unsigned long long d2, int idx, const Best& b) {
    return d2 > b.d2 || (d2 == b.d2 && idx < b.idx);
}

// grid (S, U). t: index of the centre being added. part_prev / part_cur: [U, S] partial argmax of the running
// distances after centre t-1 / after centre t.
template <typename T, int D>
__global__ void __launch_bounds__(kKcThreads) kcenter_iter_kernel(ExactCache<T> E, int t, int k, int r, unsigned long long* dist,
                                                                  int* centres, const Best* part_prev, Best* part_cur) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR;
    __shared__ uint4 crow[LPR];
    __shared__ Best smb[32];
    const int u = blockIdx.y, S = gridDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = kKcThreads >> 5;
    const int lr = lane % LPR, sub = lane / LPR;
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
    float cf[EPL];
    Elem<T>::unpack(crow[lr], cf);
    // fold the distance to centre c into this block's slice
    const int per = (n_old + S - 1) / S, p0 = blockIdx.x * per, p1 = min(n_old, p0 + per);
    unsigned long long* du = dist + (size_t)u * E.n_max;
    Best far;
    far.d2 = 0ull; far.idx = INT_MAX; far.pad = 0;
    const int group = warp * RPW + sub, ngroups = nw * RPW;
    for (int base = p0; base < p1; base += ngroups) {
        const int i = base + group;
        unsigned long long acc = 0;
        if (i < p1) {
            float xf[EPL];
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(Ku + (size_t)i * D + lr * EPL), xf);
#pragma unroll
            for (int j = 0; j < EPL; ++j) acc += fx_sqdiff(cf[j], xf[j]);
        }
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (i < p1) {
            unsigned long long nd = acc;
            if (t > 0) nd = min(nd, du[i]);
            if (lr == 0) du[i] = nd;
            if (farther(nd, i, far)) { far.d2 = nd; far.idx = i; }
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
