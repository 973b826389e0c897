// Exact dense decode attention (Eq. 1) for bf16 caches with both contractions on the tensor cores:
// the same 16-row tiles, score MMA and value MMA as the value scan of the SubGen query, over all n cached
// rows with weight 1. Grouped-query heads share every load (they sit in the N dimension of the MMAs).
#pragma once
#include "subgen_kernels.cuh"
#include "subgen_query_mma.cuh"

namespace sgk {

// grid (splits, U). The step's own token has been appended before the launch; n = E.n_unit[u] rows are scanned.
template <int D, int G>
__global__ void __launch_bounds__(kQmThreads, 4) exact_mma_kernel(ExactCache<__nv_bfloat16> E, const __nv_bfloat16* __restrict__ q,
                                                                  __nv_bfloat16* __restrict__ out) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, STR = D + 2, NW = kQmThreads / 32;
    __shared__ float sm[NW * G * STR];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, tq = lane & 3;
    const int b = u / E.Hkv, kvh = u % E.Hkv;
    const int n = E.n_unit[u];
    const size_t qrow0 = (size_t)b * E.H + (size_t)kvh * G;

    uint32_t qb[NC][4];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        uint4 r = make_uint4(0, 0, 0, 0);
        if (g < G) r = ldg16(q + (qrow0 + g) * D + c * 32 + tq * 8);
        qb[c][0] = r.x; qb[c][1] = r.y; qb[c][2] = r.z; qb[c][3] = r.w;
    }
    MmaState<D> S;
    S.m0 = S.m1 = -INFINITY;
    S.tau0 = S.tau1 = 0.f;
#pragma unroll
    for (int j = 0; j < D / 16; ++j) S.acc[j][0] = S.acc[j][1] = S.acc[j][2] = S.acc[j][3] = 0.f;

    const T* Ku = E.Kc + (size_t)u * E.n_max * D;
    const T* Vu = E.Vc + (size_t)u * E.n_max * D;
    const int total = (n + 15) >> 4;
    int item = 0;
    if (lane == 0) item = (int)atomicAdd(&E.qnext[u], 1u);
    item = __shfl_sync(0xffffffffu, item, 0);
    while (item < total) {
        int next = 0;
        if (lane == 0) next = (int)atomicAdd(&E.qnext[u], 1u);     // asked for early, needed late
        const int base = item * 16;
        const int ia = min(base + g, n - 1), ib = min(base + g + 8, n - 1);
        const bool va = base + g < n, vb = base + g + 8 < n;
        const T* pv[4];
        pv[0] = Vu + (size_t)min(base + 2 * tq, n - 1) * D;
        pv[1] = Vu + (size_t)min(base + 2 * tq + 1, n - 1) * D;
        pv[2] = Vu + (size_t)min(base + 2 * tq + 8, n - 1) * D;
        pv[3] = Vu + (size_t)min(base + 2 * tq + 9, n - 1) * D;
        uint4 ka[NC], kb[NC], v[4][D / 64];
        load_keys<D>(Ku + (size_t)ia * D, Ku + (size_t)ib * D, tq, ka, kb);
        load_values<D>(pv, g, v);
        float p[4];
        tile_scores<D, D>(S, ka, kb, va, vb, qb, p);
        S.tau0 += p[0] + p[2];
        S.tau1 += p[1] + p[3];
        tile_values<D>(S, p, v, g, tq);
        item = __shfl_sync(0xffffffffu, next, 0);
    }
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
    float* part_u = E.part + (size_t)u * splits * G * STR;
    block_combine<D, G>(sm, part_u + (size_t)blockIdx.x * G * STR);
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
        E.ticket[u] = 0;
        E.qnext[u] = 0;
    }
}

}  // namespace sgk
