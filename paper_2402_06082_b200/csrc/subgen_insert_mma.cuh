// Insert kernel for bf16 caches: the nearest-representative search with a tensor-core pre-filter.
//
// Which cluster a key joins is decided by the exact fixed-point distance D2. Computing D2 for every
// representative costs far more instructions per byte than HBM needs time to deliver the row, so the scan
// first forms an approximate squared distance ||x||^2 + ||k||^2 - 2<x,k> with the inner products on the
// tensor cores (m16n8k16, the key in column 0 of the B operand) and evaluates D2 exactly only for rows
// whose approximation is within a proven guard band of delta^2:
//     |approx - D2/2^32| < 2^-15 (||x||^2 + ||k||^2)      (fp32 accumulation of <= 128 exact products,
//                                                           fp32 norms; see the design notes)
//     flagged  <=>  approx <= delta^2 + 2^-13 (||x||^2 + ||k||^2)
// Every row with D2 <= floor(delta^2 2^32) is flagged, so "no flagged row has D2 <= threshold" is
// exactly the paper's "farther than delta from every representative" and the lexicographic minimum of
// (D2, index) over the flagged rows is the argmin whenever the key joins.
#pragma once
#include "subgen_query_mma.cuh"

namespace sgk {

constexpr int kInsertMmaThreads = 128;

template <int D, bool BND>
__global__ void __launch_bounds__(kInsertMmaThreads, 6) insert_mma_kernel(Cache<__nv_bfloat16> C, const __nv_bfloat16* __restrict__ k_new,
                                                                    const __nv_bfloat16* __restrict__ v_new) {
    typedef __nv_bfloat16 T;
    constexpr int EPL = 8, LPR = D / EPL, NC = D / 32;
    __shared__ uint4 krow[LPR], vrow[LPR];
    __shared__ Best smb[32];
    __shared__ unsigned long long sm_w[2];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5, g = lane >> 2, tq = lane & 3;
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
    const int e = n - w;
    if (tid < LPR) krow[tid] = w ? ringk[tid] : knew_u[tid];
    __syncthreads();
    const int m = C.m_unit[u];
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const float* xnu = C.xn + (size_t)u * C.m_max;

    // B operand (key in column 0) and ||k||^2
    uint32_t kb[NC][4];
    float kn = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const uint4 r = krow[c * 4 + tq];
        float f[8];
        Elem<T>::unpack(r, f);
#pragma unroll
        for (int j = 0; j < 8; ++j) kn = fmaf(f[j], f[j], kn);
        kb[c][0] = g == 0 ? r.x : 0u; kb[c][1] = g == 0 ? r.y : 0u;
        kb[c][2] = g == 0 ? r.z : 0u; kb[c][3] = g == 0 ? r.w : 0u;
    }
    kn += __shfl_xor_sync(0xffffffffu, kn, 1);
    kn += __shfl_xor_sync(0xffffffffu, kn, 2);
    const float d2f = (float)((double)threshold2<BND>(C, u) * (1.0 / 4294967296.0));

    const int per = (((m + splits - 1) / splits) + 15) & ~15;       // slices are whole tiles
    const int c0 = blockIdx.x * per, c1 = min(m, c0 + per);
    Best b;
    b.d2 = ~0ull; b.idx = INT_MAX; b.pad = 0;
    // exact D2 of one flagged row, by the whole warp
    auto exact_row = [&](int row) {
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
        if (better(acc, row, b)) { b.d2 = acc; b.idx = row; }
    };
    // approximate distances of one 16-row tile and the exact follow-up of its flagged rows
    auto filter_tile = [&](int base, const uint4 (&ka)[NC], const uint4 (&kc)[NC], bool va, bool vb) {
        const float xa = va ? xnu[base + g] : 0.f, xb = vb ? xnu[base + g + 8] : 0.f;
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            mma_bf16_16816(sc, ka[c].x, kc[c].x, ka[c].y, kc[c].y, kb[c][0], kb[c][1]);
            mma_bf16_16816(sc, ka[c].z, kc[c].z, ka[c].w, kc[c].w, kb[c][2], kb[c][3]);
        }
        // lanes with tq == 0 hold <x, k> of rows g (sc[0]) and g+8 (sc[2])
        const float na = xa + kn, nb = xb + kn;
        const bool fa = va && tq == 0 && (na - 2.f * sc[0]) <= d2f + 1.220703125e-4f * na;
        const bool fb = vb && tq == 0 && (nb - 2.f * sc[2]) <= d2f + 1.220703125e-4f * nb;
        unsigned ma = __ballot_sync(0xffffffffu, fa), mb = __ballot_sync(0xffffffffu, fb);
        while (ma) { exact_row(base + ((__ffs(ma) - 1) >> 2)); ma &= ma - 1; }      // rare
        while (mb) { exact_row(base + 8 + ((__ffs(mb) - 1) >> 2)); mb &= mb - 1; }
    };
    for (int base = c0 + warp * 16; base < c1; base += nw * 16) {
        const bool va = base + g < c1, vb = base + g + 8 < c1;
        uint4 ka[NC], kc[NC];
        load_keys<D>(Xu + (size_t)(va ? base + g : c1 - 1) * D, Xu + (size_t)(vb ? base + g + 8 : c1 - 1) * D, tq, ka, kc);
        filter_tile(base, ka, kc, va, vb);
    }
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

}  // namespace sgk
