// Insert kernel for bf16 caches: the nearest-representative search with a tensor-core pre-filter over packed
// heads of the representatives.
//
// Which cluster a key joins is decided by the exact fixed-point distance D2. D2 is a sum of non-negative terms,
// so the distance over the first kHeadDims coordinates is a lower bound of it. The scan therefore reads only the
// packed heads (kHeadDims coordinates per representative, a quarter of a d = 128 row) and their squared norms,
// forms the approximate head distance ||xh||^2 + ||kh||^2 - 2<xh,kh> with the inner products on the tensor cores
// (m16n8k16, the key's head in column 0 of the B operand) and evaluates D2 exactly, from the full row, only for
// representatives whose head distance is within a proven guard band of the threshold:
//     |approx - exact head distance| < 2^-15 (||xh||^2 + ||kh||^2)   (fp32 accumulation of <= 32 exact products,
//                                                                     fp32 norms)
//     flagged  <=>  approx <= delta^2 + 2^-13 (||xh||^2 + ||kh||^2)
// Every row with D2 <= floor(delta^2 2^32) is flagged, so "no flagged row has D2 <= threshold" is exactly the
// paper's "farther than delta from every representative" and the lexicographic minimum of (D2, index) over the
// flagged rows is the argmin whenever the key joins. On keys that cluster, the flagged rows are the few
// representatives near the key; on keys whose first coordinates carry no information every row is flagged and
// the scan costs what a scan of the full rows costs.
#pragma once
#include "subgen_query_mma.cuh"

namespace sgk {

constexpr int kInsertMmaThreads = 128;

// MODE 0: the whole insertion of a step. A host-buffer step cannot overlap with its successor (the host waits for the
// result), so there the search for the NEXT step's leaving token is launched behind the step, where it runs while the
// host is busy, and the next step only applies it:
// MODE 1: search only, for the token that the next step will take out of the window (windows of one row or more:
//         that token is in the ring already); leaves the nearest representative in next_best[u]. k_new, v_new unused.
// MODE 2: apply only (grid.x = 1): takes the nearest representative from next_best[u]. Valid while nothing but that
//         search has run on the handle since the step before (the host keeps track).
template <int D, bool BND, int MODE = 0>
__global__ void __launch_bounds__(kInsertMmaThreads, 6) insert_mma_kernel(Cache<__nv_bfloat16> C, const __nv_bfloat16* __restrict__ k_new,
                                                                    const __nv_bfloat16* __restrict__ v_new) {
    typedef __nv_bfloat16 T;
    constexpr int EPL = 8, LPR = D / EPL;
    __shared__ uint4 krow[LPR], vrow[LPR];
    __shared__ Best smb[32];
    __shared__ unsigned long long sm_w[2];
    __shared__ int sm_last;
    const int u = C.order ? C.order[blockIdx.y] : (int)blockIdx.y, splits = gridDim.x, tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5, g = lane >> 2, tq = lane & 3;
    // The search for the nearest representative needs nothing that the previous step's scans write and nothing of
    // this call's inputs (the token that leaves the window has been in the ring since an earlier insertion), so it
    // runs before the wait for the rest of the stream, under the tail of the previous step's value scan. What it reads
    // was written by earlier insertion kernels, the latest of which released the unit's epoch = tokens seen: the
    // acquire load makes all of it visible and replaces the token counter, which the previous step's value scan may
    // still be about to advance. The wait comes before the first touch of an input (window 0: right here) and before
    // the insertion is applied; the successor (the cluster scan, which loads the call's queries before its own wait)
    // is let go only after the wait, i.e. once everything that precedes this call in the stream has completed.
    const int w = C.w;
    if (w == 0) pdl_wait();
    __shared__ int sm_n;
    if (tid == 0) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(C.epoch + u) : "memory");
        sm_n = v;
    }
    __syncthreads();
    const int n = sm_n;
    const uint4* knew_u = reinterpret_cast<const uint4*>(k_new + (size_t)u * D);
    const uint4* vnew_u = reinterpret_cast<const uint4*>(v_new + (size_t)u * D);
    const int slot = w ? n % w : 0;
    uint4* ringk = w ? reinterpret_cast<uint4*>(C.ringK + ((size_t)u * w + slot) * D) : nullptr;
    uint4* ringv = w ? reinterpret_cast<uint4*>(C.ringV + ((size_t)u * w + slot) * D) : nullptr;
    if (w && n < w) {                       // window not full yet: nothing leaves it
        if (MODE == 1) pdl_wait();
        if (MODE != 1 && blockIdx.x == 0) {
            pdl_wait();
            pdl_trigger();
            if (tid < LPR) ringk[tid] = knew_u[tid];
            else if (tid < 2 * LPR) ringv[tid - LPR] = vnew_u[tid - LPR];
            __syncthreads();
            if (tid == 0) release_unit(C, u, n + 1);          // the value scan of this step may read the window now
        }
        return;
    }
    const int e = n - w;
    // key and value of the token that leaves the window: both fetched now, so that the block that ends up applying
    // the insertion does not wait for the value row after the scan
    // (ring rows past the L1: this runs before the dependency wait)
    if (tid < LPR) krow[tid] = w ? __ldcg(ringk + tid) : knew_u[tid];
    else if (tid < 2 * LPR) vrow[tid - LPR] = w ? __ldcg(ringv + (tid - LPR)) : vnew_u[tid - LPR];
    __syncthreads();
    const int m = C.m_unit[u];
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const T* Xhu = C.Xh + (size_t)u * C.m_max * kHeadDims;
    const float* xhnu = C.xhn + (size_t)u * C.m_max;

    // B operand (head of the key in column 0) and the squared norm of that head. D2 is a sum of non-negative
    // terms, so the distance over the first kHeadDims coordinates bounds it from below: a representative whose
    // head distance is already beyond the threshold (plus the guard for the approximate arithmetic) cannot be
    // joined, and only the others need their full row.
    uint32_t kb[4];
    float kn = 0.f;
    {
        const uint4 r = krow[tq];
        float f[8];
        Elem<T>::unpack(r, f);
#pragma unroll
        for (int j = 0; j < 8; ++j) kn = fmaf(f[j], f[j], kn);
        kb[0] = g == 0 ? r.x : 0u; kb[1] = g == 0 ? r.y : 0u;
        kb[2] = g == 0 ? r.z : 0u; kb[3] = g == 0 ? r.w : 0u;
    }
    kn += __shfl_xor_sync(0xffffffffu, kn, 1);
    kn += __shfl_xor_sync(0xffffffffu, kn, 2);
    const float d2f = (float)((double)threshold2<BND>(C, u) * (1.0 / 4294967296.0));

    const int per = (((m + splits - 1) / splits) + 15) & ~15;       // slices are whole tiles
    const int c0 = blockIdx.x * per, c1 = MODE == 2 ? c0 : min(m, c0 + per);     // MODE 2: nothing to scan
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
    // kTiles tiles of 16 heads per warp and turn: all loads first, then the approximate head distances by MMA
    // (lanes with tq == 0 hold <x, k> of rows g and g + 8) and the exact follow-up of the flagged rows
    constexpr int kTiles = 4;
    for (int base = c0 + warp * 16 * kTiles; base < c1; base += nw * 16 * kTiles) {
        uint4 ka[kTiles], kc[kTiles];
        float xa[kTiles], xb[kTiles];
#pragma unroll
        for (int i = 0; i < kTiles; ++i) {
            const int ra = base + i * 16 + g, rb = ra + 8;
            const bool va = ra < c1, vb = rb < c1;
            ka[i] = ldg16(Xhu + (size_t)(va ? ra : c1 - 1) * kHeadDims + tq * 8);
            kc[i] = ldg16(Xhu + (size_t)(vb ? rb : c1 - 1) * kHeadDims + tq * 8);
            xa[i] = va ? xhnu[ra] : 0.f;
            xb[i] = vb ? xhnu[rb] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < kTiles; ++i) {
            const int ra = base + i * 16 + g, rb = ra + 8;
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            mma_bf16_16816(sc, ka[i].x, kc[i].x, ka[i].y, kc[i].y, kb[0], kb[1]);
            mma_bf16_16816(sc, ka[i].z, kc[i].z, ka[i].w, kc[i].w, kb[2], kb[3]);
            const float na = xa[i] + kn, nb = xb[i] + kn;
            const bool fa = ra < c1 && tq == 0 && (na - 2.f * sc[0]) <= d2f + 1.220703125e-4f * na;
            const bool fb = rb < c1 && tq == 0 && (nb - 2.f * sc[2]) <= d2f + 1.220703125e-4f * nb;
            unsigned ma = __ballot_sync(0xffffffffu, fa), mb = __ballot_sync(0xffffffffu, fb);
            while (ma) { exact_row(base + i * 16 + ((__ffs(ma) - 1) >> 2)); ma &= ma - 1; }
            while (mb) { exact_row(base + i * 16 + 8 + ((__ffs(mb) - 1) >> 2)); mb &= mb - 1; }
        }
    }
    if (MODE == 2) {
        const ulonglong2 raw = __ldcg(reinterpret_cast<const ulonglong2*>(C.next_best + u));
        b.d2 = raw.x; b.idx = (int)(raw.y & 0xffffffffull);
    } else {
        b = block_best(b, smb);
    }
    if (MODE != 2 && splits > 1) {
        if (tid == 0) {
            C.part1[(size_t)u * splits + blockIdx.x] = b;
            // arrival ticket: the release half publishes this block's candidate, the acquire half lets the last block
            // read everybody else's
            unsigned old;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(&C.ticket1[u]) : "memory");
            sm_last = (old == (unsigned)splits - 1u);
        }
        __syncthreads();
        if (!sm_last) return;
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
    if (MODE == 1) {
        if (tid == 0) C.next_best[u] = b;
        pdl_wait();                         // this kernel's completion stands for that of everything before it
        return;
    }
    // From here on the state that the previous step's scans read is overwritten, and the call's inputs are read.
    pdl_wait();
    pdl_trigger();
    // the new token's rows are asked for now and stored after the insertion (one round trip less at the end)
    uint4 fresh = make_uint4(0, 0, 0, 0);
    if (w) {
        if (tid < LPR) fresh = knew_u[tid];
        else if (tid < 2 * LPR) fresh = vnew_u[tid - LPR];
    }
    apply_insert<T, D, BND>(C, u, e, b, m, krow, vrow, sm_w);
    if (w) {
        if (tid < LPR) ringk[tid] = fresh;
        else if (tid < 2 * LPR) ringv[tid - LPR] = fresh;
    }
    // everything the value scan of this step reads (M, the window row, mu) has been written by this block
    __syncthreads();
    if (tid == 0) release_unit(C, u, n + 1);
}

// Units ranked by their cluster count, largest first (ties: lower unit first): order[rank] = unit. Blocks are handed
// to the SMs in grid order, so with several waves of one block per unit the long units start first and the short ones
// fill the end. Units of about one size (largest count within 5/4 of the smallest) keep their own order: nothing is
// gained there, and neighbouring units share a sequence's rows. One thread per unit, O(U) each; launched after a prefill.
__global__ void unit_order_kernel(Cache<__nv_bfloat16> C, int U, int* order) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const int mu = C.m_unit[u];
    int rank = 0, mn = mu, mx = mu;
    for (int v = 0; v < U; ++v) {
        const int mv = __ldg(C.m_unit + v);
        rank += (mv > mu) || (mv == mu && v < u);
        mn = min(mn, mv);
        mx = max(mx, mv);
    }
    if ((long long)mx * 4 <= (long long)mn * 5) order[u] = u;
    else order[rank] = u;
}

// The units' epochs (see acquire_unit) set to their token counts: launched before the first stream step that follows
// a prefill, a checkpoint load or the handle's creation, whose kernels advance the counts without touching the epochs.
__global__ void epoch_sync_kernel(Cache<__nv_bfloat16> C, int U) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u < U) {
        C.epoch[u] = C.n_unit[u];
        C.m_hist[u] = C.m_hist[U + u] = C.m_unit[u];
    }
}

}  // namespace sgk
