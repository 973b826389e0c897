// Chunked prefill for bf16 caches: builds the same state as token-by-token insertion, in parallel.
//
// Only two things in Algorithm 1 are sequential in the token index: which representatives exist when a
// key arrives (UpdateSoftmaxNormalizer) and the order in which coins overwrite a slot. Everything else is
// a function of (token, unit, slot) alone, because the coins are counter-based and the running mu is an
// integer prefix sum. The prefill therefore runs as
//
//   values (UpdateMatrixProduct, whole prompt at once)
//     W kernel      W(v_e) for every inserted token, input range check
//     scan kernel   tot_e = mu_before + sum_{e' <= e} W_e'   (64-bit integers: any order gives the same bits)
//     coin kernel   slot i keeps the LAST token whose coin u*(tot_e) < W_e 2^32 succeeds (as u < ceil(W_e 2^32 / tot_e);
//                   atomicMax on the token index)
//     gather kernel copies the winners' rows into M
//   keys (UpdateSoftmaxNormalizer), chunk by chunk of kChunk tokens
//     score kernel  chunk x existing representatives as a dense contraction on the tensor cores
//                   (approximate squared distances), exact fixed-point D2 only inside the guard band
//     resolve kernel opens new representatives in stream order (a key opens only if it is farther than
//                   delta from every representative, including those opened earlier in the chunk), assigns
//                   every key, ranks keys inside their cluster (the count each cluster coin sees), flips
//                   the cluster coins and writes the last successful key of every (cluster, slot)
//   finish kernel   window rows, token counts, mu
#pragma once
#include "subgen_insert_mma.cuh"

namespace sgk {

constexpr int kChunk = 128;            // tokens per chunk
constexpr int kScoreThreads = 128;
constexpr int kResolveThreads = 512;

struct PrefillArgs {
    const __nv_bfloat16* K;            // new tokens
    const __nv_bfloat16* V;
    int n_uniform;                     // tokens per sequence (dense layout) ...
    const int* cu;                     // ... or packed offsets (device), NULL for dense
    int total;                         // packed: tokens over all sequences
    int Lmax;                          // longest insert range over all units (row stride of the scratch arrays)
    unsigned long long* Wbuf;          // [U, Lmax] W of the e-th inserted token of this call
    unsigned long long* Tot;           // [U, Lmax] inclusive prefix incl. mu_before
    unsigned long long* Thr;           // [U, Lmax] coin threshold ceil(W 2^32 / tot): the coin succeeds iff u < Thr
    int* Mwin;                         // [U, s] winning token per M slot, -1 none
    Best* pbest;                       // [U, slices, kChunk] partial nearest old representative per chunk token
    int* mhist;                        // [U, 2] cluster count after chunk c in slot c & 1 (both slots: the count before
                                       //        the call, until chunks 0 and 1 have been resolved)
    int slices;
};

// Token ranges of unit u for this call.
struct Range {
    int n_prev, n_add, n_tot, ins_lo, ins_hi;
    size_t row0;
};
template <typename T>
__device__ __forceinline__ Range unit_range(const Cache<T>& C, const PrefillArgs& a, int u) {
    Range r;
    const int b = u / C.Hkv, h = u % C.Hkv;
    r.n_add = a.cu ? a.cu[b + 1] - a.cu[b] : a.n_uniform;
    r.row0 = a.cu ? (size_t)h * a.total + a.cu[b] : (size_t)u * a.n_uniform;
    r.n_prev = C.n_unit[u];
    r.n_tot = r.n_prev + r.n_add;
    r.ins_lo = max(0, r.n_prev - C.w);
    r.ins_hi = max(0, r.n_tot - C.w);
    return r;
}
// Row of token e: still in the window from an earlier call, or among the new tokens.
template <int D>
__device__ __forceinline__ const __nv_bfloat16* key_row(const Cache<__nv_bfloat16>& C, const PrefillArgs& a, const Range& r, int u,
                                                        int e) {
    return e < r.n_prev ? C.ringK + ((size_t)u * C.w + e % C.w) * D : a.K + (r.row0 + (e - r.n_prev)) * D;
}
template <int D>
__device__ __forceinline__ const __nv_bfloat16* val_row(const Cache<__nv_bfloat16>& C, const PrefillArgs& a, const Range& r, int u,
                                                        int e) {
    return e < r.n_prev ? C.ringV + ((size_t)u * C.w + e % C.w) * D : a.V + (r.row0 + (e - r.n_prev)) * D;
}

// ---------------------------------------------------------------------------------------------
// W(v_e) and the input range check. grid (blocks, U); a row group of D/8 lanes per token.
template <int D>
__global__ void prefill_w_kernel(Cache<__nv_bfloat16> C, PrefillArgs a) {
    typedef __nv_bfloat16 T;
    constexpr int LPR = D / 8, RPW = 32 / LPR;
    const int u = blockIdx.y, lane = threadIdx.x & 31, lr = lane % LPR, sub = lane / LPR;
    const Range r = unit_range(C, a, u);
    const int groups = gridDim.x * (blockDim.x >> 5) * RPW;
    const int gid = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * RPW + sub;
    const int len = r.ins_hi - r.ins_lo;
    bool bad = false;
    for (int base = 0; base < len; base += groups) {
        const int i = base + gid;
        unsigned long long acc = 0;
        if (i < len) {
            float vf[8], kf[8];
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(val_row<D>(C, a, r, u, r.ins_lo + i) + lr * 8), vf);
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, r.ins_lo + i) + lr * 8), kf);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                acc += fx_sq(vf[j]);
                bad |= !(fabsf(vf[j]) <= kMaxAbsInput) || !(fabsf(kf[j]) <= kMaxAbsInput);
            }
        }
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (i < len && lr == 0) a.Wbuf[(size_t)u * a.Lmax + i] = acc;
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(&C.status[u], 2);
}

// Inclusive prefix sums of W plus mu_before. One block per unit.
__global__ void prefill_scan_kernel(Cache<__nv_bfloat16> C, PrefillArgs a) {
    __shared__ unsigned long long wsum[32];
    __shared__ unsigned long long carry;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
    const Range r = unit_range(C, a, u);
    const int len = r.ins_hi - r.ins_lo;
    if (tid == 0) carry = C.mu[u];
    __syncthreads();
    for (int base = 0; base < len; base += blockDim.x) {
        const int i = base + tid;
        unsigned long long x = i < len ? a.Wbuf[(size_t)u * a.Lmax + i] : 0ull;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) wsum[warp] = x;
        __syncthreads();
        unsigned long long pre = carry;
        for (int wv = 0; wv < warp; ++wv) pre += wsum[wv];
        if (i < len) {
            const unsigned long long W = a.Wbuf[(size_t)u * a.Lmax + i], tot = pre + x;
            a.Tot[(size_t)u * a.Lmax + i] = tot;
            // u * tot < W 2^32  <=>  u < ceil(W 2^32 / tot): one long division per token instead of a 128-bit
            // product per coin (W <= tot < 2^63, so the shifted remainder never overflows)
            unsigned long long q = 0, rem = W;
            if (W) {
                if (W == tot) q = 1ull << 32;
                else {
                    for (int bit = 0; bit < 32; ++bit) {
                        rem <<= 1;
                        q <<= 1;
                        if (rem >= tot) { rem -= tot; q |= 1ull; }
                    }
                    if (rem) ++q;
                }
            }
            a.Thr[(size_t)u * a.Lmax + i] = q;
        }
        __syncthreads();
        if (tid == blockDim.x - 1) {
            unsigned long long tot = carry;
            for (int wv = 0; wv < nw; ++wv) tot += wsum[wv];
            carry = tot;
        }
        __syncthreads();
    }
}

// Value coins: for every slot of M the last token of the call whose coin succeeded. One Philox block serves the
// four slots of a group, so a warp takes one group over one segment of tokens, 32 consecutive tokens per pass, the
// latest first, and stops once all four slots have their winner: the position of a slot's last success is uniform in
// the cumulative weight, so a group's scan ends after four fifths of the tokens on average, and the common pass (no
// coin of the 128 succeeds) costs one minimum and one comparison after the Philox block.
// grid (ceil(groups / warps per block), segments, U); segments are a multiple of 32 tokens long.
__global__ void prefill_coin_kernel(Cache<__nv_bfloat16> C, PrefillArgs a, int seg_len) {
    const int u = blockIdx.z, lane = threadIdx.x & 31, blk = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const Range r = unit_range(C, a, u);
    const int len = r.ins_hi - r.ins_lo;
    const int i0 = blockIdx.y * seg_len, i1 = min(len, i0 + seg_len);
    if (blk * 4 >= C.s || i0 >= i1) return;
    const unsigned long long* Tb = a.Thr + (size_t)u * a.Lmax;
    const uint32_t uid = unit_id(C, u);
    int win[4] = {-1, -1, -1, -1};
    unsigned found = 0;
    for (int top = i1; top > i0 && found != 15u; top -= 32) {
        const int i = top - 1 - lane;
        const unsigned long long thr = i >= i0 ? Tb[i] : 0ull;            // 0 (also for W = 0): never sampled
        const uint4 rr = philox4x32_10(make_uint4((uint32_t)(r.ins_lo + i), uid, (uint32_t)blk, 1u), C.key0, C.key1);
        const uint32_t mn = min(min(rr.x, rr.y), min(rr.z, rr.w));
        if (__any_sync(0xffffffffu, (unsigned long long)mn < thr)) {
            const uint32_t wd[4] = {rr.x, rr.y, rr.z, rr.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const unsigned hit = __ballot_sync(0xffffffffu, (unsigned long long)wd[q] < thr);
                if (hit && !(found >> q & 1u)) {                           // lowest lane = latest token
                    win[q] = r.ins_lo + top - 1 - (__ffs(hit) - 1);
                    found |= 1u << q;
                }
            }
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (win[q] >= 0 && blk * 4 + q < C.s) atomicMax(&a.Mwin[(size_t)u * C.s + blk * 4 + q], win[q]);
    }
}

// Copies the winners into M. grid (blocks, U); a row group per slot.
template <int D>
__global__ void prefill_gather_kernel(Cache<__nv_bfloat16> C, PrefillArgs a) {
    typedef __nv_bfloat16 T;
    constexpr int LPR = D / 8, RPW = 32 / LPR;
    const int u = blockIdx.y, lane = threadIdx.x & 31, lr = lane % LPR, sub = lane / LPR;
    const Range r = unit_range(C, a, u);
    const int groups = gridDim.x * (blockDim.x >> 5) * RPW;
    const int gid = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * RPW + sub;
    for (int i = gid; i < C.s; i += groups) {
        const int e = a.Mwin[(size_t)u * C.s + i];
        if (e < 0) continue;
        reinterpret_cast<uint4*>(C.Mk + ((size_t)u * C.s + i) * D)[lr] = reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e))[lr];
        reinterpret_cast<uint4*>(C.Mv + ((size_t)u * C.s + i) * D)[lr] = reinterpret_cast<const uint4*>(val_row<D>(C, a, r, u, e))[lr];
        if (lr == 0) {
            const unsigned long long W = a.Wbuf[(size_t)u * a.Lmax + (e - r.ins_lo)];
            C.MW[(size_t)u * C.s + i] = W;
            C.MinvW[(size_t)u * C.s + i] = 1.f / (float)W;
            C.Mtok[(size_t)u * C.s + i] = e;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Score kernel: chunk keys against the representatives that exist at the start of the chunk.
// grid (slices, U), 4 warps. Every warp walks tiles of 16 representatives (A operand, straight from global
// memory) over the 16 column tiles of 8 chunk keys (B operand, from the staged chunk in shared memory),
// forms ||x||^2 + ||k||^2 - 2<x,k> and evaluates the exact D2 of every pair inside the guard band.
// Output: per slice and chunk token the lexicographic minimum (D2, index) over the flagged pairs.
template <int D>
__global__ void __launch_bounds__(kScoreThreads) prefill_score_kernel(Cache<__nv_bfloat16> C, PrefillArgs a, int chunk) {
    typedef __nv_bfloat16 T;
    constexpr int NC = D / 32, LPR = D / 8, NW = kScoreThreads / 32, KS = D + 32;     // padded row: D*2 + 64 bytes
    __shared__ __align__(16) T keys[kChunk * KS];
    __shared__ float kn[kChunk];
    __shared__ unsigned long long wb_d2[NW][kChunk];
    __shared__ int wb_idx[NW][kChunk];
    const int u = blockIdx.y, slices = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, tq = lane & 3;
    const Range r = unit_range(C, a, u);
    const int e0 = r.ins_lo + chunk * kChunk, cl = min(kChunk, r.ins_hi - e0);
    if (cl <= 0) return;
    const int m = C.m_unit[u];
    Best* outp = a.pbest + ((size_t)u * slices + blockIdx.x) * kChunk;
    const int per = (((m + slices - 1) / slices) + 15) & ~15;
    const int c0 = blockIdx.x * per, c1 = min(m, c0 + per);
    if (c0 >= c1) {                                           // nothing to scan: report "none"
        for (int j = tid; j < kChunk; j += kScoreThreads) { Best bb; bb.d2 = ~0ull; bb.idx = INT_MAX; bb.pad = 0; outp[j] = bb; }
        return;
    }
    // stage the chunk (rows beyond cl are zero) and its squared norms
    for (int p = tid; p < kChunk * LPR; p += kScoreThreads) {
        const int j = p / LPR, part = p % LPR;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < cl) v = reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e0 + j))[part];
        *reinterpret_cast<uint4*>(keys + (size_t)j * KS + part * 8) = v;
    }
    for (int j = tid; j < NW * kChunk; j += kScoreThreads) {
        wb_d2[j / kChunk][j % kChunk] = ~0ull;
        wb_idx[j / kChunk][j % kChunk] = INT_MAX;
    }
    __syncthreads();
    for (int j = tid; j < kChunk; j += kScoreThreads) {
        float acc = 0.f;
        for (int p = 0; p < LPR; ++p) {
            float f[8];
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(keys + (size_t)j * KS + p * 8), f);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc = fmaf(f[q], f[q], acc);
        }
        kn[j] = acc;
    }
    __syncthreads();
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const float* xnu = C.xn + (size_t)u * C.m_max;
    const float d2f = (float)((double)C.delta2_fx * (1.0 / 4294967296.0));

    for (int base = c0 + warp * 16; base < c1; base += NW * 16) {
        const bool va = base + g < c1, vb = base + g + 8 < c1;
        uint4 ka[NC], kc[NC];
        load_keys<D>(Xu + (size_t)(va ? base + g : c1 - 1) * D, Xu + (size_t)(vb ? base + g + 8 : c1 - 1) * D, tq, ka, kc);
        const float xa = va ? xnu[base + g] : 0.f, xb = vb ? xnu[base + g + 8] : 0.f;
        for (int nt = 0; nt < (cl + 7) / 8; ++nt) {
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            const T* kt = keys + (size_t)(nt * 8 + g) * KS + tq * 8;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const uint4 bq = *reinterpret_cast<const uint4*>(kt + c * 32);
                mma_bf16_16816(sc, ka[c].x, kc[c].x, ka[c].y, kc[c].y, bq.x, bq.y);
                mma_bf16_16816(sc, ka[c].z, kc[c].z, ka[c].w, kc[c].w, bq.z, bq.w);
            }
            // sc: (centre g, token 2tq), (g, 2tq+1), (g+8, 2tq), (g+8, 2tq+1)
            const int j0 = nt * 8 + 2 * tq;
            const float n0 = kn[j0], n1 = kn[j0 + 1];
            const bool f0 = va && j0 < cl && (xa + n0 - 2.f * sc[0]) <= d2f + 1.220703125e-4f * (xa + n0);
            const bool f1 = va && j0 + 1 < cl && (xa + n1 - 2.f * sc[1]) <= d2f + 1.220703125e-4f * (xa + n1);
            const bool f2 = vb && j0 < cl && (xb + n0 - 2.f * sc[2]) <= d2f + 1.220703125e-4f * (xb + n0);
            const bool f3 = vb && j0 + 1 < cl && (xb + n1 - 2.f * sc[3]) <= d2f + 1.220703125e-4f * (xb + n1);
            unsigned msk[4] = {__ballot_sync(0xffffffffu, f0), __ballot_sync(0xffffffffu, f1), __ballot_sync(0xffffffffu, f2),
                               __ballot_sync(0xffffffffu, f3)};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                while (msk[q]) {                                   // exact D2 of one flagged pair, by the warp
                    const int src = __ffs(msk[q]) - 1;
                    msk[q] &= msk[q] - 1;
                    const int row = base + (src >> 2) + ((q & 2) ? 8 : 0);
                    const int tokj = nt * 8 + 2 * (src & 3) + (q & 1);
                    unsigned long long acc = 0;
                    if (lane < LPR) {
                        float xf[8], kf[8];
                        Elem<T>::unpack(*reinterpret_cast<const uint4*>(Xu + (size_t)row * D + lane * 8), xf);
                        Elem<T>::unpack(*reinterpret_cast<const uint4*>(keys + (size_t)tokj * KS + lane * 8), kf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc += fx_sqdiff(xf[e], kf[e]);
                    }
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                    if (lane == 0) {
                        Best cur;
                        cur.d2 = wb_d2[warp][tokj]; cur.idx = wb_idx[warp][tokj];
                        if (better(acc, row, cur)) { wb_d2[warp][tokj] = acc; wb_idx[warp][tokj] = row; }
                    }
                }
            }
            __syncwarp();
        }
    }
    __syncthreads();
    for (int j = tid; j < kChunk; j += kScoreThreads) {
        Best bb;
        bb.d2 = wb_d2[0][j]; bb.idx = wb_idx[0][j]; bb.pad = 0;
        for (int wv = 1; wv < NW; ++wv)
            if (better(wb_d2[wv][j], wb_idx[wv][j], bb)) { bb.d2 = wb_d2[wv][j]; bb.idx = wb_idx[wv][j]; }
        outp[j] = bb;
    }
}

// ---------------------------------------------------------------------------------------------
// Resolve kernel: one block per unit.
template <int D>
__global__ void __launch_bounds__(kResolveThreads) prefill_resolve_kernel(Cache<__nv_bfloat16> C, PrefillArgs a, int chunk) {
    typedef __nv_bfloat16 T;
    constexpr int LPR = D / 8, GPB = kResolveThreads / LPR;     // row groups per block
    __shared__ __align__(16) T keys[kChunk * D];
    __shared__ unsigned long long old_d2[kChunk], new_d2[kChunk], succ[kChunk], later[kChunk];
    __shared__ int old_idx[kChunk], new_idx[kChunk], cid[kChunk], nnew[kChunk], opened_at[kChunk];
    __shared__ unsigned char is_open[kChunk], has_later[kChunk], dropped[kChunk];
    __shared__ float kn[kChunk];
    __shared__ int sm_opened, sm_full;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int lr = tid % LPR, grp = tid / LPR;
    const Range r = unit_range(C, a, u);
    const int e0 = r.ins_lo + chunk * kChunk, cl = min(kChunk, r.ins_hi - e0);
    if (cl <= 0) return;
    const int t = C.t;
    const unsigned long long thr = C.delta2_fx;
    T* Xu = C.X + (size_t)u * C.m_max * D;
    T* Su = C.S + (size_t)u * C.m_max * t * D;
    int* cntu = C.cnt + (size_t)u * C.m_max;
    int* stoku = C.stok + (size_t)u * C.m_max * t;

    // the chunk's keys and their norms depend on no earlier kernel of this call ...
    for (int p = tid; p < cl * LPR; p += kResolveThreads) {
        const int j = p / LPR, part = p % LPR;
        reinterpret_cast<uint4*>(keys + (size_t)j * D)[part] = reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e0 + j))[part];
    }
    __syncthreads();
    for (int j = tid; j < cl; j += kResolveThreads) {                // ||k||^2 of a key that may become a representative
        float acc = 0.f;
        for (int p = 0; p < LPR; ++p) {
            float f[8];
            Elem<T>::unpack(reinterpret_cast<const uint4*>(keys + (size_t)j * D)[p], f);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc = fmaf(f[q], f[q], acc);
        }
        kn[j] = acc;
    }
    // ... the score kernel's results and the state the previous chunk left do: wait for them, then let the next
    // kernel in the stream start staging its keys
    pdl_wait();
    pdl_trigger();
    const int m_old = C.m_unit[u];
    for (int j = tid; j < cl; j += kResolveThreads) {
        Best bb; bb.d2 = ~0ull; bb.idx = INT_MAX; bb.pad = 0;
        if (m_old > 0)
            for (int sidx = 0; sidx < a.slices; ++sidx) {
                const Best p = a.pbest[((size_t)u * a.slices + sidx) * kChunk + j];
                if (better(p.d2, p.idx, bb)) bb = p;
            }
        old_d2[j] = bb.d2; old_idx[j] = bb.idx;
        new_d2[j] = ~0ull; new_idx[j] = INT_MAX;
        succ[j] = 0ull; is_open[j] = 0; dropped[j] = 0; opened_at[j] = -1;
    }
    if (tid == 0) { sm_opened = 0; sm_full = 0; }
    __syncthreads();

    // Openings in stream order. Key j opens a representative iff its nearest representative so far (old ones
    // from the score kernel, new ones from this loop) is farther than delta.
    for (int j = 0; j < cl; ++j) {
        const bool far_old = old_d2[j] > thr, far_new = new_d2[j] > thr;        // uniform: shared memory
        if (!(far_old && far_new)) continue;
        const int cidx = m_old + sm_opened;
        if (cidx >= C.m_max) {                                                   // capacity: the key is dropped from D
            __syncthreads();
            if (tid == 0) { dropped[j] = 1; sm_full = 1; }
            __syncthreads();
            continue;
        }
        // distances of all later keys to the new representative
        float xf[8];
        Elem<T>::unpack(reinterpret_cast<const uint4*>(keys + (size_t)j * D)[lr], xf);
        for (int ib = j + 1; ib < cl; ib += GPB) {
            const int i = ib + grp;
            unsigned long long acc = 0;
            if (i < cl) {
                float kf[8];
                Elem<T>::unpack(reinterpret_cast<const uint4*>(keys + (size_t)i * D)[lr], kf);
#pragma unroll
                for (int q = 0; q < 8; ++q) acc += fx_sqdiff(xf[q], kf[q]);
            }
#pragma unroll
            for (int off = 1; off < LPR; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (i < cl && lr == 0 && acc < new_d2[i]) { new_d2[i] = acc; new_idx[i] = cidx; }    // later ones have larger indices
        }
        __syncthreads();
        if (tid == 0) { is_open[j] = 1; opened_at[j] = cidx; sm_opened = sm_opened + 1; }
        __syncthreads();
    }
    __syncthreads();
    // assignment, counts, coins
    for (int j = tid; j < cl; j += kResolveThreads) {
        int c;
        if (is_open[j]) c = opened_at[j];
        else if (dropped[j]) c = -1;
        else if (new_d2[j] <= thr && (old_d2[j] > thr || new_d2[j] < old_d2[j])) c = new_idx[j];
        else c = old_idx[j];
        cid[j] = c;
    }
    __syncthreads();
    for (int j = tid; j < cl; j += kResolveThreads) {
        const int c = cid[j];
        int rank = 1;
        bool lat = false;
        for (int i = 0; i < cl; ++i) {
            if (i < j && cid[i] == c) ++rank;
            if (i > j && cid[i] == c) lat = true;
        }
        has_later[j] = lat;
        nnew[j] = c < 0 ? 0 : ((c < m_old ? cntu[c] : 0) + rank);
    }
    __syncthreads();
    const int nblk = (t + 3) >> 2;
    for (int p = tid; p < cl * nblk; p += kResolveThreads) {
        const int j = p / nblk, blk = p % nblk;
        if (cid[j] < 0) continue;
        const uint4 rr = philox4x32_10(make_uint4((uint32_t)(e0 + j), unit_id(C, u), (uint32_t)blk, 0u), C.key0, C.key1);
        const uint32_t words[4] = {rr.x, rr.y, rr.z, rr.w};
        unsigned long long bits = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (blk * 4 + q < t && coin_cluster(words[q], (uint32_t)nnew[j])) bits |= 1ull << (blk * 4 + q);
        if (bits) atomicOr(&succ[j], bits);
    }
    __syncthreads();
    for (int j = tid; j < cl; j += kResolveThreads) {
        unsigned long long lm = 0;
        for (int i = j + 1; i < cl; ++i) if (cid[i] == cid[j]) lm |= succ[i];
        later[j] = lm;
    }
    __syncthreads();
    // writes: a warp per key
    const unsigned long long tmask = t == 64 ? ~0ull : ((1ull << t) - 1ull);
    for (int j = warp; j < cl; j += kResolveThreads / 32) {
        const int c = cid[j];
        if (c < 0) continue;
        const int e = e0 + j;
        const uint4* src = reinterpret_cast<const uint4*>(keys + (size_t)j * D);
        const bool opened = is_open[j];
        if (opened) {
            if (lane < LPR) reinterpret_cast<uint4*>(Xu + (size_t)c * D)[lane] = src[lane];
            {   // packed head of the representative and its squared norm
                float hn = 0.f;
                if (lane < kHeadDims / 8) {
                    const uint4 r = src[lane];
                    reinterpret_cast<uint4*>(C.Xh + ((size_t)u * C.m_max + c) * kHeadDims)[lane] = r;
                    float f[8];
                    Elem<T>::unpack(r, f);
#pragma unroll
                    for (int q = 0; q < 8; ++q) hn = fmaf(f[q], f[q], hn);
                }
                hn += __shfl_xor_sync(0xffffffffu, hn, 1);
                hn += __shfl_xor_sync(0xffffffffu, hn, 2);
                if (lane == 0) C.xhn[(size_t)u * C.m_max + c] = hn;
            }
            if (!has_later[j])                                      // otherwise every slot gets its id from the key that wins it
                for (int q = lane; q < t; q += 32) stoku[(size_t)c * t + q] = e;
            if (lane == 0) { C.ctok[(size_t)u * C.m_max + c] = e; C.xn[(size_t)u * C.m_max + c] = kn[j]; }
        }
        const bool alone = opened && !has_later[j];                 // stays a singleton: its samples remain implied
        if (!alone) {
            unsigned long long wins = succ[j] & ~later[j] & tmask;
            while (wins) {
                const int q = __ffsll((long long)wins) - 1;
                wins &= wins - 1;
                if (lane < LPR) reinterpret_cast<uint4*>(Su + ((size_t)c * t + q) * D)[lane] = src[lane];
                if (lane == 0) stoku[(size_t)c * t + q] = e;
            }
            // first key of the chunk to join a cluster that was a singleton before the chunk: write out the
            // implied copies of the representative in the slots nobody in the chunk wins
            if (c < m_old && nnew[j] == 2) {
                unsigned long long fill = ~(succ[j] | later[j]) & tmask;
                const uint4* xr = reinterpret_cast<const uint4*>(Xu + (size_t)c * D);
                while (fill) {
                    const int q = __ffsll((long long)fill) - 1;
                    fill &= fill - 1;
                    if (lane < LPR) reinterpret_cast<uint4*>(Su + ((size_t)c * t + q) * D)[lane] = xr[lane];
                }
            }
        }
        if (!has_later[j] && lane == 0) cntu[c] = nnew[j];          // last key of its cluster in this chunk
    }
    __syncthreads();
    if (tid == 0) {
        C.pairs[u] += (unsigned long long)cl * (unsigned long long)m_old;
        C.m_unit[u] = m_old + sm_opened;
        a.mhist[2 * u + (chunk & 1)] = m_old + sm_opened;
        if (sm_full) atomicOr(&C.status[u], 1);
        const int j = cl - 1;
        if (e0 + j == r.ins_hi - 1) {                               // the most recent insertion of this unit
            C.last_cid[u] = cid[j];
            C.last_open[u] = is_open[j] || dropped[j];
            C.last_d2[u] = (new_d2[j] <= thr && (old_d2[j] > thr || new_d2[j] < old_d2[j])) ? new_d2[j] : old_d2[j];
        }
    }
}

// Window rows of the tokens that stay in the window, token count, mu. grid (blocks, U).
template <int D>
__global__ void prefill_finish_kernel(Cache<__nv_bfloat16> C, PrefillArgs a) {
    constexpr int LPR = D / 8;
    const int u = blockIdx.y, w = C.w;
    const Range r = unit_range(C, a, u);
    if (w) {
        const int lo = max(r.n_prev, r.n_tot - w);
        const int cnt = (r.n_tot - lo) * LPR;
        for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < cnt; p += gridDim.x * blockDim.x) {
            const int tok = lo + p / LPR, part = p % LPR;
            reinterpret_cast<uint4*>(C.ringK + ((size_t)u * w + tok % w) * D)[part] =
                reinterpret_cast<const uint4*>(a.K + (r.row0 + (tok - r.n_prev)) * D)[part];
            reinterpret_cast<uint4*>(C.ringV + ((size_t)u * w + tok % w) * D)[part] =
                reinterpret_cast<const uint4*>(a.V + (r.row0 + (tok - r.n_prev)) * D)[part];
        }
    }
}

// Last kernel of a prefill call: counters (after every block of every other kernel has read them).
// Both slots of mhist start as the cluster count before the call. One thread per unit.
__global__ void prefill_mhist_kernel(Cache<__nv_bfloat16> C, PrefillArgs a, int U) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u < U) { a.mhist[2 * u] = C.m_unit[u]; a.mhist[2 * u + 1] = C.m_unit[u]; }
}

// Alias rows of every cluster (see Cache::alias) from the slot tokens the chunks left. grid (blocks, U).
__global__ void prefill_alias_kernel(Cache<__nv_bfloat16> C) {
    const int u = blockIdx.y, m = C.m_unit[u], t = C.t;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < m; c += gridDim.x * blockDim.x) {
        const size_t cc = (size_t)u * C.m_max + c;
        C.ndist[cc] = (unsigned char)distinct_slots(C.stok + cc * t, t, C.alias + cc * t);
    }
}

__global__ void prefill_commit_kernel(Cache<__nv_bfloat16> C, PrefillArgs a, int U) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const Range r = unit_range(C, a, u);
    if (r.ins_hi > r.ins_lo) C.mu[u] = a.Tot[(size_t)u * a.Lmax + (r.ins_hi - r.ins_lo - 1)];
    C.n_unit[u] = r.n_tot;
}

}  // namespace sgk
