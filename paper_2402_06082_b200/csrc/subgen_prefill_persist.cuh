// Chunked prefill of the keys (UpdateSoftmaxNormalizer applied to a whole prompt) as ONE persistent kernel, d = 128.
//
// The launch-per-chunk path (score kernel + resolve kernel per chunk of 128 keys) spends most of its time between
// kernels when a unit has few representatives: every chunk is a dependency chain of two launches. A unit's chunks
// are sequential anyway and units share nothing, so here one thread block owns one unit and walks its chunks in a
// loop; nothing is launched, nothing is exchanged between blocks, nobody waits for another block. Per chunk:
//
//   stage     the 128 keys (full rows for the exact distances and the writes, 64-coordinate heads as operand A)
//   score     tiles of 128 representatives: D[key][representative] = <kh, xh> by tcgen05.mma (M = N = 128, K = 64),
//             two accumulators in tensor memory so that the MMAs of tile j+1 run under the read-back of tile j,
//             three staged tiles of heads; a pair whose head distance (a lower bound of D2) is inside the guard
//             band of delta^2 gets its exact fixed-point D2 from the full rows
//   resolve   openings in stream order, assignment, ranks, cluster coins, writes (the logic of
//             prefill_resolve_kernel, fed from shared memory instead of from a scratch array)
//
// Two blocks share an SM (about 108 KB of shared memory and 256 of the 512 tensor-memory columns each). The only
// waits are on this block's own MMA commits (mbarrier try_wait, bounded: on expiry the unit gets status bit 4, the
// block frees its tensor memory and returns).
#pragma once
#include "subgen_score_tc.cuh"

namespace sgk {

constexpr int kPpThreads = 256;
constexpr int kPpWarps = kPpThreads / 32;
constexpr int kPpCand = 1024;      // flagged (key, representative) pairs the list holds
constexpr int kPpFlush = 512;      // the list is worked off at the end of a tile once it holds this many

struct PpSmem {                                   // after a 1024-byte aligned base
    unsigned char A[128 * 128];                   // heads of the chunk keys, K-major, 128-byte swizzle
    unsigned char B[3][kTcTileN * 128];           // three tiles of representative heads, same layout
    __nv_bfloat16 keys[kChunk * 128];             // the chunk's full rows
    float kn_thr[kChunk];                         // 1/2 ((1-g) ||kh||^2 - delta^2) per key
    float kn_full[kChunk];                        // ||k||^2 per key
    float hx[kChunk];                             // 1/2 (1-g) ||kh||^2 per key (a key as a new representative)
    float xa[3][kTcTileN];                        // 1/2 (1-g) ||xh||^2 per representative of a staged tile (+inf: no row)
    unsigned long long old_d2[kChunk], new_d2[kChunk], succ[kChunk], later[kChunk];
    int old_idx[kChunk], new_idx[kChunk], cid[kChunk], nnew[kChunk], opened_at[kChunk];
    unsigned cand[kPpCand];                       // key | representative << 7
    unsigned char is_open[kChunk], has_later[kChunk], dropped[kChunk];
    unsigned long long mbar[2];
    unsigned long long sm_w[2];                   // bounded handles: {unused, ||k||^2 | ||k head||^2 << 32} of the key inserted on its own
    unsigned tmem_base, ncand, failed, far_mask[4]; // far_mask: keys with no old representative within delta
    int opened, full;
};
constexpr size_t kPpSmemBytes = sizeof(PpSmem) + 1024;

constexpr int kPpPhases = 8;   // staging, MMA wait, read-back, tile store + issue, exact follow-up | openings, ranks + coins, writes

// phase_ns: NULL, or [U][kPpPhases] SM cycles thread 0 of the unit's block spent in each phase (profiling).
// BND: the handle runs the bounded-m variant. A key that needs a cluster when the budget is used up ends its chunk
// early: the keys before it are resolved as a shorter chunk, the key itself is inserted on its own (threshold
// doubling and merge sweep, make_room), and the walk resumes behind it under the new threshold and cluster numbering.
template <bool BND>
__global__ void __launch_bounds__(kPpThreads, 2) prefill_keys_persist_kernel(Cache<__nv_bfloat16> C, PrefillArgs a,
                                                                            unsigned long long* phase_ns) {
    typedef __nv_bfloat16 T;
    constexpr int D = 128, LPR = 16;
    extern __shared__ unsigned char dyn_raw[];
    PpSmem& sm = *reinterpret_cast<PpSmem*>((reinterpret_cast<uintptr_t>(dyn_raw) + 1023) & ~(uintptr_t)1023);
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Range r = unit_range(C, a, u);
    const int len = r.ins_hi - r.ins_lo;
    if (len <= 0) return;
    const int t = C.t;
    unsigned long long thr = BND ? C.thr2[u] : C.delta2_fx;       // bounded handles: the threshold in force
    T* Xu = C.X + (size_t)u * C.m_max * D;
    T* Su = C.S + (size_t)u * C.m_max * t * D;
    int* cntu = C.cnt + (size_t)u * C.m_max;
    int* stoku = C.stok + (size_t)u * C.m_max * t;
    float d2f = (float)((double)thr * (1.0 / 4294967296.0));
    constexpr float kOneMinusG = 1.f - 1.220703125e-4f;
    const uint32_t sA = (uint32_t)__cvta_generic_to_shared(sm.A);
    const uint32_t sB = (uint32_t)__cvta_generic_to_shared(sm.B[0]);
    const uint32_t sBar0 = (uint32_t)__cvta_generic_to_shared(&sm.mbar[0]);

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(&sm.tmem_base)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sBar0) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sBar0 + 8u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        sm.ncand = 0;
        sm.failed = 0;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm.tmem_base;
    int m = C.m_unit[u];
    unsigned uses[2] = {0u, 0u};                  // completed waits per barrier (its phase parity)
    unsigned long long pairs = 0, cyc[kPpPhases] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long tick = 0;
    const bool timing = phase_ns != nullptr && tid == 0;
    auto lap = [&](int ph) { if (timing) { const long long now = clock64(); cyc[ph] += (unsigned long long)(now - tick); tick = now; } };
    bool ok = true;
    const int tok_row = (warp & 3) * 32 + lane;   // the accumulator row (key of the chunk) this thread reads back
    const int col_half = warp >> 2;               // ... and which 64 of its 128 columns

    // representative heads of tile j: global -> registers (tile_fetch), registers -> B[buf], xa[buf] (tile_store).
    // Representatives are written by this very block (earlier chunks), so they are read past L1.
    constexpr int kPer = kTcTileN * kTcHeadPieces / kPpThreads;       // 16-byte pieces per thread and tile
    uint4 R[kPer];
    auto tile_fetch = [&](int j, int limit) {
        const int row0 = j * kTcTileN;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int p = i * kPpThreads + tid, rr = p / kTcHeadPieces, q = p % kTcHeadPieces;
            R[i] = make_uint4(0, 0, 0, 0);
            if (row0 + rr < limit) R[i] = __ldcg(reinterpret_cast<const uint4*>(Xu + (size_t)(row0 + rr) * D + q * 8));
        }
    };
    auto tile_store = [&](int buf, int j, int limit) {
        unsigned char* dst = sm.B[buf];
        const int row0 = j * kTcTileN;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int p = i * kPpThreads + tid, rr = p / kTcHeadPieces, q = p % kTcHeadPieces;
            *reinterpret_cast<uint4*>(dst + sw128_offset(rr, q)) = R[i];
            float f[8], hn = 0.f;
            Elem<T>::unpack(R[i], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) hn = fmaf(f[e], f[e], hn);
            hn += __shfl_xor_sync(0xffffffffu, hn, 1);
            hn += __shfl_xor_sync(0xffffffffu, hn, 2);
            hn += __shfl_xor_sync(0xffffffffu, hn, 4);
            if (q == 0) sm.xa[buf][rr] = row0 + rr < limit ? 0.5f * kOneMinusG * hn : INFINITY;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores -> visible to the MMA
    };
    auto issue_mma = [&](int buf, int acc) {                           // one thread: 4 MMAs of K = 16, then commit
        const uint32_t sBb = buf < 0 ? sA : sB + (uint32_t)buf * (uint32_t)(kTcTileN * 128);   // buf < 0: the chunk against itself
        const uint32_t dcol = tmem + (uint32_t)acc * 128u;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const uint32_t off = (uint32_t)(ks * 32);
            const uint64_t da = umma_desc_sw128(sA + off), db = umma_desc_sw128(sBb + off);
            const uint32_t accum = ks ? 1u : 0u;
            asm volatile(
                "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                ::"r"(dcol), "l"(da), "l"(db), "r"(kTcIdesc), "r"(accum), "r"(0u) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(sBar0 + 8u * (uint32_t)acc) : "memory");
    };
    const uint4* keys4 = reinterpret_cast<const uint4*>(sm.keys);

    for (int pos = 0; pos < len && ok;) {
        const int e0 = r.ins_lo + pos, cl = min(kChunk, r.ins_hi - e0);
        if (timing) tick = clock64();
        // ---- stage the chunk: full rows, heads as operand A (rows beyond cl are zero), per-key bookkeeping ----
        for (int p = tid; p < kChunk * LPR; p += kPpThreads) {
            const int j = p / LPR, part = p % LPR;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (j < cl) v = reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e0 + j))[part];
            reinterpret_cast<uint4*>(sm.keys)[p] = v;
            if (part < kTcHeadPieces) *reinterpret_cast<uint4*>(sm.A + sw128_offset(j, part)) = v;
        }
        if (tid < kChunk) {
            sm.old_d2[tid] = ~0ull; sm.old_idx[tid] = INT_MAX;
            sm.new_d2[tid] = ~0ull; sm.new_idx[tid] = INT_MAX;
            sm.succ[tid] = 0ull; sm.is_open[tid] = 0; sm.dropped[tid] = 0; sm.opened_at[tid] = -1;
        }
        if (tid == 0) { sm.opened = 0; sm.full = 0; sm.ncand = 0; }
        // the next chunk's rows are wanted in about one chunk's time: ask for them now (one 128-byte line per thread)
        {
            const int j = tid >> 1, en = e0 + kChunk + j;
            if (en < r.ins_hi) {
                const char* nx = reinterpret_cast<const char*>(key_row<D>(C, a, r, u, en)) + (tid & 1) * 128;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nx));
            }
        }
        __syncthreads();
        if (tid < kChunk) {                                            // squared norms of this key: head and full row
            float head = 0.f, acc = 0.f;
            for (int p = 0; p < LPR; ++p) {
                float f[8];
                Elem<T>::unpack(keys4[tid * LPR + p], f);
#pragma unroll
                for (int q = 0; q < 8; ++q) acc = fmaf(f[q], f[q], acc);
                if (p == kTcHeadPieces - 1) head = acc;
            }
            sm.kn_full[tid] = acc;
            sm.kn_thr[tid] = 0.5f * (kOneMinusG * head - d2f);
            sm.hx[tid] = 0.5f * kOneMinusG * head;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the stores of A -> visible to the MMA

        // ---- score: tiles of 128 representatives, then the chunk against itself (the "Gram" tile, B = A) ----
        // Tile k < JT: heads of representatives [128 k, 128 k + 128); tile JT: the chunk's own heads, whose products
        // stay in tensor memory for the opening loop below. Tile k uses accumulator k & 1 and is issued as soon as
        // tile k - 2 has been read back.
        const int JT = (m + kTcTileN - 1) / kTcTileN, NT = JT + 1;
        if (JT > 0) {
            tile_fetch(0, m);
            tile_store(0, 0, m);
            if (JT > 1) { tile_fetch(1, m); tile_store(1, 1, m); }
            if (JT > 2) tile_fetch(2, m);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        const float my_kn = sm.kn_thr[tok_row];
        lap(0);
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue_mma(0 < JT ? 0 : -1, 0);
            if (NT > 1) issue_mma(1 < JT ? 1 : -1, 1);
        }
        // exact D2 of the listed pairs [0, cnt): warp w owns the keys with index % 8 == w. Called by all threads.
        auto flush_list = [&](unsigned cnt) {
            for (unsigned base = 0; base < cnt; base += 32) {
                const bool have = base + lane < cnt;
                const unsigned cd = have ? sm.cand[base + lane] : 0u;
                unsigned mine = __ballot_sync(0xffffffffu, have && (cd & 7u) == (unsigned)warp);
                while (mine) {                                         // four pairs per turn, two per half-warp
                    int sel[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        sel[x] = mine ? __ffs(mine) - 1 : -1;
                        if (mine) mine &= mine - 1;
                    }
                    const int half = lane >> 4, l16 = lane & 15;
                    unsigned long long d2acc[2];
                    unsigned cdv[2];
                    uint4 xr[2], kr[2];
#pragma unroll
                    for (int y = 0; y < 2; ++y) {
                        const int sidx = sel[2 * y + half];
                        cdv[y] = __shfl_sync(0xffffffffu, cd, sidx < 0 ? 0 : sidx);
                        if (sidx >= 0) {
                            xr[y] = __ldcg(reinterpret_cast<const uint4*>(Xu + (size_t)(cdv[y] >> 7) * D + l16 * 8));
                            kr[y] = keys4[(int)(cdv[y] & 127u) * LPR + l16];
                        } else {
                            xr[y] = make_uint4(0, 0, 0, 0);
                            kr[y] = make_uint4(0, 0, 0, 0);
                        }
                    }
#pragma unroll
                    for (int y = 0; y < 2; ++y) {
                        float xf[8], kf[8];
                        Elem<T>::unpack(xr[y], xf);
                        Elem<T>::unpack(kr[y], kf);
                        d2acc[y] = 0;
#pragma unroll
                        for (int e = 0; e < 8; ++e) d2acc[y] += fx_sqdiff(xf[e], kf[e]);
#pragma unroll
                        for (int off = 8; off > 0; off >>= 1) d2acc[y] += __shfl_xor_sync(0xffffffffu, d2acc[y], off);
                    }
#pragma unroll
                    for (int x = 0; x < 4; ++x) {                      // lane 0 applies them in turn: they may share a key
                        const int y = x >> 1, hsrc = (x & 1) * 16;
                        const unsigned long long d2 = __shfl_sync(0xffffffffu, d2acc[y], hsrc);
                        const unsigned cdx = __shfl_sync(0xffffffffu, cdv[y], hsrc);
                        if (lane == 0 && sel[x] >= 0) {
                            const int tokj = (int)(cdx & 127u), row = (int)(cdx >> 7);
                            Best cur;
                            cur.d2 = sm.old_d2[tokj]; cur.idx = sm.old_idx[tokj];
                            if (better(d2, row, cur)) { sm.old_d2[tokj] = d2; sm.old_idx[tokj] = row; }
                        }
                    }
                }
            }
        };
        for (int j = 0; j < NT; ++j) {
            const int acc = j & 1;
            {   // wait for the MMAs of this tile (bounded)
                const uint32_t parity = uses[acc] & 1u;
                unsigned fin = 0, spins = 0;
                while (!fin && spins < kTcSpinLimit) {
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                                 : "=r"(fin) : "r"(sBar0 + 8u * (uint32_t)acc), "r"(parity) : "memory");
                    ++spins;
                }
                if (!fin) sm.failed = 1;
                uses[acc] += 1u;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            lap(1);
            if (j == JT) break;                                        // the Gram tile stays in tensor memory
            // read-back: this thread's key row, its 64 columns of the accumulator, both loads before one wait;
            // the 64 threshold tests make a bit mask first (no memory operation between them), pushes come after
            bool crossed = false;
            {
                uint32_t v[64];
                const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(acc * 128 + col_half * 64);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t* w = v + hh * 32;
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                        : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]), "=r"(w[8]),
                          "=r"(w[9]), "=r"(w[10]), "=r"(w[11]), "=r"(w[12]), "=r"(w[13]), "=r"(w[14]), "=r"(w[15]), "=r"(w[16]),
                          "=r"(w[17]), "=r"(w[18]), "=r"(w[19]), "=r"(w[20]), "=r"(w[21]), "=r"(w[22]), "=r"(w[23]), "=r"(w[24]),
                          "=r"(w[25]), "=r"(w[26]), "=r"(w[27]), "=r"(w[28]), "=r"(w[29]), "=r"(w[30]), "=r"(w[31])
                        : "r"(taddr + (uint32_t)(hh * 32)) : "memory");
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const float4* xat4 = reinterpret_cast<const float4*>(sm.xa[j % 3] + col_half * 64);
                unsigned long long mask = 0;
#pragma unroll
                for (int q4 = 0; q4 < 16; ++q4) {
                    const float4 x = xat4[q4];
                    mask |= (unsigned long long)(__uint_as_float(v[4 * q4 + 0]) >= x.x + my_kn) << (4 * q4 + 0);
                    mask |= (unsigned long long)(__uint_as_float(v[4 * q4 + 1]) >= x.y + my_kn) << (4 * q4 + 1);
                    mask |= (unsigned long long)(__uint_as_float(v[4 * q4 + 2]) >= x.z + my_kn) << (4 * q4 + 2);
                    mask |= (unsigned long long)(__uint_as_float(v[4 * q4 + 3]) >= x.w + my_kn) << (4 * q4 + 3);
                }
                if (tok_row >= cl) mask = 0;
                while (mask) {                                         // rare
                    const int q = __ffsll((long long)mask) - 1;
                    mask &= mask - 1;
                    const unsigned slot = atomicAdd(&sm.ncand, 1u);
                    if (slot < (unsigned)kPpCand) sm.cand[slot] = (unsigned)tok_row | ((unsigned)(j * kTcTileN + col_half * 64 + q) << 7);
                    crossed |= slot >= (unsigned)kPpFlush;
                }
            }
            lap(2);
            // tile j+2 goes into the buffer tile j-1 used (its MMAs ended before the previous read-back)
            if (j + 2 < JT) tile_store((j + 2) % 3, j + 2, m);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            const int over = __syncthreads_or(crossed);                // uniform: the list is at least half full
            if (sm.failed) { ok = false; break; }
            if (j + 2 < NT && tid == 0) {                              // this accumulator is free again
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_mma(j + 2 < JT ? (j + 2) % 3 : -1, acc);
            }
            if (j + 3 < JT) tile_fetch(j + 3, m);
            lap(3);
            if (over) {
                // At most kPpFlush pairs were listed before this tile, so only this tile can have overrun the list:
                // then every pair of the tile is evaluated.
                const unsigned nc = sm.ncand;
                flush_list(nc < (unsigned)kPpCand ? nc : (unsigned)kPpCand);
                if (nc > (unsigned)kPpCand) {
                    const int row0 = j * kTcTileN, nrow = min(kTcTileN, m - row0);
                    for (int tokj = warp; tokj < cl; tokj += kPpWarps)
                        for (int rr = 0; rr < nrow; ++rr) {
                            unsigned long long dd = 0;
                            if (lane < LPR) {
                                float xf[8], kf[8];
                                Elem<T>::unpack(__ldcg(reinterpret_cast<const uint4*>(Xu + (size_t)(row0 + rr) * D + lane * 8)), xf);
                                Elem<T>::unpack(keys4[tokj * LPR + lane], kf);
#pragma unroll
                                for (int e = 0; e < 8; ++e) dd += fx_sqdiff(xf[e], kf[e]);
                            }
#pragma unroll
                            for (int off = 16; off > 0; off >>= 1) dd += __shfl_xor_sync(0xffffffffu, dd, off);
                            if (lane == 0) {
                                Best cur;
                                cur.d2 = sm.old_d2[tokj]; cur.idx = sm.old_idx[tokj];
                                if (better(dd, row0 + rr, cur)) { sm.old_d2[tokj] = dd; sm.old_idx[tokj] = row0 + rr; }
                            }
                        }
                }
                __syncthreads();
                if (tid == 0) sm.ncand = 0;
                __syncthreads();
                lap(4);
            }
        }
        if (!ok) break;
        flush_list(sm.ncand);                                          // nobody pushes any more: the count is final
        __syncthreads();
        lap(4);

        // ---- resolve: openings in stream order, assignment, ranks, coins, writes ----
        const int m_old = m;
        // Only a key with no old representative within delta can open one; it does iff no representative opened
        // earlier in this chunk is within delta either. For a new representative j the later keys that may be within
        // delta of it are read off column j of the Gram tile (same lower bound and guard band as for the old
        // representatives); those pairs get their exact D2 from the rows in shared memory.
        if (col_half == 0) {
            const unsigned fm = __ballot_sync(0xffffffffu, tok_row < cl && sm.old_d2[tok_row] > thr);
            if (lane == 0) sm.far_mask[warp] = fm;
        }
        __syncthreads();
        int n_open = 0, stop = -1;                                     // stop: the key that found the budget used up (BND)
        const uint32_t gaddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((JT & 1) * 128);
        for (int wd = 0; wd < 4 && stop < 0; ++wd) {
            unsigned fm = sm.far_mask[wd];                             // uniform
            while (fm) {
                const int j = wd * 32 + __ffs(fm) - 1;
                fm &= fm - 1;
                if (!(sm.new_d2[j] > thr)) continue;                   // uniform: written before the last barrier
                const int cidx = m_old + n_open;
                if (cidx >= C.m_max) {
                    if (BND) { stop = j; break; }                      // the chunk ends before this key
                    if (tid == 0) { sm.dropped[j] = 1; sm.full = 1; }  // capacity: the key is dropped from D
                    continue;
                }
                if (col_half == 0) {
                    uint32_t gv;
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n" : "=r"(gv) : "r"(gaddr + (uint32_t)j) : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int i = tok_row;
                    const bool flag = i > j && i < cl && __uint_as_float(gv) >= sm.kn_thr[i] + sm.hx[j];
                    unsigned msk = __ballot_sync(0xffffffffu, flag);
                    const int half = lane >> 4, l16 = lane & 15;
                    while (msk) {                                      // two flagged keys per turn, one per half-warp
                        const int la = __ffs(msk) - 1;
                        msk &= msk - 1;
                        int lb = -1;
                        if (msk) { lb = __ffs(msk) - 1; msk &= msk - 1; }
                        const int li = half ? lb : la;
                        unsigned long long dd = 0;
                        if (li >= 0) {
                            float xf[8], kf[8];
                            Elem<T>::unpack(keys4[j * LPR + l16], xf);
                            Elem<T>::unpack(keys4[((warp & 3) * 32 + li) * LPR + l16], kf);
#pragma unroll
                            for (int q = 0; q < 8; ++q) dd += fx_sqdiff(xf[q], kf[q]);
                        }
#pragma unroll
                        for (int off = 8; off > 0; off >>= 1) dd += __shfl_xor_sync(0xffffffffu, dd, off);
                        if (l16 == 0 && li >= 0) {
                            const int i2 = (warp & 3) * 32 + li;
                            if (dd < sm.new_d2[i2]) { sm.new_d2[i2] = dd; sm.new_idx[i2] = cidx; }   // later ones have larger indices
                        }
                    }
                }
                if (tid == 0) { sm.is_open[j] = 1; sm.opened_at[j] = cidx; }
                ++n_open;
                __syncthreads();
            }
        }
        if (tid == 0) sm.opened = n_open;
        const int ce = stop >= 0 ? stop : cl;                          // keys resolved in this turn
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        lap(5);
        if (tid < ce) {
            const int j = tid;
            int c;
            if (sm.is_open[j]) c = sm.opened_at[j];
            else if (sm.dropped[j]) c = -1;
            else if (sm.new_d2[j] <= thr && (sm.old_d2[j] > thr || sm.new_d2[j] < sm.old_d2[j])) c = sm.new_idx[j];
            else c = sm.old_idx[j];
            sm.cid[j] = c;
        }
        __syncthreads();
        if (tid < ce) {
            const int j = tid, c = sm.cid[j];
            int rank = 1;
            bool lat = false;
            for (int i = 0; i < ce; ++i) {
                if (i < j && sm.cid[i] == c) ++rank;
                if (i > j && sm.cid[i] == c) lat = true;
            }
            sm.has_later[j] = lat;
            sm.nnew[j] = c < 0 ? 0 : ((c < m_old ? __ldcg(cntu + c) : 0) + rank);
        }
        __syncthreads();
        const int nblk = (t + 3) >> 2;
        for (int p = tid; p < ce * nblk; p += kPpThreads) {
            const int j = p / nblk, blk = p % nblk;
            if (sm.cid[j] < 0) continue;
            const uint4 rr = philox4x32_10(make_uint4((uint32_t)(e0 + j), unit_id(C, u), (uint32_t)blk, 0u), C.key0, C.key1);
            const uint32_t words[4] = {rr.x, rr.y, rr.z, rr.w};
            unsigned long long bits = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (blk * 4 + q < t && coin_cluster(words[q], (uint32_t)sm.nnew[j])) bits |= 1ull << (blk * 4 + q);
            if (bits) atomicOr(&sm.succ[j], bits);
        }
        __syncthreads();
        if (tid < ce) {
            const int j = tid;
            unsigned long long lm = 0;
            for (int i = j + 1; i < ce; ++i) if (sm.cid[i] == sm.cid[j]) lm |= sm.succ[i];
            sm.later[j] = lm;
        }
        __syncthreads();
        lap(6);
        const unsigned long long tmask = t == 64 ? ~0ull : ((1ull << t) - 1ull);
        for (int j = warp; j < ce; j += kPpWarps) {                    // writes: a warp per key
            const int c = sm.cid[j];
            if (c < 0) continue;
            const int e = e0 + j;
            const uint4* src = keys4 + j * LPR;
            const bool opened = sm.is_open[j];
            if (opened) {
                if (lane < LPR) reinterpret_cast<uint4*>(Xu + (size_t)c * D)[lane] = src[lane];
                float hn = 0.f;                                        // packed head of the representative and its norm
                if (lane < kHeadDims / 8) {
                    const uint4 hr = src[lane];
                    reinterpret_cast<uint4*>(C.Xh + ((size_t)u * C.m_max + c) * kHeadDims)[lane] = hr;
                    float f[8];
                    Elem<T>::unpack(hr, f);
#pragma unroll
                    for (int q = 0; q < 8; ++q) hn = fmaf(f[q], f[q], hn);
                }
                hn += __shfl_xor_sync(0xffffffffu, hn, 1);
                hn += __shfl_xor_sync(0xffffffffu, hn, 2);
                if (lane == 0) C.xhn[(size_t)u * C.m_max + c] = hn;
                if (!sm.has_later[j])                                  // otherwise every slot gets its id from the key that wins it
                    for (int q = lane; q < t; q += 32) stoku[(size_t)c * t + q] = e;
                if (lane == 0) { C.ctok[(size_t)u * C.m_max + c] = e; C.xn[(size_t)u * C.m_max + c] = sm.kn_full[j]; }
            }
            const bool alone = opened && !sm.has_later[j];             // stays a singleton: its samples remain implied
            if (!alone) {
                unsigned long long wins = sm.succ[j] & ~sm.later[j] & tmask;
                while (wins) {
                    const int q = __ffsll((long long)wins) - 1;
                    wins &= wins - 1;
                    if (lane < LPR) reinterpret_cast<uint4*>(Su + ((size_t)c * t + q) * D)[lane] = src[lane];
                    if (lane == 0) stoku[(size_t)c * t + q] = e;
                }
                // first key of the chunk to join a cluster that was a singleton before the chunk: write out the
                // implied copies of the representative in the slots nobody in the chunk wins
                if (c < m_old && sm.nnew[j] == 2) {
                    unsigned long long fill = ~(sm.succ[j] | sm.later[j]) & tmask;
                    const uint4* xr = reinterpret_cast<const uint4*>(Xu + (size_t)c * D);
                    uint4 xv = make_uint4(0, 0, 0, 0);
                    if (lane < LPR) xv = __ldcg(xr + lane);
                    while (fill) {
                        const int q = __ffsll((long long)fill) - 1;
                        fill &= fill - 1;
                        if (lane < LPR) reinterpret_cast<uint4*>(Su + ((size_t)c * t + q) * D)[lane] = xv;
                    }
                }
            }
            if (!sm.has_later[j] && lane == 0) cntu[c] = sm.nnew[j];   // last key of its cluster in this chunk
        }
        __syncthreads();                                               // the writes above are read by the next chunk
        pairs += (unsigned long long)ce * (unsigned long long)m_old;
        m = m_old + sm.opened;
        const bool last_turn = stop < 0 && pos + ce == len;
        if (tid == 0) {
            if (sm.full) atomicOr(&C.status[u], 1);
            if (last_turn && ce > 0) {                                 // the most recent insertion of this unit
                const int j = ce - 1;
                C.last_cid[u] = sm.cid[j];
                C.last_open[u] = sm.is_open[j] || sm.dropped[j];
                C.last_d2[u] = (sm.new_d2[j] <= thr && (sm.old_d2[j] > thr || sm.new_d2[j] < sm.old_d2[j])) ? sm.new_d2[j] : sm.old_d2[j];
            }
        }
        __syncthreads();                                               // sm.opened is reset by the next chunk's staging
        lap(7);
        pos += ce;
        if constexpr (BND) {
            if (stop >= 0) {
                // The key at `stop` is farther than the threshold from every representative and no cluster is free:
                // the cluster half of its insertion on its own (make_room doubles the threshold and sweeps, then the
                // key joins or opens under the new threshold).
                const int e = e0 + stop;
                if (tid == 0) {
                    float kh = 0.f;
                    for (int p = 0; p < kHeadDims / 8; ++p) {
                        float f[8];
                        Elem<T>::unpack(keys4[stop * LPR + p], f);
#pragma unroll
                        for (int q = 0; q < 8; ++q) kh = fmaf(f[q], f[q], kh);
                    }
                    sm.sm_w[0] = 0ull;
                    sm.sm_w[1] = (unsigned long long)__float_as_uint(sm.kn_full[stop]) | ((unsigned long long)__float_as_uint(kh) << 32);
                }
                __syncthreads();
                Best far;
                far.d2 = ~0ull; far.idx = INT_MAX; far.pad = 0;
                bool joined, full;
                int m_ref = m;
                const int m_new = apply_cluster<T, D, true>(C, u, e, far, m_ref, keys4 + stop * LPR, sm.sm_w, joined, full);
                __syncthreads();
                if (tid == 0 && pos + 1 == len) {
                    C.last_cid[u] = joined ? far.idx : (full ? -1 : m_ref);
                    C.last_open[u] = joined ? 0 : 1;
                    C.last_d2[u] = far.d2;
                }
                m = m_new;
                thr = C.thr2[u];
                d2f = (float)((double)thr * (1.0 / 4294967296.0));
                pos += 1;
                __syncthreads();
            }
        }
    }
    if (tid == 0) {
        if (ok) {
            C.pairs[u] += pairs;
            C.m_unit[u] = m;
        } else {
            atomicOr(&C.status[u], 4);
        }
        if (phase_ns)
            for (int i = 0; i < kPpPhases; ++i) phase_ns[kPpPhases * u + i] = cyc[i];
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
}

}  // namespace sgk
