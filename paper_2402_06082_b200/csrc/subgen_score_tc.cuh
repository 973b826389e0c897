// Prefill score kernel on the 5th-generation tensor cores (tcgen05), d = 128.
//
// One chunk of 128 keys (A, M = 128) against tiles of 128 representatives (B, N = 128): D[token][centre] =
// <kh, xh> over the first 64 coordinates (the "head") by tcgen05.mma.cta_group::1.kind::f16 (bf16 x bf16 ->
// fp32), K = 64 in four K = 16 steps, the accumulator in 128 columns of tensor memory. Four blocks share an SM
// (54 KB of shared memory and a quarter of the tensor memory each), so one block's MMAs, read-back and exact
// follow-up overlap the others'; within a block the MMAs of tile j+1 are issued as soon as tile j has been
// read back and run during its exact follow-up. Operands sit in shared memory in the K-major 128-byte-swizzle
// layout the MMA descriptors describe: 8-row groups of 128-byte rows (1024 bytes per group, 16-byte pieces
// XOR-ed with the row index inside the group); only the heads are staged, the exact distances read full rows
// from global memory. The tiles are gathered with
// ordinary 16-byte loads and stored straight into that layout (the rows of a unit are contiguous but the chunk
// may come from the window ring, so no tensor map is involved), followed by a proxy fence before the MMA reads
// them.
//
// The MMA result is only a filter. D2 is a sum of non-negative terms, so the head distance bounds it from
// below: a pair is flagged when <kh,xh> >= 1/2[(1-g)(||xh||^2+||kh||^2) - delta^2] (the guard band of the insert
// kernel rearranged), and every flagged pair gets its exact fixed-point D2 over all coordinates.
// Each thread owns one token row of the accumulator (tensor-memory lane = row) and scans its 128 columns.
//
// Waits: the only wait is on the mbarrier that the MMA commit arrives on; it is bounded, and when the bound is
// hit the block sets the unit's status bit 4, frees its tensor memory and returns.
#pragma once
#include "subgen_prefill.cuh"

namespace sgk {

constexpr int kTcThreads = 128;
constexpr int kTcTileN = 128;
constexpr int kTcHeadPieces = 8;                 // 16-byte pieces of a row that make up the 64-coordinate head
constexpr int kTcCand = 512;                     // flagged pairs kept per tile before the exhaustive fallback
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kTcTileN >> 3) << 17) | ((128u >> 4) << 24);
constexpr unsigned kTcSpinLimit = 1u << 22;

struct TcSmem {                                  // after a 1024-byte aligned base
    unsigned char A[128 * 128];                  // heads of the chunk keys: [row][128 B swizzled]
    unsigned char B[2][kTcTileN * 128];          // two buffers of representative heads, same layout
    float kn[kChunk];                            // 1/2 ((1-g) ||kh||^2 - delta^2) per token
    float xa[2][kTcTileN];                       // 1/2 (1-g) ||xh||^2 per representative of the tile (+inf: no row)
    unsigned long long wb_d2[kChunk];            // best exact (D2, index) per token; token j belongs to warp j % 4
    int wb_idx[kChunk];
    unsigned cand[kTcCand];                      // token | row_in_tile << 8
    unsigned long long mbar;
    unsigned tmem_base, ncand, failed;
};
constexpr size_t kTcSmemBytes = sizeof(TcSmem) + 1024;

__device__ __forceinline__ uint32_t sw128_offset(int row, int piece16) {      // piece16: 0..7 over the 128-byte head
    return (uint32_t)(row * 128 + (((piece16 & 7) ^ (row & 7)) << 4));
}
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    // start address >> 4 | LBO = 1 (16 B) << 16 | SBO = 1024 B >> 4 << 32 | version 1 << 46 | layout SWIZZLE_128B (2) << 61
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__global__ void __launch_bounds__(kTcThreads, 4) prefill_score_tc_kernel(Cache<__nv_bfloat16> C, PrefillArgs a, int chunk) {
    typedef __nv_bfloat16 T;
    constexpr int D = 128, LPR = 16;
    extern __shared__ unsigned char dyn_raw[];
    TcSmem& sm = *reinterpret_cast<TcSmem*>((reinterpret_cast<uintptr_t>(dyn_raw) + 1023) & ~(uintptr_t)1023);
    const int u = blockIdx.y, slices = gridDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Range r = unit_range(C, a, u);
    const int e0 = r.ins_lo + chunk * kChunk, cl = min(kChunk, r.ins_hi - e0);
    if (cl <= 0) return;
    const T* Xu = C.X + (size_t)u * C.m_max * D;
    const float d2f = (float)((double)C.delta2_fx * (1.0 / 4294967296.0));
    constexpr float kOneMinusG = 1.f - 1.220703125e-4f;
    const uint32_t sA = (uint32_t)__cvta_generic_to_shared(sm.A);
    const uint32_t sB0 = (uint32_t)__cvta_generic_to_shared(sm.B[0]), sB1 = (uint32_t)__cvta_generic_to_shared(sm.B[1]);
    const uint32_t sBar = (uint32_t)__cvta_generic_to_shared(&sm.mbar);

    // ---- set-up: tensor memory (128 columns), the barrier, the chunk ----
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(&sm.tmem_base)), "r"(128u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sBar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        sm.ncand = 0;
        sm.failed = 0;
    }
    for (int p = tid; p < kChunk * kTcHeadPieces; p += kTcThreads) {   // heads of the chunk keys -> A (rows beyond cl are zero)
        const int j = p / kTcHeadPieces, q = p % kTcHeadPieces;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < cl) v = reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e0 + j))[q];
        *reinterpret_cast<uint4*>(sm.A + sw128_offset(j, q)) = v;
    }
    for (int j = tid; j < kChunk; j += kTcThreads) { sm.wb_d2[j] = ~0ull; sm.wb_idx[j] = INT_MAX; }
    __syncthreads();
    {
        const int j = tid;                                             // one token per thread
        float acc = 0.f;
        for (int q = 0; q < kTcHeadPieces; ++q) {
            float f[8];
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(sm.A + sw128_offset(j, q)), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc = fmaf(f[e], f[e], acc);
        }
        sm.kn[j] = 0.5f * (kOneMinusG * acc - d2f);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the stores of A -> visible to the MMA
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm.tmem_base;
    const float my_kn = sm.kn[tid];
    // Everything above touches only the chunk's keys. Tiles of 128 representatives are dealt to the blocks of the
    // unit round-robin. The resolve kernel of the previous chunk may still be running: it appends representatives
    // and never touches those that exist, so the tiles that lay entirely below the count the chunk before it left
    // (m_safe, read from L2) are scored at once; then the kernel waits for its predecessor and scores the rest with
    // the final count. Who wrote m_safe: for chunk c >= 2 the resolve kernel of chunk c - 2, which had completed
    // before the score kernel of chunk c - 1 passed its own wait, and this kernel is scheduled only after every
    // block of the resolve kernel of chunk c - 1 has passed its wait, which is later still. For chunk 1 the writer
    // is the history-initialisation kernel, three launches back and complete for the same reason. For chunk 0 that
    // kernel is the immediate predecessor, so chunk 0 is launched the ordinary way (the host does that), which makes
    // everything earlier in the stream complete before this kernel starts.
    Best* outp = a.pbest + ((size_t)u * slices + blockIdx.x) * kChunk;
    const int m_safe = __ldcg(a.mhist + 2 * u + (chunk & 1));        // count after chunk - 2
    const int JA = m_safe / kTcTileN;                                  // tiles [0, JA) are final

    // representative heads of tile j: global -> registers (tile_fetch), registers -> B[buf], xa[buf] (tile_store)
    constexpr int kPer = kTcTileN * kTcHeadPieces / kTcThreads;      // pieces per thread and tile
    uint4 R[kPer];
    auto tile_fetch = [&](int j, int limit) {
        const int row0 = j * kTcTileN;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int p = i * kTcThreads + tid, rr = p / kTcHeadPieces, q = p % kTcHeadPieces;
            R[i] = make_uint4(0, 0, 0, 0);
            if (row0 + rr < limit) R[i] = ldg16(Xu + (size_t)(row0 + rr) * D + q * 8);
        }
    };
    auto tile_store = [&](int buf, int j, int limit) {
        unsigned char* dst = sm.B[buf];
        const int row0 = j * kTcTileN;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int p = i * kTcThreads + tid, rr = p / kTcHeadPieces, q = p % kTcHeadPieces;
            *reinterpret_cast<uint4*>(dst + sw128_offset(rr, q)) = R[i];
            // squared norm of the head: the eight lanes that hold the row's pieces add up
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
    auto issue_mma = [&](int buf) {                                    // one thread: 4 MMAs of K = 16, then commit
        const uint32_t sBb = buf ? sB1 : sB0;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const uint32_t off = (uint32_t)(ks * 32);
            const uint64_t da = umma_desc_sw128(sA + off), db = umma_desc_sw128(sBb + off);
            const uint32_t accum = ks ? 1u : 0u;
            asm volatile(
                "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                ::"r"(tmem), "l"(da), "l"(db), "r"(kTcIdesc), "r"(accum), "r"(0u) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(sBar) : "memory");
    };
    // exact D2 of (token tokj, representative row), by one warp; only warp tokj % 4 ever handles token tokj
    auto exact_pair = [&](int tokj, int row) {
        unsigned long long acc = 0;
        if (lane < LPR) {
            float xf[8], kf[8];
            Elem<T>::unpack(*reinterpret_cast<const uint4*>(Xu + (size_t)row * D + lane * 8), xf);
            Elem<T>::unpack(reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e0 + tokj))[lane], kf);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc += fx_sqdiff(xf[e], kf[e]);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) {
            Best cur;
            cur.d2 = sm.wb_d2[tokj]; cur.idx = sm.wb_idx[tokj];
            if (better(acc, row, cur)) { sm.wb_d2[tokj] = acc; sm.wb_idx[tokj] = row; }
        }
    };

    // A run of cnt tiles j0, j0 + slices, ...: two tiles of heads are staged ahead in shared memory and a third is
    // in flight in registers; the MMAs of a tile are issued right after its predecessor has been read back from
    // tensor memory. done: MMA commits of this block so far (barrier phase and buffer of the next tile).
    int done = 0;
    bool ok = true;
    auto run = [&](int j0, int cnt, int limit) {
        if (cnt <= 0 || !ok) return;
        tile_fetch(j0, limit);
        tile_store(done & 1, j0, limit);
        if (cnt > 1) { tile_fetch(j0 + slices, limit); tile_store((done + 1) & 1, j0 + slices, limit); }
        if (cnt > 2) tile_fetch(j0 + 2 * slices, limit);
        __syncthreads();
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue_mma(done & 1);
        }
        for (int i = 0; i < cnt; ++i) {
            const int buf = (done + i) & 1;
            // wait for the MMAs of this tile (bounded)
            {
                const uint32_t parity = (uint32_t)((done + i) & 1);
                unsigned fin = 0, spins = 0;
                while (!fin && spins < kTcSpinLimit) {
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                                 : "=r"(fin) : "r"(sBar), "r"(parity) : "memory");
                    ++spins;
                }
                if (!fin) sm.failed = 1;
            }
            __syncthreads();
            if (sm.failed) { ok = false; return; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // read-back: this thread's token row, 128 columns in four pieces of 32
            const float* xat = sm.xa[buf];
#pragma unroll 1
            for (int cc = 0; cc < kTcTileN; cc += 32) {
                uint32_t v[32];
                const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)cc;
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                      "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                      "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                      "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (tid < cl) {
#pragma unroll
                    for (int q = 0; q < 32; ++q) {
                        if (__uint_as_float(v[q]) >= xat[cc + q] + my_kn) {          // rare
                            const unsigned slot = atomicAdd(&sm.ncand, 1u);
                            if (slot < (unsigned)kTcCand) sm.cand[slot] = (unsigned)tid | ((unsigned)(cc + q) << 8);
                        }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();
            // the accumulator is free: start the next tile (its heads were staged at least one barrier ago)
            if (i + 1 < cnt && tid == 0) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_mma(buf ^ 1);
            }
            // exact distances of the flagged pairs of this tile; warp w owns the tokens with index % 4 == w
            const unsigned nc = sm.ncand;
            const int row0 = (j0 + i * slices) * kTcTileN;
            if (nc <= (unsigned)kTcCand) {
                // four pairs per turn, two per half-warp with both rows of each pair requested before any is used:
                // a pair's exact distance is a chain of two global loads and a reduction, so the pairs of a tile
                // are evaluated side by side instead of one after the other
                for (unsigned base = 0; base < nc; base += 32) {
                    const bool have = base + lane < nc;
                    const unsigned cd = have ? sm.cand[base + lane] : 0u;
                    unsigned mine = __ballot_sync(0xffffffffu, have && (cd & 3u) == (unsigned)warp);
                    while (mine) {
                        int sel[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            sel[x] = mine ? __ffs(mine) - 1 : -1;
                            if (mine) mine &= mine - 1;
                        }
                        const int half = lane >> 4, l16 = lane & 15;
                        unsigned long long acc[2];
                        unsigned cdv[2];
                        uint4 xr[2], kr[2];
#pragma unroll
                        for (int y = 0; y < 2; ++y) {
                            const int sidx = sel[2 * y + half];
                            cdv[y] = __shfl_sync(0xffffffffu, cd, sidx < 0 ? 0 : sidx);
                            if (sidx >= 0) {
                                xr[y] = *reinterpret_cast<const uint4*>(Xu + (size_t)(row0 + (int)(cdv[y] >> 8)) * D + l16 * 8);
                                kr[y] = reinterpret_cast<const uint4*>(key_row<D>(C, a, r, u, e0 + (int)(cdv[y] & 255u)))[l16];
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
                            acc[y] = 0;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[y] += fx_sqdiff(xf[e], kf[e]);
#pragma unroll
                            for (int off = 8; off > 0; off >>= 1) acc[y] += __shfl_xor_sync(0xffffffffu, acc[y], off);
                        }
                        // lane 0 applies the (up to) four results one after the other: they may concern one token
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int y = x >> 1, hsrc = (x & 1) * 16;
                            const unsigned long long d2 = __shfl_sync(0xffffffffu, acc[y], hsrc);
                            const unsigned cdx = __shfl_sync(0xffffffffu, cdv[y], hsrc);
                            if (lane == 0 && sel[x] >= 0) {
                                const int tokj = (int)(cdx & 255u), row = row0 + (int)(cdx >> 8);
                                Best cur;
                                cur.d2 = sm.wb_d2[tokj]; cur.idx = sm.wb_idx[tokj];
                                if (better(d2, row, cur)) { sm.wb_d2[tokj] = d2; sm.wb_idx[tokj] = row; }
                            }
                        }
                    }
                }
            } else {                                                          // too many to list: every pair of the tile
                const int nrow = min(kTcTileN, limit - row0);
                for (int tokj = warp; tokj < cl; tokj += kTcThreads / 32)
                    for (int rr = 0; rr < nrow; ++rr) exact_pair(tokj, row0 + rr);
            }
            __syncthreads();
            if (tid == 0) sm.ncand = 0;
            if (i + 2 < cnt) {                                                // this tile's buffer is free since its MMAs ended
                tile_store(buf, j0 + (i + 2) * slices, limit);
                if (i + 3 < cnt) tile_fetch(j0 + (i + 3) * slices, limit);
            }
        }
        done += cnt;
    };
    const int bx = (int)blockIdx.x;
    const int nA = JA > bx ? (JA - bx + slices - 1) / slices : 0;      // this block's tiles below JA
    run(bx, nA, JA * kTcTileN);
    pdl_wait();
    pdl_trigger();
    const int m = C.m_unit[u];
    const int JT = (m + kTcTileN - 1) / kTcTileN;
    const int jB = bx + nA * slices;                                   // this block's first tile at or above JA
    const int nB = JT > jB ? (JT - jB + slices - 1) / slices : 0;
    run(jB, nB, m);
    __syncthreads();
    if (ok) {
        for (int j = tid; j < kChunk; j += kTcThreads) {
            Best bb;
            bb.d2 = sm.wb_d2[j]; bb.idx = sm.wb_idx[j]; bb.pad = 0;
            outp[j] = bb;
        }
    } else {
        for (int j = tid; j < kChunk; j += kTcThreads) { Best bb; bb.d2 = ~0ull; bb.idx = INT_MAX; bb.pad = 0; outp[j] = bb; }
        if (tid == 0) atomicOr(&C.status[u], 4);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128u) : "memory");
}

}  // namespace sgk
