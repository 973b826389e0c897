// Host side of the SubGen library: handles, memory layout, launches, C ABI (see include/subgen.h).
#include "../../include/subgen.h"

#include <cuda.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <string>
#include <type_traits>
#include <vector>

#include "subgen_kernels.cuh"
#include "subgen_query_mma.cuh"
#include "subgen_insert_mma.cuh"
#include "subgen_step_fused.cuh"
#include "subgen_prefill.cuh"
#include "subgen_score_tc.cuh"
#include "subgen_prefill_persist.cuh"
#include "subgen_exact_mma.cuh"
#include "subgen_kcenter.cuh"

using namespace sgk;

namespace {

thread_local std::string g_err;

int fail(int code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

#define CUDA_TRY(expr)                                                                      \
    do {                                                                                    \
        cudaError_t err__ = (expr);                                                         \
        if (err__ != cudaSuccess) return fail(SUBGEN_ECUDA, "%s: %s", #expr, cudaGetErrorString(err__)); \
    } while (0)

constexpr size_t kAlign = 256;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
    size_t X, S, xn, cnt, ctok, stok, Mk, Mv, MW, Mtok, ringK, ringV;
    size_t n_unit, m_unit, mu, status, last_cid, last_open, last_d2, part1, part2, ticket1, ticket2, qnext, qnext2, part_tau, MinvW, pairs;
    size_t thr2, level, Xh, xhn, alias, ndist, epoch, order, m_hist, next_best;
    size_t stage_q, stage_k, stage_v, stage_out, cu, stats;
    size_t book_begin, book_end;   // bookkeeping region cleared at creation
    size_t total;
};

struct Dims {
    int B, H, Hkv, G, D, t, s, w, m_max, splits, U;
    int Gs;                        // columns the query scratch is sized for: G * max(1, nq_max)
    int sp_insert, sp_tau, sp_z;   // blocks per unit of the three step kernels (splits = their maximum)
    int sp_fused;                  // blocks per unit of the one-kernel step
    size_t E;   // bytes per element
};

bool resolve(const subgen_config* c, Dims* o, const char** why) {
    if (!c) { *why = "config is NULL"; return false; }
    Dims d;
    d.B = c->B; d.H = c->H; d.Hkv = c->Hkv ? c->Hkv : c->H; d.D = c->d; d.t = c->t; d.s = c->s; d.w = c->window;
    d.m_max = c->m_max ? c->m_max : 8192;
    if (d.B <= 0 || d.H <= 0 || d.Hkv <= 0) { *why = "B, H, Hkv must be positive"; return false; }
    if (d.H % d.Hkv) { *why = "H must be a multiple of Hkv"; return false; }
    d.G = d.H / d.Hkv;
    if (d.G != 1 && d.G != 2 && d.G != 4 && d.G != 8) { *why = "H / Hkv must be 1, 2, 4 or 8"; return false; }
    if (c->nq_max < 0 || d.G * (c->nq_max ? c->nq_max : 1) > 8) { *why = "(H / Hkv) * nq_max must be <= 8"; return false; }
    d.Gs = d.G * (c->nq_max ? c->nq_max : 1);
    if (d.D != 64 && d.D != 128) { *why = "d must be 64 or 128"; return false; }
    if (d.t < 1 || d.t > 64) { *why = "t must be in 1..64"; return false; }
    if (d.s < 1 || d.s > 65536) { *why = "s must be in 1..65536"; return false; }
    if (d.w < 0) { *why = "window must be >= 0"; return false; }
    if (d.m_max < 1) { *why = "m_max must be positive"; return false; }
    if (!(c->delta >= 0.f) || !isfinite(c->delta) || c->delta > 32768.f) { *why = "delta must be finite, in [0, 32768]"; return false; }
    if (c->dtype != SUBGEN_DTYPE_FP32 && c->dtype != SUBGEN_DTYPE_BF16) { *why = "unknown dtype"; return false; }
    if (c->unit_stride < 0 || (c->unit_stride && c->unit_stride < d.Hkv) || c->unit_offset < 0 ||
        (long long)(d.B - 1) * (c->unit_stride ? c->unit_stride : d.Hkv) + c->unit_offset + d.Hkv - 1 > 0x7fffffffLL) {
        *why = "unit_stride must be 0 or >= Hkv, unit_offset >= 0, and the largest unit index must fit 31 bits";
        return false;
    }
    if (c->step_mode < SUBGEN_STEP_AUTO || c->step_mode > SUBGEN_STEP_SPLIT) { *why = "unknown step_mode"; return false; }
    if ((long long)d.B * d.Hkv > 65535) { *why = "B * Hkv must be <= 65535"; return false; }
    d.E = c->dtype == SUBGEN_DTYPE_FP32 ? 4 : 2;
    d.U = d.B * d.Hkv;
    if (c->splits < 0 || c->splits > 128) { *why = "splits must be in 0..128"; return false; }
    const bool bf16 = c->dtype == SUBGEN_DTYPE_BF16;
    if (c->splits) {
        d.sp_insert = d.sp_tau = d.sp_z = c->splits;
    } else {
        // Aim at one resident wave: the kernels hand out work inside a unit dynamically, so blocks that are all
        // resident finish together, while a partial second wave leaves most SMs idle at the end.
        // Resident blocks per SM (128 threads each): insert 6, cluster scan 6, value scan 4.
        auto fit = [&](int per_sm, int lo) {
            int sp = (148 * per_sm) / d.U;
            return sp < lo ? lo : (sp > 64 ? 64 : sp);
        };
        if (bf16) {
            d.sp_insert = fit(6, 1); d.sp_tau = fit(6, 1); d.sp_z = fit(4, 1);
            if (d.sp_z > 16) d.sp_z = 16;      // the last block merges sp_z numerator partials of G*d floats each
            // Cluster scan with more than a third of a wave of units: one wave can no longer be filled evenly (two
            // blocks per unit overshoot it, one leaves slots empty), and a wave and a bit is the worst shape. Then
            // aim at two and a half waves or more of smaller blocks, whose end is ragged by a small share only
            // (measured: 512 units 0.301 -> 0.261 ms per step, 1024 units 0.231 -> 0.216, 2048 units 1.237 -> 1.197).
            if (d.U > 296) {
                const int sp = (5 * 148 * 6 / 2 + d.U - 1) / d.U;
                d.sp_tau = sp < 1 ? 1 : (sp > 8 ? 8 : sp);
            }
        }
        else { d.sp_insert = d.sp_tau = d.sp_z = fit(8, 1); }
    }
    if (const char* env = getenv("SUBGEN_SPLITS")) {       // tuning aid: "insert,cluster,value"
        int a = 0, b = 0, e = 0;
        if (sscanf(env, "%d,%d,%d", &a, &b, &e) == 3 && a > 0 && b > 0 && e > 0 && a <= 128 && b <= 128 && e <= 128) {
            d.sp_insert = a; d.sp_tau = b; d.sp_z = e;
        }
    }
    d.splits = d.sp_insert > d.sp_tau ? d.sp_insert : d.sp_tau;
    if (d.sp_z > d.splits) d.splits = d.sp_z;
    // one-kernel step: 256-thread blocks, two per SM, one resident wave
    d.sp_fused = c->splits ? c->splits : (148 * 2) / d.U;
    d.sp_fused = d.sp_fused < 1 ? 1 : (d.sp_fused > 64 ? 64 : d.sp_fused);
    if (const char* env = getenv("SUBGEN_FUSED_SPLITS")) {
        const int a = atoi(env);
        if (a > 0 && a <= 128) d.sp_fused = a;
    }
    if (d.sp_fused > d.splits) d.splits = d.sp_fused;
    *o = d;
    return true;
}

Layout make_layout(const Dims& d) {
    Layout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const size_t U = d.U, row = (size_t)d.D * d.E;
    L.X = take(U * d.m_max * row);
    L.S = take(U * d.m_max * d.t * row);
    L.Xh = take(U * d.m_max * (size_t)kHeadDims * d.E);
    L.Mk = take(U * d.s * row);
    L.Mv = take(U * d.s * row);
    L.ringK = take(U * (size_t)d.w * row);
    L.ringV = take(U * (size_t)d.w * row);
    L.stage_q = take((size_t)d.B * d.H * row);
    L.stage_k = take(U * row);
    L.stage_v = take(U * row);
    L.stage_out = take((size_t)d.B * d.H * row);
    L.cu = take(((size_t)d.B + 1) * sizeof(int));
    L.part1 = take(U * d.splits * sizeof(Best));
    L.part2 = take(U * (d.splits + 2) * d.Gs * (size_t)(d.D + 2) * sizeof(float));   // + 2: the evenly cut value scan
    L.part_tau = take(U * d.splits * d.Gs * 2 * sizeof(float));
    L.book_begin = off;
    L.cnt = take(U * d.m_max * sizeof(int));
    L.xn = take(U * d.m_max * sizeof(float));
    L.xhn = take(U * d.m_max * sizeof(float));
    L.alias = take(U * d.m_max * (size_t)d.t + 16 * 64);   // + one item's worth: the cluster scan loads 16 rows at a time
    L.ndist = take(U * d.m_max + 16);
    L.n_unit = take(U * sizeof(int));
    L.m_unit = take(U * sizeof(int));
    L.mu = take(U * sizeof(uint64_t));
    L.status = take(U * sizeof(int));
    L.last_open = take(U * sizeof(int));
    L.ticket1 = take(U * sizeof(unsigned));
    L.ticket2 = take(U * sizeof(unsigned));
    L.qnext = take(U * sizeof(unsigned));
    L.qnext2 = take(U * sizeof(unsigned));
    L.pairs = take(U * sizeof(uint64_t));
    L.epoch = take(U * sizeof(int));
    L.order = take(U * sizeof(int));
    L.m_hist = take(2 * U * sizeof(int));
    L.next_best = take(U * sizeof(Best));
    L.thr2 = take(U * sizeof(uint64_t));
    L.level = take(U * sizeof(int));
    L.MinvW = take(U * d.s * sizeof(float));
    L.MW = take(U * d.s * sizeof(uint64_t));
    L.stats = take(8 * sizeof(uint64_t));
    L.book_end = off;
    // regions initialised to all-ones (-1 / UINT64_MAX)
    L.ctok = take(U * d.m_max * sizeof(int));
    L.stok = take(U * d.m_max * d.t * sizeof(int));
    L.Mtok = take(U * d.s * sizeof(int));
    L.last_cid = take(U * sizeof(int));
    L.last_d2 = take(U * sizeof(uint64_t));
    L.total = off;
    return L;
}

}  // namespace

struct subgen {
    subgen_config cfg;
    Dims d;
    Layout L;
    char* ws = nullptr;
    bool owns = false;
    cudaStream_t st = nullptr;
    std::vector<int> n_host;     // tokens seen per sequence (mirror of the device counters)
    uint64_t launches = 0;
    bool prof = false;
    std::vector<cudaEvent_t> ev;  // four per profiled step
    size_t ev_used = 0;
    std::vector<cudaEvent_t> pev; // prefill: start, after the value phase, then (score, resolve) ends per chunk, end
    size_t pev_used = 0;
    char* scratch = nullptr;      // prefill scratch (library-owned, grows on demand)
    size_t scratch_bytes = 0;
    bool seq_prefill = false;     // SUBGEN_PREFILL=seq: token-by-token prefill also for bf16
    bool mma_score = false;       // SUBGEN_PREFILL=mma: chunk scoring with warp-level MMAs instead of tcgen05 (d = 128)
    int persist = -1;             // key phase as one persistent kernel (d = 128): -1 chosen from the unit count,
                                  // 0 / 1 forced by SUBGEN_PREFILL=chunk / persist
    bool pf_persist = false;      // the most recent profiled prefill used the persistent kernel
    volatile unsigned* done_host = nullptr;   // subgen_step_host: a pinned word the stream writes after each step
    CUdeviceptr done_dev = 0;
    unsigned done_seq = 0;
    cudaStream_t st2 = nullptr;   // prefill: the key phase runs here, beside the value phase on st (fork / join by events)
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    bool order_ready = false;     // the units are ranked by cluster count (set by a prefill of a many-unit handle)
    bool search_ready = false;    // next_best holds the search for the next step's leaving token (host-buffer steps)
    int step_seq = 0;             // one-kernel steps since the epochs were last set
    bool epoch_stale = true;      // the units' epochs may lag their token counts (creation, prefill, checkpoint load)
    bool fused = false;           // stream steps run as one kernel (bf16, not bounded): few units, or SUBGEN_STEP=fused
    unsigned long long* pf_phase_dev = nullptr;   // its per-unit phase times (inside scratch)
};

namespace {

// Every unit's threshold back to delta^2 (bounded handles). Synchronous.
cudaError_t reset_thresholds(subgen* h) {
    const unsigned long long d2 = (unsigned long long)floor((double)h->cfg.delta * (double)h->cfg.delta * 4294967296.0);
    std::vector<unsigned long long> v((size_t)h->d.U, d2);
    cudaError_t e = cudaStreamSynchronize(h->st);
    if (e == cudaSuccess) e = cudaMemcpy(h->ws + h->L.thr2, v.data(), v.size() * 8, cudaMemcpyHostToDevice);
    return e;
}

template <typename T> Cache<T> make_cache(const subgen* h) {
    const Dims& d = h->d;
    const Layout& L = h->L;
    char* w = h->ws;
    Cache<T> C;
    C.B = d.B; C.H = d.H; C.Hkv = d.Hkv; C.G = d.G; C.t = d.t; C.s = d.s; C.w = d.w; C.m_max = d.m_max;
    C.delta2_fx = (unsigned long long)floor((double)h->cfg.delta * (double)h->cfg.delta * 4294967296.0);
    C.key0 = (uint32_t)h->cfg.seed; C.key1 = (uint32_t)(h->cfg.seed >> 32);
    C.X = (T*)(w + L.X); C.S = (T*)(w + L.S); C.xn = (float*)(w + L.xn);
    C.Xh = (T*)(w + L.Xh); C.xhn = (float*)(w + L.xhn); C.alias = (unsigned char*)(w + L.alias); C.ndist = (unsigned char*)(w + L.ndist);
    C.cnt = (int*)(w + L.cnt); C.ctok = (int*)(w + L.ctok); C.stok = (int*)(w + L.stok);
    C.Mk = (T*)(w + L.Mk); C.Mv = (T*)(w + L.Mv);
    C.MW = (unsigned long long*)(w + L.MW); C.Mtok = (int*)(w + L.Mtok);
    C.ringK = (T*)(w + L.ringK); C.ringV = (T*)(w + L.ringV);
    C.n_unit = (int*)(w + L.n_unit); C.m_unit = (int*)(w + L.m_unit);
    C.mu = (unsigned long long*)(w + L.mu); C.status = (int*)(w + L.status);
    C.last_cid = (int*)(w + L.last_cid); C.last_open = (int*)(w + L.last_open);
    C.last_d2 = (unsigned long long*)(w + L.last_d2);
    C.part1 = (Best*)(w + L.part1); C.part2 = (float*)(w + L.part2);
    C.ticket1 = (unsigned*)(w + L.ticket1); C.ticket2 = (unsigned*)(w + L.ticket2);
    C.qnext = (unsigned*)(w + L.qnext); C.qnext2 = (unsigned*)(w + L.qnext2);
    C.part_tau = (float*)(w + L.part_tau); C.MinvW = (float*)(w + L.MinvW);
    C.pairs = (unsigned long long*)(w + L.pairs);
    C.epoch = (int*)(w + L.epoch);
    C.m_hist = (int*)(w + L.m_hist);
    C.next_best = (Best*)(w + L.next_best);
    C.order = h->order_ready ? (const int*)(w + L.order) : nullptr;
    C.bounded = h->cfg.bounded ? 1 : 0;
    C.uid_stride = h->cfg.unit_stride ? h->cfg.unit_stride : d.Hkv;
    C.uid_off = h->cfg.unit_offset;
    C.thr2 = (unsigned long long*)(w + L.thr2); C.level = (int*)(w + L.level);
    return C;
}

// Launch with the programmatic stream serialization attribute: the kernel may be scheduled while its predecessor
// in the stream still runs and orders itself with pdl_wait(). SUBGEN_PDL=0 falls back to ordinary launches.
// plain = true launches the ordinary way (a full dependency on everything earlier in the stream): used for the
// first kernel of a call when that kernel touches the caller's inputs before its dependency wait.
// A failed launch is remembered in g_launch_err, which take_launch_error() returns and clears.
thread_local cudaError_t g_launch_err = cudaSuccess;

cudaError_t take_launch_error() {
    cudaError_t e = g_launch_err;
    g_launch_err = cudaSuccess;
    const cudaError_t last = cudaGetLastError();
    return e != cudaSuccess ? e : last;
}

template <typename... KArgs, typename... Args>
void launch_pdl_opt(bool plain, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    static const bool off = [] { const char* e = getenv("SUBGEN_PDL"); return e && e[0] == '0'; }();
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = (off || plain) ? 0 : 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
    if (e != cudaSuccess && g_launch_err == cudaSuccess) g_launch_err = e;
}
template <typename... KArgs, typename... Args>
void launch_pdl_smem(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    launch_pdl_opt(false, kern, grid, block, smem, st, args...);
}
template <typename... KArgs, typename... Args>
void launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
    launch_pdl_opt(false, kern, grid, block, 0, st, args...);
}

// The two query kernels of a bf16 handle for G columns. first_plain: the cluster scan is the first kernel of the
// call (read-only queries) and loads the caller's q before its dependency wait, so it is launched the ordinary way.
template <int D, int G>
void launch_query_bf16(const Cache<__nv_bfloat16>& C, dim3 grid, dim3 grid_z, cudaStream_t st, const __nv_bfloat16* q,
                       __nv_bfloat16* out, cudaEvent_t mid, int advance, int flat_ipu, int flat_slots, bool first_plain) {
    launch_pdl_opt(first_plain, query_tau_kernel<D, G>, grid, dim3(kQmThreads), 0, st, C, q);
    if (mid) cudaEventRecord(mid, st);
    if (flat_ipu) launch_pdl(query_z_flat_kernel<D, G>, grid_z, dim3(kQmThreads), st, C, q, out, (int)grid.x, advance, flat_ipu, flat_slots);
    else launch_pdl(query_z_kernel<D, G>, grid_z, dim3(kQmThreads), st, C, q, out, (int)grid.x, advance);
}

// fp32 caches: CUDA-core dot products (full fp32 products). bf16 caches: tensor-core kernels.
template <typename T, int D>
void launch_query(const Cache<T>& C, int G, dim3 grid, dim3 grid_z, cudaStream_t st, const void* q, void* out, cudaEvent_t mid, int advance = 1,
                  int flat_ipu = 0, int flat_slots = 0, bool first_plain = false) {
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        const T* qq = (const T*)q;
        T* oo = (T*)out;
        switch (G) {
            case 1: launch_query_bf16<D, 1>(C, grid, grid_z, st, qq, oo, mid, advance, flat_ipu, flat_slots, first_plain); break;
            case 2: launch_query_bf16<D, 2>(C, grid, grid_z, st, qq, oo, mid, advance, flat_ipu, flat_slots, first_plain); break;
            case 4: launch_query_bf16<D, 4>(C, grid, grid_z, st, qq, oo, mid, advance, flat_ipu, flat_slots, first_plain); break;
            default: launch_query_bf16<D, 8>(C, grid, grid_z, st, qq, oo, mid, advance, flat_ipu, flat_slots, first_plain); break;
        }
    } else {
        switch (G) {
            // launched the ordinary way when it is the first kernel of its call (it loads q before its dependency wait)
            case 1: launch_pdl_opt(first_plain, query_kernel<T, D, 1>, grid, dim3(kQueryThreads), 0, st, C, (const T*)q, (T*)out, advance); break;
            case 2: launch_pdl_opt(first_plain, query_kernel<T, D, 2>, grid, dim3(kQueryThreads), 0, st, C, (const T*)q, (T*)out, advance); break;
            case 4: launch_pdl_opt(first_plain, query_kernel<T, D, 4>, grid, dim3(kQueryThreads), 0, st, C, (const T*)q, (T*)out, advance); break;
            default: launch_pdl_opt(first_plain, query_kernel<T, D, 8>, grid, dim3(kQueryThreads), 0, st, C, (const T*)q, (T*)out, advance); break;
        }
        if (mid) cudaEventRecord(mid, st);
    }
}

// The value scan can be cut evenly over the grid when every unit has the same number of 16-row items, i.e. the same
// window fill. That pays when the per-unit split needs more than one wave of blocks (many units: measured +2 % on
// the step at 2048 units); with one wave or less the per-unit split with its work queue is faster (fewer units
// per block, no second partial). Returns items per unit (0: use the per-unit split) and the grid size.
// n_shift: 1 for a stream step (the step's token is already in the ring), 0 for a read-only query.
int flat_value_scan(const subgen* h, int n_shift, int* grid) {
    static const bool off = [] { const char* e = getenv("SUBGEN_FLAT"); return e && e[0] == '0'; }();
    if (off || h->cfg.dtype != SUBGEN_DTYPE_BF16) return 0;
    const Dims& d = h->d;
    if ((long long)d.U * d.sp_z <= 148 * 4) return 0;
    int wn0 = -1;
    for (int b = 0; b < d.B; ++b) {
        const long long n = (long long)h->n_host[b] + n_shift;
        const int wn = n < d.w ? (int)n : d.w;
        if (wn0 < 0) wn0 = wn;
        else if (wn != wn0) return 0;
    }
    const int ipu = ((d.s + 15) >> 4) + ((wn0 + 15) >> 4);
    const long long total = (long long)d.U * ipu;
    const long long nb = total < 148 * 4 ? total : 148 * 4;
    // a unit's partials must fit the room part2 has for it
    const long long per_unit = (nb + d.U - 1) / d.U + 1;
    if (per_unit > d.splits + 2) return 0;
    *grid = (int)nb;
    return ipu;
}

template <typename T, int D>
int launch_step_td(subgen* h, const void* q, const void* k, const void* v, void* out) {
    Cache<T> C = make_cache<T>(h);
    const dim3 grid_i(h->d.sp_insert, h->d.U), grid_t(h->d.sp_tau, h->d.U), grid_z(h->d.sp_z, h->d.U);
    cudaEvent_t* e = nullptr;
    if (h->prof) {
        if (h->ev_used + 4 > h->ev.size()) {
            for (int i = 0; i < 4; ++i) {
                cudaEvent_t x;
                CUDA_TRY(cudaEventCreate(&x));
                h->ev.push_back(x);
            }
        }
        e = &h->ev[h->ev_used];
        h->ev_used += 4;
        CUDA_TRY(cudaEventRecord(e[0], h->st));
    }
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (h->fused) {
            const dim3 grid_f(h->d.sp_fused, h->d.U);
            // The kernel works on the token that leaves the window before its dependency wait; it takes the token
            // count from the unit's epoch plus the number of steps since the epochs were set. The first step after
            // that is launched the ordinary way: it reads what the epoch kernel, its direct predecessor, wrote.
            const bool first = h->epoch_stale;
            if (first) {
                epoch_sync_kernel<<<(h->d.U + 255) / 256, 256, 0, h->st>>>(C, h->d.U);
                h->epoch_stale = false;
                h->step_seq = 0;
                h->launches += 1;
            }
            const int seq = h->step_seq++;
            if (e) CUDA_TRY(cudaEventRecord(e[1], h->st));          // the whole step is reported as the middle interval
            switch (h->d.G) {
                case 1: launch_pdl_opt(first, step_fused_kernel<D, 1>, grid_f, dim3(kFsThreads), 0, h->st, C, (const T*)q, (const T*)k, (const T*)v, (T*)out, seq); break;
                case 2: launch_pdl_opt(first, step_fused_kernel<D, 2>, grid_f, dim3(kFsThreads), 0, h->st, C, (const T*)q, (const T*)k, (const T*)v, (T*)out, seq); break;
                case 4: launch_pdl_opt(first, step_fused_kernel<D, 4>, grid_f, dim3(kFsThreads), 0, h->st, C, (const T*)q, (const T*)k, (const T*)v, (T*)out, seq); break;
                default: launch_pdl_opt(first, step_fused_kernel<D, 8>, grid_f, dim3(kFsThreads), 0, h->st, C, (const T*)q, (const T*)k, (const T*)v, (T*)out, seq); break;
            }
            if (e) { CUDA_TRY(cudaEventRecord(e[2], h->st)); CUDA_TRY(cudaEventRecord(e[3], h->st)); }
            CUDA_TRY(take_launch_error());
            h->launches += 1;
            return SUBGEN_OK;
        }
        if (h->epoch_stale) {            // ordinary launch: a full dependency on the prefill (or load) before it
            epoch_sync_kernel<<<(h->d.U + 255) / 256, 256, 0, h->st>>>(C, h->d.U);
            h->epoch_stale = false;
            h->launches += 1;
        }
        if (C.bounded) launch_pdl(insert_mma_kernel<D, true>, grid_i, dim3(kInsertMmaThreads), h->st, C, (const T*)k, (const T*)v);
        else if (h->search_ready) launch_pdl(insert_mma_kernel<D, false, 2>, dim3(1, h->d.U), dim3(kInsertMmaThreads), h->st, C, (const T*)k, (const T*)v);
        else launch_pdl(insert_mma_kernel<D, false>, grid_i, dim3(kInsertMmaThreads), h->st, C, (const T*)k, (const T*)v);
        h->search_ready = false;
    } else {
        if (C.bounded) launch_pdl(insert_kernel<T, D, true>, grid_i, dim3(kInsertThreads), h->st, C, (const T*)k, (const T*)v);
        else launch_pdl(insert_kernel<T, D, false>, grid_i, dim3(kInsertThreads), h->st, C, (const T*)k, (const T*)v);
    }
    if (e) CUDA_TRY(cudaEventRecord(e[1], h->st));
    int flat_grid = 0;
    const int flat_ipu = flat_value_scan(h, 1, &flat_grid);
    launch_query<T, D>(C, h->d.G, grid_t, flat_ipu ? dim3(flat_grid) : grid_z, h->st, q, out, e ? e[2] : nullptr, 1, flat_ipu, h->d.splits + 2);
    if (e) CUDA_TRY(cudaEventRecord(e[3], h->st));
    CUDA_TRY(take_launch_error());
    h->launches += std::is_same<T, __nv_bfloat16>::value ? 3 : 2;
    return SUBGEN_OK;
}

// Read-only query with nq queries per head: the nq queries of the G heads of a KV head become G * nq columns.
template <typename T, int D>
int launch_query_only_td(subgen* h, const void* q, int nq, void* out) {
    Cache<T> C = make_cache<T>(h);
    C.H = h->d.H * nq;
    C.G = h->d.G * nq;
    const dim3 grid_t(h->d.sp_tau, h->d.U), grid_z(h->d.sp_z, h->d.U);
    int flat_grid = 0;
    const int flat_ipu = flat_value_scan(h, 0, &flat_grid);
    launch_query<T, D>(C, C.G, grid_t, flat_ipu ? dim3(flat_grid) : grid_z, h->st, q, out, nullptr, 0, flat_ipu, h->d.splits + 2, true);
    CUDA_TRY(take_launch_error());
    h->launches += std::is_same<T, __nv_bfloat16>::value ? 2 : 1;
    return SUBGEN_OK;
}

int launch_step(subgen* h, const void* q, const void* k, const void* v, void* out) {
    const bool f32 = h->cfg.dtype == SUBGEN_DTYPE_FP32;
    if (h->d.D == 64) return f32 ? launch_step_td<float, 64>(h, q, k, v, out) : launch_step_td<__nv_bfloat16, 64>(h, q, k, v, out);
    return f32 ? launch_step_td<float, 128>(h, q, k, v, out) : launch_step_td<__nv_bfloat16, 128>(h, q, k, v, out);
}

template <typename T, int D>
int launch_prefill_td(subgen* h, const void* K, const void* V, int n, const int* cu_dev, int total) {
    Cache<T> C = make_cache<T>(h);
    if (C.bounded) prefill_seq_kernel<T, D, true><<<h->d.U, kPrefillThreads, 0, h->st>>>(C, (const T*)K, (const T*)V, n, cu_dev, total);
    else prefill_seq_kernel<T, D, false><<<h->d.U, kPrefillThreads, 0, h->st>>>(C, (const T*)K, (const T*)V, n, cu_dev, total);
    CUDA_TRY(take_launch_error());
    h->launches += 1;
    return SUBGEN_OK;
}

// bf16: values for the whole call at once, keys chunk by chunk (subgen_prefill.cuh).
// add[b]: tokens appended to sequence b by this call (host copy).
template <int D>
int launch_prefill_chunked(subgen* h, const void* K, const void* V, int n, const int* cu_dev, int total, const int* add) {
    typedef __nv_bfloat16 T;
    Cache<T> C = make_cache<T>(h);
    const Dims& d = h->d;
    int Lmax = 0;
    for (int b = 0; b < d.B; ++b) {
        const int lo = h->n_host[b] > d.w ? h->n_host[b] - d.w : 0;
        const int hi = h->n_host[b] + add[b] > d.w ? h->n_host[b] + add[b] - d.w : 0;
        Lmax = hi - lo > Lmax ? hi - lo : Lmax;
    }
    const bool tc = D == 128 && !h->mma_score;           // tcgen05 scoring (d = 128), else warp-level MMAs
    int slices = tc ? (148 * 4) / d.U : (148 * 4 + d.U - 1) / d.U;
    slices = slices < 1 ? 1 : (slices > 32 ? 32 : slices);
    PrefillArgs a;
    a.K = (const T*)K; a.V = (const T*)V; a.n_uniform = n; a.cu = cu_dev; a.total = total; a.Lmax = Lmax; a.slices = slices;
    a.Wbuf = nullptr; a.Tot = nullptr; a.Thr = nullptr; a.Mwin = nullptr; a.pbest = nullptr; a.mhist = nullptr;
    int launches = 0;
    bool join = false;
    if (Lmax > 0) {
        const size_t b_w = align_up((size_t)d.U * Lmax * 8), b_m = align_up((size_t)d.U * d.s * 4);
        const size_t b_p = align_up((size_t)d.U * slices * kChunk * sizeof(Best));
        const size_t b_h = align_up((size_t)d.U * 2 * sizeof(int));
        const size_t b_ns = align_up((size_t)d.U * kPpPhases * sizeof(unsigned long long));
        const size_t need = 3 * b_w + b_m + b_p + b_h + b_ns;
        if (need > h->scratch_bytes) {
            if (h->scratch) { CUDA_TRY(cudaStreamSynchronize(h->st)); CUDA_TRY(cudaFree(h->scratch)); h->scratch = nullptr; h->scratch_bytes = 0; }
            cudaError_t e = cudaMalloc((void**)&h->scratch, need);
            if (e != cudaSuccess) return fail(SUBGEN_ENOMEM, "subgen_prefill: cudaMalloc(%zu) for scratch failed: %s", need, cudaGetErrorString(e));
            h->scratch_bytes = need;
        }
        a.Wbuf = (unsigned long long*)h->scratch;
        a.Tot = (unsigned long long*)(h->scratch + b_w);
        a.Thr = (unsigned long long*)(h->scratch + 2 * b_w);
        a.Mwin = (int*)(h->scratch + 3 * b_w);
        a.pbest = (Best*)(h->scratch + 3 * b_w + b_m);
        a.mhist = (int*)(h->scratch + 3 * b_w + b_m + b_p);
        unsigned long long* phase_ns = (unsigned long long*)(h->scratch + 3 * b_w + b_m + b_p + b_h);
        auto mark = [&]() -> int {                       // profiling: one event on the stream
            if (!h->prof) return SUBGEN_OK;
            if (h->pev_used == h->pev.size()) {
                cudaEvent_t x;
                CUDA_TRY(cudaEventCreate(&x));
                h->pev.push_back(x);
            }
            CUDA_TRY(cudaEventRecord(h->pev[h->pev_used++], h->st));
            return SUBGEN_OK;
        };
        h->pev_used = 0;
        if (int rc = mark()) return rc;
        // The value phase (weights, running sums, coins, gather into M) and the key phase (clusters) share nothing
        // until the commit, so the key phase goes to the handle's second stream (higher priority: its few long-lived
        // blocks take their places first), forked from and joined back into the caller's stream by events, while the
        // value phase stays on the caller's stream. Two blocks of the persistent key kernel hold all registers of
        // their SM, so the coin kernel runs on the SMs that the key kernel leaves free or half used and on the
        // others once their units are done (256 units: 28.3 -> 26.4 ms; capping the key kernel's registers to let
        // both share every SM cost more in its read-back than the sharing returned).
        // With profiling on, both stay in one stream so that each can be timed.
        static const bool no_overlap = [] { const char* e = getenv("SUBGEN_PREFILL_OVERLAP"); return e && e[0] == '0'; }();
        const bool overlap = !h->prof && h->st2 && !no_overlap;
        auto value_phase = [&](cudaStream_t sv) -> int {
            CUDA_TRY(cudaMemsetAsync(a.Mwin, 0xFF, (size_t)d.U * d.s * 4, sv));
            constexpr int RPW = 32 / (D / 8);
            int bx = (Lmax + 8 * RPW - 1) / (8 * RPW);
            bx = bx > 64 ? 64 : bx;
            prefill_w_kernel<D><<<dim3(bx, d.U), 256, 0, sv>>>(C, a);
            prefill_scan_kernel<<<d.U, 1024, 0, sv>>>(C, a);
            // a warp per group of four slots and segment; one segment when the groups alone give enough warps (a scan
            // that ends early saves most over a whole prompt), more for handles with few units
            const int groups = (d.s + 3) / 4;
            long long want = (20000LL + (long long)d.U * groups - 1) / ((long long)d.U * groups);
            int segs = (int)(want < 1 ? 1 : want);
            int seg_len = (Lmax + segs - 1) / segs;
            seg_len = seg_len < 1024 ? 1024 : seg_len;
            seg_len = (seg_len + 31) / 32 * 32;
            segs = (Lmax + seg_len - 1) / seg_len;
            prefill_coin_kernel<<<dim3((groups + 3) / 4, segs, d.U), 128, 0, sv>>>(C, a, seg_len);
            int gx = (d.s + 8 * RPW - 1) / (8 * RPW);
            gx = gx > 32 ? 32 : gx;
            prefill_gather_kernel<D><<<dim3(gx, d.U), 256, 0, sv>>>(C, a);
            launches += 4;
            return SUBGEN_OK;
        };
        // Key phase. Many units with few representatives each: one persistent block per unit walks its chunks
        // (subgen_prefill_persist.cuh). Few units: a score and a resolve kernel per chunk, the representatives of a
        // unit spread over many blocks.
        // Bounded handles always walk their chunks in the persistent kernel: it is the one that can end a chunk at
        // the key that finds the budget used up and insert that key on its own.
        const bool persist = tc && (C.bounded || (h->persist >= 0 ? h->persist == 1 : d.U >= 24));
        h->pf_persist = persist && h->prof;
        auto key_phase = [&](cudaStream_t sk) -> int {
            if (persist) {
                h->pf_phase_dev = phase_ns;
                if (C.bounded) prefill_keys_persist_kernel<true><<<d.U, kPpThreads, kPpSmemBytes, sk>>>(C, a, h->prof ? phase_ns : nullptr);
                else prefill_keys_persist_kernel<false><<<d.U, kPpThreads, kPpSmemBytes, sk>>>(C, a, h->prof ? phase_ns : nullptr);
                launches += 1;
                if (int rc = mark()) return rc;
                return SUBGEN_OK;
            }
            const int nchunks = (Lmax + kChunk - 1) / kChunk;
            prefill_mhist_kernel<<<(d.U + 255) / 256, 256, 0, sk>>>(C, a, d.U);
            launches += 1;
            for (int c = 0; c < nchunks; ++c) {
                // both kernels stage their chunk keys before they wait for their predecessor in the stream;
                // chunk 0 reads the cluster-count history its immediate predecessor wrote before it waits: ordinary launch
                if (tc) launch_pdl_opt(c == 0, prefill_score_tc_kernel, dim3(slices, d.U), dim3(kTcThreads), kTcSmemBytes, sk, C, a, c);
                else prefill_score_kernel<D><<<dim3(slices, d.U), kScoreThreads, 0, sk>>>(C, a, c);
                if (int rc = mark()) return rc;
                launch_pdl(prefill_resolve_kernel<D>, dim3(d.U), dim3(kResolveThreads), sk, C, a, c);
                if (int rc = mark()) return rc;
            }
            launches += 2 * nchunks;
            return SUBGEN_OK;
        };
        if (overlap) {
            CUDA_TRY(cudaEventRecord(h->ev_fork, h->st));
            CUDA_TRY(cudaStreamWaitEvent(h->st2, h->ev_fork, 0));
            if (int rc = key_phase(h->st2)) return rc;
            CUDA_TRY(cudaEventRecord(h->ev_join, h->st2));
            join = true;
            if (int rc = value_phase(h->st)) return rc;
        } else {
            if (int rc = value_phase(h->st)) return rc;
            if (int rc = mark()) return rc;
            if (int rc = key_phase(h->st)) return rc;
        }
    }
    if (join) CUDA_TRY(cudaStreamWaitEvent(h->st, h->ev_join, 0));   // the clusters are complete
    int longest = 0;
    for (int b = 0; b < d.B; ++b) longest = add[b] > longest ? add[b] : longest;
    int fx = (int)(((size_t)(longest < d.w ? longest : d.w) * (D / 8) + 255) / 256);
    fx = fx < 1 ? 1 : (fx > 16 ? 16 : fx);
    if (Lmax > 0) { prefill_alias_kernel<<<dim3(8, d.U), 256, 0, h->st>>>(C); launches += 1; }
    prefill_finish_kernel<D><<<dim3(fx, d.U), 256, 0, h->st>>>(C, a);
    prefill_commit_kernel<<<(d.U + 255) / 256, 256, 0, h->st>>>(C, a, d.U);
    launches += 2;
    CUDA_TRY(take_launch_error());
    h->launches += launches;
    return SUBGEN_OK;
}

int launch_prefill(subgen* h, const void* K, const void* V, int n, const int* cu_dev, int total, const int* add) {
    const bool f32 = h->cfg.dtype == SUBGEN_DTYPE_FP32;
    if (!f32 && !h->seq_prefill)
        return h->d.D == 64 ? launch_prefill_chunked<64>(h, K, V, n, cu_dev, total, add)
                            : launch_prefill_chunked<128>(h, K, V, n, cu_dev, total, add);
    if (h->d.D == 64)
        return f32 ? launch_prefill_td<float, 64>(h, K, V, n, cu_dev, total)
                   : launch_prefill_td<__nv_bfloat16, 64>(h, K, V, n, cu_dev, total);
    return f32 ? launch_prefill_td<float, 128>(h, K, V, n, cu_dev, total)
               : launch_prefill_td<__nv_bfloat16, 128>(h, K, V, n, cu_dev, total);
}

// After a prefill of a bf16 handle that steps with one grid row per unit (three-kernel step): rank the units by
// cluster count, for the block order of the step's insertion kernel and cluster scan.
void rank_units(subgen* h) {
    static const bool off = [] { const char* e = getenv("SUBGEN_ORDER"); return e && e[0] == '0'; }();
    h->order_ready = false;
    if (off || h->cfg.dtype != SUBGEN_DTYPE_BF16 || h->fused) return;
    Cache<__nv_bfloat16> C = make_cache<__nv_bfloat16>(h);
    unit_order_kernel<<<(h->d.U + 255) / 256, 256, 0, h->st>>>(C, h->d.U, (int*)(h->ws + h->L.order));
    h->launches += 1;
    h->order_ready = true;
}

void destroy_side_stream(subgen* h) {
    if (h->st2) { cudaStreamSynchronize(h->st2); cudaStreamDestroy(h->st2); h->st2 = nullptr; }
    if (h->ev_fork) { cudaEventDestroy(h->ev_fork); h->ev_fork = nullptr; }
    if (h->ev_join) { cudaEventDestroy(h->ev_join); h->ev_join = nullptr; }
}

int check_device() {
    int n = 0;
    cudaError_t e = cudaGetDeviceCount(&n);
    if (e != cudaSuccess || n <= 0)
        return fail(SUBGEN_ECUDA, "no usable CUDA device (%s); this library has no CPU path",
                    e != cudaSuccess ? cudaGetErrorString(e) : "device count is 0");
    return SUBGEN_OK;
}

}  // namespace

extern "C" {

const char* subgen_last_error(void) { return g_err.c_str(); }

size_t subgen_workspace_bytes(const subgen_config* cfg) {
    Dims d;
    const char* why = "";
    if (!resolve(cfg, &d, &why)) { fail(SUBGEN_EINVAL, "subgen_workspace_bytes: %s", why); return 0; }
    return make_layout(d).total;
}

subgen_t* subgen_create_ex(const subgen_config* cfg) {
    Dims d;
    const char* why = "";
    if (!resolve(cfg, &d, &why)) { fail(SUBGEN_EINVAL, "subgen_create: %s", why); return nullptr; }
    if (check_device() != SUBGEN_OK) return nullptr;
    subgen* h = new subgen();
    h->cfg = *cfg;
    h->d = d;
    h->L = make_layout(d);
    h->st = (cudaStream_t)cfg->stream;
    if (cfg->workspace) {
        if (cfg->workspace_bytes < h->L.total || ((uintptr_t)cfg->workspace % kAlign)) {
            fail(SUBGEN_ENOMEM, "subgen_create: workspace needs %zu bytes, 256-byte aligned (got %zu)", h->L.total,
                 cfg->workspace_bytes);
            delete h;
            return nullptr;
        }
        h->ws = (char*)cfg->workspace;
    } else {
        cudaError_t e = cudaMalloc((void**)&h->ws, h->L.total);
        if (e != cudaSuccess) {
            fail(SUBGEN_ENOMEM, "subgen_create: cudaMalloc(%zu) failed: %s", h->L.total, cudaGetErrorString(e));
            delete h;
            return nullptr;
        }
        h->owns = true;
    }
    cudaError_t e1 = cudaMemsetAsync(h->ws + h->L.book_begin, 0, h->L.book_end - h->L.book_begin, h->st);
    cudaError_t e2 = cudaMemsetAsync(h->ws + h->L.book_end, 0xFF, h->L.total - h->L.book_end, h->st);
    // rows of M can be read (with weight zero) before their slot is filled: they must hold finite numbers
    if (e1 == cudaSuccess) e1 = cudaMemsetAsync(h->ws + h->L.Mk, 0, h->L.ringK - h->L.Mk, h->st);
    if (e1 != cudaSuccess || e2 != cudaSuccess) {
        fail(SUBGEN_ECUDA, "subgen_create: cudaMemsetAsync failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
        if (h->owns) cudaFree(h->ws);
        delete h;
        return nullptr;
    }
    h->n_host.assign(d.B, 0);
    int prio_lo = 0, prio_hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) != cudaSuccess) { cudaGetLastError(); prio_hi = 0; }
    if (cfg->dtype == SUBGEN_DTYPE_BF16 &&
        (cudaStreamCreateWithPriority(&h->st2, cudaStreamNonBlocking, prio_hi) != cudaSuccess ||
         cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess)) {
        fail(SUBGEN_ECUDA, "subgen_create: second stream: %s", cudaGetErrorString(cudaGetLastError()));
        destroy_side_stream(h);
        if (h->owns) cudaFree(h->ws);
        delete h;
        return nullptr;
    }
    // the tcgen05 score kernel needs more dynamic shared memory than the default limit; the attribute is per device,
    // so it is set for the device of every handle that can launch the kernel
    if (cfg->dtype == SUBGEN_DTYPE_BF16 && d.D == 128 &&
        (cudaFuncSetAttribute(prefill_score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes) != cudaSuccess ||
         cudaFuncSetAttribute(prefill_keys_persist_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPpSmemBytes) != cudaSuccess ||
         cudaFuncSetAttribute(prefill_keys_persist_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPpSmemBytes) != cudaSuccess)) {
        fail(SUBGEN_ECUDA, "subgen_create: cudaFuncSetAttribute failed: %s", cudaGetErrorString(cudaGetLastError()));
        destroy_side_stream(h);
        if (h->owns) cudaFree(h->ws);
        delete h;
        return nullptr;
    }
    if (const char* env = getenv("SUBGEN_PREFILL")) {
        h->seq_prefill = strcmp(env, "seq") == 0; h->mma_score = strcmp(env, "mma") == 0;
        if (strcmp(env, "chunk") == 0) h->persist = 0;
        if (strcmp(env, "persist") == 0) h->persist = 1;
    }
    // Stream steps as one kernel when the units are too few for the three-kernel chain to hide its own latency
    // (SUBGEN_STEP=fused / split forces either way). Bounded handles and fp32 handles keep their kernels.
    const bool can_fuse = cfg->dtype == SUBGEN_DTYPE_BF16 && !cfg->bounded;
    h->fused = can_fuse && d.U <= 148;
    if (cfg->step_mode == SUBGEN_STEP_FUSED) h->fused = can_fuse;
    if (cfg->step_mode == SUBGEN_STEP_SPLIT) h->fused = false;
    if (const char* env = getenv("SUBGEN_STEP")) {
        if (strcmp(env, "fused") == 0) h->fused = can_fuse;
        if (strcmp(env, "split") == 0) h->fused = false;
    }
    if (h->cfg.bounded) {
        // merges renumber the clusters in the middle of a chunk; only the persistent key kernel (bf16, d = 128) ends
        // a chunk at such a key. Other bounded handles insert their prompts token by token.
        if (!(cfg->dtype == SUBGEN_DTYPE_BF16 && d.D == 128) || h->mma_score) h->seq_prefill = true;
        if (reset_thresholds(h) != cudaSuccess) {
            fail(SUBGEN_ECUDA, "subgen_create: threshold initialisation failed");
            destroy_side_stream(h);
            if (h->owns) cudaFree(h->ws);
            delete h;
            return nullptr;
        }
    }
    return h;
}

subgen_t* subgen_create(int B, int H, int d, float delta, int t, int s, int window, uint64_t seed) {
    subgen_config c;
    memset(&c, 0, sizeof c);
    c.B = B; c.H = H; c.Hkv = H; c.d = d; c.delta = delta; c.t = t; c.s = s; c.window = window; c.seed = seed;
    c.dtype = SUBGEN_DTYPE_BF16;
    return subgen_create_ex(&c);
}

void subgen_destroy(subgen_t* h) {
    if (!h) return;
    cudaStreamSynchronize(h->st);
    for (cudaEvent_t e : h->ev) cudaEventDestroy(e);
    for (cudaEvent_t e : h->pev) cudaEventDestroy(e);
    destroy_side_stream(h);
    if (h->owns) cudaFree(h->ws);
    if (h->scratch) cudaFree(h->scratch);
    if (h->done_host) cudaFreeHost((void*)h->done_host);
    delete h;
}

int subgen_prefill(subgen_t* h, const void* K, const void* V, int n) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_prefill: handle is NULL");
    if (n < 0) return fail(SUBGEN_EINVAL, "subgen_prefill: n must be >= 0");
    if (n == 0) return SUBGEN_OK;
    if (!K || !V) return fail(SUBGEN_EINVAL, "subgen_prefill: K and V must not be NULL");
    for (int b = 0; b < h->d.B; ++b)
        if ((long long)h->n_host[b] + n > INT_MAX - 1) return fail(SUBGEN_ESTATE, "subgen_prefill: stream too long");
    std::vector<int> add(h->d.B, n);
    int rc = launch_prefill(h, K, V, n, nullptr, 0, add.data());
    if (rc) return rc;
    h->epoch_stale = true;
    h->search_ready = false;
    rank_units(h);
    for (int b = 0; b < h->d.B; ++b) h->n_host[b] += n;
    return SUBGEN_OK;
}

int subgen_prefill_varlen(subgen_t* h, const void* K, const void* V, const int* cu) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_prefill_varlen: handle is NULL");
    if (!cu) return fail(SUBGEN_EINVAL, "subgen_prefill_varlen: cu_seqlens is NULL");
    if (cu[0] != 0) return fail(SUBGEN_EINVAL, "subgen_prefill_varlen: cu_seqlens[0] must be 0");
    for (int b = 0; b < h->d.B; ++b) {
        if (cu[b + 1] < cu[b]) return fail(SUBGEN_EINVAL, "subgen_prefill_varlen: cu_seqlens must be non-decreasing");
        if ((long long)h->n_host[b] + (cu[b + 1] - cu[b]) > INT_MAX - 1)
            return fail(SUBGEN_ESTATE, "subgen_prefill_varlen: stream too long");
    }
    const int total = cu[h->d.B];
    if (total == 0) return SUBGEN_OK;
    if (!K || !V) return fail(SUBGEN_EINVAL, "subgen_prefill_varlen: K and V must not be NULL");
    int* cu_dev = (int*)(h->ws + h->L.cu);
    // the offsets are consumed by the kernel launched right after, in stream order
    CUDA_TRY(cudaMemcpyAsync(cu_dev, cu, sizeof(int) * (h->d.B + 1), cudaMemcpyHostToDevice, h->st));
    CUDA_TRY(cudaStreamSynchronize(h->st));   // cu may be pageable host memory reused by the caller
    std::vector<int> add(h->d.B);
    for (int b = 0; b < h->d.B; ++b) add[b] = cu[b + 1] - cu[b];
    int rc = launch_prefill(h, K, V, 0, cu_dev, total, add.data());
    if (rc) return rc;
    h->epoch_stale = true;
    h->search_ready = false;
    rank_units(h);
    for (int b = 0; b < h->d.B; ++b) h->n_host[b] += cu[b + 1] - cu[b];
    return SUBGEN_OK;
}

int subgen_step(subgen_t* h, const void* q, const void* k, const void* v, void* out) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_step: handle is NULL");
    if (!q || !k || !v || !out) return fail(SUBGEN_EINVAL, "subgen_step: q, k, v, out must not be NULL");
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15)
        return fail(SUBGEN_EINVAL, "subgen_step: pointers must be 16-byte aligned");
    for (int b = 0; b < h->d.B; ++b)
        if (h->n_host[b] >= INT_MAX - 1) return fail(SUBGEN_ESTATE, "subgen_step: stream too long");
    int rc = launch_step(h, q, k, v, out);
    if (rc) return rc;
    for (int b = 0; b < h->d.B; ++b) h->n_host[b] += 1;
    return SUBGEN_OK;
}

int subgen_query(subgen_t* h, const void* q, int nq, void* out) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_query: handle is NULL");
    if (!q || !out) return fail(SUBGEN_EINVAL, "subgen_query: q and out must not be NULL");
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(SUBGEN_EINVAL, "subgen_query: pointers must be 16-byte aligned");
    const int cols = h->d.G * nq;
    if (nq < 1 || (nq & (nq - 1)) || cols > h->d.Gs)
        return fail(SUBGEN_EINVAL, "subgen_query: nq must be a power of two with (H / Hkv) * nq <= %d (set nq_max at creation)", h->d.Gs);
    for (int b = 0; b < h->d.B; ++b)
        if (h->n_host[b] == 0) return fail(SUBGEN_ESTATE, "subgen_query: sequence %d has no tokens yet", b);
    const bool f32 = h->cfg.dtype == SUBGEN_DTYPE_FP32;
    if (h->d.D == 64) return f32 ? launch_query_only_td<float, 64>(h, q, nq, out) : launch_query_only_td<__nv_bfloat16, 64>(h, q, nq, out);
    return f32 ? launch_query_only_td<float, 128>(h, q, nq, out) : launch_query_only_td<__nv_bfloat16, 128>(h, q, nq, out);
}

// q, k, v from mapped host memory into the handle's staging buffers, 16 bytes per thread.
__global__ void stage_inputs_kernel(const uint4* __restrict__ q, const uint4* __restrict__ k, const uint4* __restrict__ v,
                                    uint4* dq, uint4* dk, uint4* dv, size_t nq, size_t nk) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nq) dq[i] = q[i];
    else if (i < nq + nk) dk[i - nq] = k[i - nq];
    else if (i < nq + 2 * nk) dv[i - nq - nk] = v[i - nq - nk];
}

// Device-side alias of a page-locked, mapped host buffer (what cudaHostAlloc / cudaHostRegister hand out under unified
// addressing); false for pageable memory.
static bool pinned_alias(const void* host, void** dev) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) { cudaGetLastError(); return false; }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return false;
    *dev = a.devicePointer;
    return true;
}

// cuStreamWriteValue32 of the driver, looked up once (NULL if this driver does not offer it).
typedef CUresult (*stream_write32_fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
static stream_write32_fn stream_write32() {
    static stream_write32_fn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &p, cudaEnableDefault, &qr) != cudaSuccess || qr != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            p = nullptr;
        }
        return (stream_write32_fn)p;
    }();
    return fn;
}

// Wait until the stream has finished the step just enqueued. Instead of a stream synchronisation the stream itself
// writes a sequence number into a pinned word once the step's kernels are done (a stream memory operation), and the
// host spins on that word: the result is seen a few microseconds earlier. Falls back to cudaStreamSynchronize when the
// driver has no such operation, and after a bounded spin.
// behind: called once the completion word has been enqueued (or, without one, after the synchronisation): work for
// the stream that the host does not wait for.
static cudaError_t wait_step_done(subgen* h, void (*behind)(subgen*) = nullptr) {
    stream_write32_fn wr = stream_write32();
    if (wr && !h->done_host) {
        void* p = nullptr;
        if (cudaHostAlloc(&p, 64, cudaHostAllocMapped) == cudaSuccess) {
            void* dp = nullptr;
            if (cudaHostGetDevicePointer(&dp, p, 0) == cudaSuccess) {
                h->done_host = (volatile unsigned*)p;
                h->done_host[0] = 0;
                h->done_dev = (CUdeviceptr)(uintptr_t)dp;
            } else {
                cudaFreeHost(p);
            }
        }
        cudaGetLastError();
    }
    if (wr && h->done_host) {
        const unsigned seq = ++h->done_seq;
        if (wr((CUstream)h->st, h->done_dev, seq, 0) == CUDA_SUCCESS) {
            if (behind) behind(h);
            for (long long spin = 0; spin < (1ll << 27); ++spin)
                if (h->done_host[0] == seq) return cudaGetLastError();
            return cudaStreamSynchronize(h->st);
        }
    }
    const cudaError_t e = cudaStreamSynchronize(h->st);
    if (behind && e == cudaSuccess) behind(h);
    return e;
}

// Three-kernel steps of bf16 handles (not bounded, window of one row or more): the search for the nearest
// representative of the token that the NEXT step takes out of the window, enqueued behind a host-buffer step and its
// completion word, where it runs while the host has the result and prepares its next call; that step then launches
// the insertion kernel in its apply-only mode. A host-buffer step cannot overlap with its successor, so without this
// the whole search stands in front of every step's scans (256 units: 2 to 5 % more calls per second, depending on how
// long the host takes between calls; launched in front of the completion word, beside the value scan, it delayed the
// word by its own completion and gained 1 %).
static void search_ahead(subgen* h) {
    static const bool off = [] { const char* e = getenv("SUBGEN_SEARCH_AHEAD"); return e && e[0] == '0'; }();
    if (off || h->cfg.dtype != SUBGEN_DTYPE_BF16 || h->fused || h->cfg.bounded || h->d.w < 1 || h->epoch_stale) return;
    Cache<__nv_bfloat16> C = make_cache<__nv_bfloat16>(h);
    const dim3 grid(h->d.sp_insert, h->d.U);
    const __nv_bfloat16* none = nullptr;
    if (h->d.D == 64) launch_pdl(insert_mma_kernel<64, false, 1>, grid, dim3(kInsertMmaThreads), h->st, C, none, none);
    else launch_pdl(insert_mma_kernel<128, false, 1>, grid, dim3(kInsertMmaThreads), h->st, C, none, none);
    if (take_launch_error() != cudaSuccess) return;
    h->launches += 1;
    h->search_ready = true;
}

int subgen_step_host(subgen_t* h, const void* q, const void* k, const void* v, void* out) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_step_host: handle is NULL");
    if (!q || !k || !v || !out) return fail(SUBGEN_EINVAL, "subgen_step_host: q, k, v, out must not be NULL");
    const size_t row = (size_t)h->d.D * h->d.E;
    const size_t qb = (size_t)h->d.B * h->d.H * row, kb = (size_t)h->d.U * row;
    void *dq, *dk, *dv, *dout;
    if (pinned_alias(q, &dq) && pinned_alias(k, &dk) && pinned_alias(v, &dv) && pinned_alias(out, &dout) &&
        !(((uintptr_t)dq | (uintptr_t)dk | (uintptr_t)dv | (uintptr_t)dout) & 15)) {
        // pinned buffers: the step's kernels read the inputs and write the result across the bus themselves
        // (each input row is read by the few blocks of its unit, the result is written once)
        // A one-kernel step with many blocks per unit would fetch every input row across the bus once per block
        // (8 units, 37 blocks each: 88 -> 65 us per call with staging); then one small kernel brings q, k, v over
        // first, every 16-byte piece once, and the step reads device memory. The result is still written into the
        // caller's buffer by the step itself. With few blocks per unit the direct reads are as fast (measured at 256
        // units x 3 blocks and 32 units x 9 blocks). SUBGEN_E2E_STAGE=0 / 1 forces either way.
        static const int stage_env = [] { const char* e = getenv("SUBGEN_E2E_STAGE"); return e ? atoi(e) : -1; }();
        const bool stage = stage_env >= 0 ? stage_env != 0 : (h->fused && h->d.sp_fused > 16);
        if (stage) {
            char* w = h->ws;
            const size_t nq = qb / 16, nk = kb / 16, total = nq + 2 * nk;
            stage_inputs_kernel<<<(unsigned)((total + 255) / 256), 256, 0, h->st>>>(
                (const uint4*)dq, (const uint4*)dk, (const uint4*)dv, (uint4*)(w + h->L.stage_q), (uint4*)(w + h->L.stage_k),
                (uint4*)(w + h->L.stage_v), nq, nk);
            h->launches += 1;
            int rc = subgen_step(h, w + h->L.stage_q, w + h->L.stage_k, w + h->L.stage_v, dout);
            if (rc) return rc;
            CUDA_TRY(wait_step_done(h));
            return SUBGEN_OK;
        }
        int rc = subgen_step(h, dq, dk, dv, dout);
        if (rc) return rc;
        CUDA_TRY(wait_step_done(h, search_ahead));
        return SUBGEN_OK;
    }
    char* w = h->ws;
    CUDA_TRY(cudaMemcpyAsync(w + h->L.stage_q, q, qb, cudaMemcpyHostToDevice, h->st));
    CUDA_TRY(cudaMemcpyAsync(w + h->L.stage_k, k, kb, cudaMemcpyHostToDevice, h->st));
    CUDA_TRY(cudaMemcpyAsync(w + h->L.stage_v, v, kb, cudaMemcpyHostToDevice, h->st));
    int rc = subgen_step(h, w + h->L.stage_q, w + h->L.stage_k, w + h->L.stage_v, w + h->L.stage_out);
    if (rc) return rc;
    CUDA_TRY(cudaMemcpyAsync(out, w + h->L.stage_out, qb, cudaMemcpyDeviceToHost, h->st));
    CUDA_TRY(cudaStreamSynchronize(h->st));
    return SUBGEN_OK;
}

int subgen_status(subgen_t* h) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_status: handle is NULL");
    std::vector<int> st(h->d.U);
    CUDA_TRY(cudaStreamSynchronize(h->st));
    CUDA_TRY(cudaMemcpy(st.data(), h->ws + h->L.status, sizeof(int) * h->d.U, cudaMemcpyDeviceToHost));
    int r = 0;
    for (int x : st) r |= x;
    return r;
}

int subgen_export_state(subgen_t* h, int seq, int kvhead, subgen_state_view* v) {
    if (!h || !v) return fail(SUBGEN_EINVAL, "subgen_export_state: NULL argument");
    if (seq < 0 || seq >= h->d.B || kvhead < 0 || kvhead >= h->d.Hkv)
        return fail(SUBGEN_EINVAL, "subgen_export_state: unit out of range");
    const size_t u = (size_t)seq * h->d.Hkv + kvhead;
    const Dims& d = h->d;
    char* w = h->ws;
    CUDA_TRY(cudaStreamSynchronize(h->st));
    auto get = [&](void* dst, size_t off, size_t bytes) { return cudaMemcpy(dst, w + off, bytes, cudaMemcpyDeviceToHost); };
    CUDA_TRY(get(&v->n, h->L.n_unit + u * 4, 4));
    CUDA_TRY(get(&v->m, h->L.m_unit + u * 4, 4));
    CUDA_TRY(get(&v->status, h->L.status + u * 4, 4));
    CUDA_TRY(get(&v->mu, h->L.mu + u * 8, 8));
    CUDA_TRY(get(&v->last_cluster, h->L.last_cid + u * 4, 4));
    CUDA_TRY(get(&v->last_opened, h->L.last_open + u * 4, 4));
    CUDA_TRY(get(&v->last_d2, h->L.last_d2 + u * 8, 8));
    v->inserted = v->n > d.w ? v->n - d.w : 0;
    if (h->cfg.bounded) {
        CUDA_TRY(get(&v->threshold2, h->L.thr2 + u * 8, 8));
        CUDA_TRY(get(&v->doublings, h->L.level + u * 4, 4));
    } else {
        v->threshold2 = (uint64_t)floor((double)h->cfg.delta * (double)h->cfg.delta * 4294967296.0);
        v->doublings = 0;
    }
    if (v->counts) CUDA_TRY(get(v->counts, h->L.cnt + u * d.m_max * 4, (size_t)d.m_max * 4));
    if (v->centre_tok) CUDA_TRY(get(v->centre_tok, h->L.ctok + u * d.m_max * 4, (size_t)d.m_max * 4));
    if (v->slot_tok) CUDA_TRY(get(v->slot_tok, h->L.stok + u * d.m_max * d.t * 4, (size_t)d.m_max * d.t * 4));
    if (v->m_tok) CUDA_TRY(get(v->m_tok, h->L.Mtok + u * d.s * 4, (size_t)d.s * 4));
    if (v->m_w) CUDA_TRY(get(v->m_w, h->L.MW + u * d.s * 8, (size_t)d.s * 8));
    return SUBGEN_OK;
}

int subgen_export_rows(subgen_t* h, int seq, int kvhead, int which, void* host, size_t bytes) {
    if (!h || !host) return fail(SUBGEN_EINVAL, "subgen_export_rows: NULL argument");
    if (seq < 0 || seq >= h->d.B || kvhead < 0 || kvhead >= h->d.Hkv)
        return fail(SUBGEN_EINVAL, "subgen_export_rows: unit out of range");
    const Dims& d = h->d;
    const size_t u = (size_t)seq * d.Hkv + kvhead, row = (size_t)d.D * d.E;
    size_t off, need;
    switch (which) {
        case 0: need = d.m_max * row; off = h->L.X + u * need; break;
        case 1: need = (size_t)d.m_max * d.t * row; off = h->L.S + u * need; break;
        case 2: need = d.s * row; off = h->L.Mk + u * need; break;
        case 3: need = d.s * row; off = h->L.Mv + u * need; break;
        case 4: need = d.w * row; off = h->L.ringK + u * need; break;
        case 5: need = d.w * row; off = h->L.ringV + u * need; break;
        default: return fail(SUBGEN_EINVAL, "subgen_export_rows: which must be 0..5");
    }
    if (bytes < need) return fail(SUBGEN_EINVAL, "subgen_export_rows: buffer needs %zu bytes", need);
    CUDA_TRY(cudaStreamSynchronize(h->st));
    if (need) CUDA_TRY(cudaMemcpy(host, h->ws + off, need, cudaMemcpyDeviceToHost));
    return SUBGEN_OK;
}

int subgen_cache_stats(subgen_t* h, subgen_stats* out) {
    if (!h || !out) return fail(SUBGEN_EINVAL, "subgen_cache_stats: NULL argument");
    unsigned long long* dev = (unsigned long long*)(h->ws + h->L.stats);
    CUDA_TRY(cudaMemsetAsync(dev, 0, 8 * sizeof(uint64_t), h->st));
    if (h->cfg.dtype == SUBGEN_DTYPE_FP32) stats_kernel<float><<<h->d.U, 256, 0, h->st>>>(make_cache<float>(h), h->d.U, dev);
    else stats_kernel<__nv_bfloat16><<<h->d.U, 256, 0, h->st>>>(make_cache<__nv_bfloat16>(h), h->d.U, dev);
    CUDA_TRY(take_launch_error());
    h->launches += 1;
    uint64_t r[8];
    CUDA_TRY(cudaMemcpyAsync(r, dev, sizeof r, cudaMemcpyDeviceToHost, h->st));
    CUDA_TRY(cudaStreamSynchronize(h->st));
    const uint64_t row = (uint64_t)h->d.D * h->d.E;
    out->units = h->d.U;
    out->clusters = r[0]; out->singleton_clusters = r[1]; out->m_filled = r[2]; out->window_rows = r[3]; out->tokens = r[4];
    out->prefill_pairs = r[5];
    // bf16: packed heads and their norms (full rows only for the few representatives the heads do not rule out);
    // fp32: the exact scan reads the full rows
    out->insert_bytes = h->cfg.dtype == SUBGEN_DTYPE_BF16 ? r[0] * ((uint64_t)kHeadDims * h->d.E + 4) : r[0] * row;
    // bf16: the cluster scan fetches every distinct sampled row once (slots that repeat a token are read from their
    // first copy) plus counts and alias rows; fp32: all t rows of every cluster with more than one member
    out->distinct_sample_rows = r[6];
    out->cluster_bytes = h->cfg.dtype == SUBGEN_DTYPE_BF16
                             ? (r[1] + r[6]) * row + r[0] * (4 + (uint64_t)h->d.t)
                             : (r[1] + (r[0] - r[1]) * (uint64_t)h->d.t) * row + r[0] * 4;
    out->value_bytes = (2 * r[2] + 2 * r[3]) * row + (uint64_t)h->d.U * h->d.s * 4;
    out->query_bytes = out->cluster_bytes + out->value_bytes;
    return SUBGEN_OK;
}

int subgen_profile_enable(subgen_t* h, int on) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_profile_enable: handle is NULL");
    h->prof = on != 0;
    return SUBGEN_OK;
}

int subgen_profile_read(subgen_t* h, double* ms, int* steps) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_profile_read: handle is NULL");
    CUDA_TRY(cudaStreamSynchronize(h->st));
    double acc[3] = {0, 0, 0};
    for (size_t i = 0; i + 4 <= h->ev_used; i += 4) {
        for (int k = 0; k < 3; ++k) {
            float x = 0;
            CUDA_TRY(cudaEventElapsedTime(&x, h->ev[i + k], h->ev[i + k + 1]));
            acc[k] += x;
        }
    }
    if (ms) { ms[0] = acc[0]; ms[1] = acc[1]; ms[2] = acc[2]; }
    if (steps) *steps = (int)(h->ev_used / 4);
    h->ev_used = 0;
    return SUBGEN_OK;
}

int subgen_profile_prefill_read(subgen_t* h, double* ms) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_profile_prefill_read: handle is NULL");
    CUDA_TRY(cudaStreamSynchronize(h->st));
    double acc[3] = {0, 0, 0};
    if (h->pev_used >= 2) {
        float x = 0;
        CUDA_TRY(cudaEventElapsedTime(&x, h->pev[0], h->pev[1]));
        acc[0] = x;
        if (h->pf_persist && h->pev_used >= 3) {
            // one kernel for all chunks: its wall time, split in the proportion of the time the units' blocks spent
            // scoring (staging included) and resolving
            float wall = 0;
            CUDA_TRY(cudaEventElapsedTime(&wall, h->pev[1], h->pev[2]));
            std::vector<unsigned long long> ns((size_t)h->d.U * kPpPhases);
            CUDA_TRY(cudaMemcpy(ns.data(), h->pf_phase_dev, ns.size() * 8, cudaMemcpyDeviceToHost));
            double ph[kPpPhases] = {0};
            for (int u = 0; u < h->d.U; ++u)
                for (int i = 0; i < kPpPhases; ++i) ph[i] += (double)ns[(size_t)kPpPhases * u + i];
            const double sc = ph[0] + ph[1] + ph[2] + ph[3] + ph[4], rs = ph[5] + ph[6] + ph[7];
            if (getenv("SUBGEN_TRACE"))
                fprintf(stderr, "subgen prefill phases (share of block time): stage %.3f wait %.3f readback %.3f store+issue %.3f "
                        "follow-up %.3f | openings %.3f ranks+coins %.3f writes %.3f; mean block cycles %.0f\n",
                        ph[0] / (sc + rs), ph[1] / (sc + rs), ph[2] / (sc + rs), ph[3] / (sc + rs), ph[4] / (sc + rs),
                        ph[5] / (sc + rs), ph[6] / (sc + rs), ph[7] / (sc + rs), (sc + rs) / h->d.U);
            if (sc + rs > 0) { acc[1] = wall * sc / (sc + rs); acc[2] = wall * rs / (sc + rs); }
        } else {
            for (size_t i = 1; i + 2 < h->pev_used; i += 2) {       // chunk: events i -> i+1 (score) -> i+2 (resolve)
                float sc = 0, rs = 0;
                CUDA_TRY(cudaEventElapsedTime(&sc, h->pev[i], h->pev[i + 1]));
                CUDA_TRY(cudaEventElapsedTime(&rs, h->pev[i + 1], h->pev[i + 2]));
                acc[1] += sc;
                acc[2] += rs;
            }
        }
    }
    if (ms) { ms[0] = acc[0]; ms[1] = acc[1]; ms[2] = acc[2]; }
    h->pev_used = 0;
    return SUBGEN_OK;
}

uint64_t subgen_launch_count(const subgen_t* h) { return h ? h->launches : 0; }

int subgen_step_kernels(const subgen_t* h) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_step_kernels: handle is NULL");
    return h->cfg.dtype == SUBGEN_DTYPE_FP32 ? 2 : (h->fused ? 1 : 3);
}

}  // extern "C"


// ---- checkpoint: a handle's state as one host blob --------------------------------------------------------

namespace {

constexpr uint64_t kCkptMagic = 0x315450434e474253ull;   // "SBGNCPT1"

struct CkptHeader {
    uint64_t magic;
    uint32_t version, dtype;
    int32_t B, H, Hkv, d, t, s, window, m_rows;
    float delta;
    uint32_t pad;
    uint64_t seed, payload_bytes;
    int32_t unit_stride, unit_offset;      // numbering of the units in the Philox counter (resolved: stride >= Hkv)
};

struct CkptArray {
    size_t off;        // offset in the workspace
    size_t unit_cap;   // bytes per unit in the workspace
    size_t unit_live;  // bytes per unit stored in the blob
};

// The arrays that make up the state between two calls, in blob order. Cluster arrays are stored up to m_rows
// clusters per unit; partials, tickets and work queues are scratch of a single call and are not part of it.
std::vector<CkptArray> ckpt_arrays(const Dims& d, const Layout& L, int m_rows) {
    const size_t row = (size_t)d.D * d.E, mm = (size_t)d.m_max, mr = (size_t)m_rows, s = (size_t)d.s, w = (size_t)d.w, t = (size_t)d.t;
    return {
        {L.X, mm * row, mr * row}, {L.S, mm * t * row, mr * t * row}, {L.xn, mm * 4, mr * 4}, {L.cnt, mm * 4, mr * 4},
        {L.Xh, mm * kHeadDims * d.E, mr * kHeadDims * d.E}, {L.xhn, mm * 4, mr * 4}, {L.alias, mm * t, mr * t}, {L.ndist, mm, mr},
        {L.ctok, mm * 4, mr * 4}, {L.stok, mm * t * 4, mr * t * 4},
        {L.Mk, s * row, s * row}, {L.Mv, s * row, s * row}, {L.MW, s * 8, s * 8}, {L.Mtok, s * 4, s * 4}, {L.MinvW, s * 4, s * 4},
        {L.ringK, w * row, w * row}, {L.ringV, w * row, w * row},
        {L.n_unit, 4, 4}, {L.m_unit, 4, 4}, {L.mu, 8, 8}, {L.status, 4, 4}, {L.last_cid, 4, 4}, {L.last_open, 4, 4},
        {L.last_d2, 8, 8}, {L.pairs, 8, 8}, {L.thr2, 8, 8}, {L.level, 4, 4},
    };
}

std::vector<CkptArray> ckpt_arrays(const subgen* h, int m_rows) { return ckpt_arrays(h->d, h->L, m_rows); }

size_t ckpt_payload(const subgen* h, int m_rows) {
    size_t n = 0;
    for (const CkptArray& a : ckpt_arrays(h, m_rows)) n += a.unit_live * (size_t)h->d.U;
    return n;
}

// Largest cluster count over the units. Synchronous.
int ckpt_m_rows(subgen* h, int* out) {
    std::vector<int> m(h->d.U);
    CUDA_TRY(cudaStreamSynchronize(h->st));
    CUDA_TRY(cudaMemcpy(m.data(), h->ws + h->L.m_unit, (size_t)h->d.U * 4, cudaMemcpyDeviceToHost));
    int r = 0;
    for (int x : m) r = x > r ? x : r;
    *out = r;
    return SUBGEN_OK;
}

}  // namespace

extern "C" {

int subgen_checkpoint_bytes(subgen_t* h, size_t* bytes) {
    if (!h || !bytes) return fail(SUBGEN_EINVAL, "subgen_checkpoint_bytes: NULL argument");
    int m_rows = 0;
    if (int rc = ckpt_m_rows(h, &m_rows)) return rc;
    *bytes = sizeof(CkptHeader) + ckpt_payload(h, m_rows);
    return SUBGEN_OK;
}

int subgen_checkpoint_save(subgen_t* h, void* host, size_t bytes, size_t* written) {
    if (!h || !host) return fail(SUBGEN_EINVAL, "subgen_checkpoint_save: NULL argument");
    int m_rows = 0;
    if (int rc = ckpt_m_rows(h, &m_rows)) return rc;
    const size_t payload = ckpt_payload(h, m_rows), need = sizeof(CkptHeader) + payload;
    if (bytes < need) return fail(SUBGEN_EINVAL, "subgen_checkpoint_save: buffer needs %zu bytes", need);
    CkptHeader hd;
    memset(&hd, 0, sizeof hd);
    hd.magic = kCkptMagic; hd.version = 2; hd.dtype = (uint32_t)h->cfg.dtype;
    hd.B = h->d.B; hd.H = h->d.H; hd.Hkv = h->d.Hkv; hd.d = h->d.D; hd.t = h->d.t; hd.s = h->d.s; hd.window = h->d.w;
    hd.m_rows = m_rows; hd.delta = h->cfg.delta; hd.seed = h->cfg.seed; hd.payload_bytes = payload;
    hd.pad = h->cfg.bounded ? 1u : 0u;
    hd.unit_stride = h->cfg.unit_stride ? h->cfg.unit_stride : h->d.Hkv; hd.unit_offset = h->cfg.unit_offset;
    memcpy(host, &hd, sizeof hd);
    char* dst = (char*)host + sizeof hd;
    for (const CkptArray& a : ckpt_arrays(h, m_rows)) {
        if (a.unit_live)
            CUDA_TRY(cudaMemcpy2D(dst, a.unit_live, h->ws + a.off, a.unit_cap, a.unit_live, (size_t)h->d.U, cudaMemcpyDeviceToHost));
        dst += a.unit_live * (size_t)h->d.U;
    }
    if (written) *written = need;
    return SUBGEN_OK;
}

int subgen_checkpoint_load(subgen_t* h, const void* host, size_t bytes) {
    if (!h || !host) return fail(SUBGEN_EINVAL, "subgen_checkpoint_load: NULL argument");
    if (bytes < sizeof(CkptHeader)) return fail(SUBGEN_EINVAL, "subgen_checkpoint_load: blob shorter than its header");
    CkptHeader hd;
    memcpy(&hd, host, sizeof hd);
    if (hd.magic != kCkptMagic || hd.version != 2) return fail(SUBGEN_EINVAL, "subgen_checkpoint_load: not a checkpoint of this library version");
    const Dims& d = h->d;
    if (hd.B != d.B || hd.H != d.H || hd.Hkv != d.Hkv || hd.d != d.D || hd.t != d.t || hd.s != d.s || hd.window != d.w ||
        (int)hd.dtype != h->cfg.dtype || hd.seed != h->cfg.seed || memcmp(&hd.delta, &h->cfg.delta, sizeof(float)) != 0 ||
        hd.pad != (h->cfg.bounded ? 1u : 0u) || hd.unit_stride != (h->cfg.unit_stride ? h->cfg.unit_stride : d.Hkv) ||
        hd.unit_offset != h->cfg.unit_offset)
        return fail(SUBGEN_EINVAL, "subgen_checkpoint_load: the checkpoint was written with another configuration "
                    "(B, H, Hkv, d, t, s, window, dtype, delta, seed, the bounded flag and the unit numbering must match; "
                    "only m_max may differ)");
    if (hd.m_rows < 0 || hd.m_rows > d.m_max)
        return fail(SUBGEN_EINVAL, "subgen_checkpoint_load: the checkpoint holds %d clusters per unit, this handle's m_max is %d", hd.m_rows, d.m_max);
    const size_t payload = ckpt_payload(h, hd.m_rows);
    if (hd.payload_bytes != payload || bytes < sizeof hd + payload) return fail(SUBGEN_EINVAL, "subgen_checkpoint_load: truncated or damaged blob");
    CUDA_TRY(cudaStreamSynchronize(h->st));
    // back to the state of a new handle, then the stored arrays on top
    CUDA_TRY(cudaMemset(h->ws + h->L.book_begin, 0, h->L.book_end - h->L.book_begin));
    CUDA_TRY(cudaMemset(h->ws + h->L.book_end, 0xFF, h->L.total - h->L.book_end));
    const char* src = (const char*)host + sizeof hd;
    for (const CkptArray& a : ckpt_arrays(h, hd.m_rows)) {
        if (a.unit_live)
            CUDA_TRY(cudaMemcpy2D(h->ws + a.off, a.unit_cap, src, a.unit_live, a.unit_live, (size_t)d.U, cudaMemcpyHostToDevice));
        src += a.unit_live * (size_t)d.U;
    }
    std::vector<int> n(d.U);
    CUDA_TRY(cudaMemcpy(n.data(), h->ws + h->L.n_unit, (size_t)d.U * 4, cudaMemcpyDeviceToHost));
    for (int b = 0; b < d.B; ++b) h->n_host[b] = n[(size_t)b * d.Hkv];
    h->epoch_stale = true;
    h->search_ready = false;
    h->order_ready = false;
    return SUBGEN_OK;
}

int subgen_grow(subgen_t* h, int m_max, void* workspace, size_t workspace_bytes) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_grow: handle is NULL");
    if (h->cfg.bounded) return fail(SUBGEN_ESTATE, "subgen_grow: m_max of a bounded handle is its budget and stays as created");
    if (m_max <= h->d.m_max) return fail(SUBGEN_EINVAL, "subgen_grow: m_max must exceed the current %d", h->d.m_max);
    Dims d2 = h->d;
    d2.m_max = m_max;
    const Layout L2 = make_layout(d2);
    int m_rows = 0;
    if (int rc = ckpt_m_rows(h, &m_rows)) return rc;                 // synchronises the stream
    char* ws2 = (char*)workspace;
    cudaError_t e = cudaSuccess;
    if (workspace) {
        if (workspace_bytes < L2.total || ((uintptr_t)workspace % kAlign))
            return fail(SUBGEN_ENOMEM, "subgen_grow: workspace needs %zu bytes, 256-byte aligned (got %zu)", L2.total, workspace_bytes);
        if (ws2 < h->ws + h->L.total && h->ws < ws2 + L2.total) return fail(SUBGEN_EINVAL, "subgen_grow: the new workspace overlaps the old one");
    } else {
        e = cudaMalloc((void**)&ws2, L2.total);
        if (e != cudaSuccess) return fail(SUBGEN_ENOMEM, "subgen_grow: cudaMalloc(%zu) failed: %s", L2.total, cudaGetErrorString(e));
    }
    // a new handle's workspace, then the state arrays on top: every array keeps its per-unit layout, only the room
    // per unit changes, so each is one strided device copy
    e = cudaMemsetAsync(ws2 + L2.book_begin, 0, L2.book_end - L2.book_begin, h->st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ws2 + L2.book_end, 0xFF, L2.total - L2.book_end, h->st);
    const std::vector<CkptArray> from = ckpt_arrays(h->d, h->L, m_rows), to = ckpt_arrays(d2, L2, m_rows);
    for (size_t i = 0; i < from.size() && e == cudaSuccess; ++i)
        if (from[i].unit_live)
            e = cudaMemcpy2DAsync(ws2 + to[i].off, to[i].unit_cap, h->ws + from[i].off, from[i].unit_cap, from[i].unit_live,
                                  (size_t)h->d.U, cudaMemcpyDeviceToDevice, h->st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->st);
    if (e != cudaSuccess) {
        if (!workspace) cudaFree(ws2);
        return fail(SUBGEN_ECUDA, "subgen_grow: %s", cudaGetErrorString(e));
    }
    if (h->owns) cudaFree(h->ws);
    h->owns = workspace == nullptr;
    h->cfg.workspace = workspace;
    h->cfg.workspace_bytes = workspace ? workspace_bytes : 0;
    h->ws = ws2;
    h->L = L2;
    h->d = d2;
    h->cfg.m_max = m_max;
    h->epoch_stale = true;
    h->search_ready = false;
    h->order_ready = false;
    return SUBGEN_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Exact comparison path.

struct subgen_exact {
    int B, H, Hkv, G, D, n_max, dtype, U, splits;
    size_t E;
    char *Kc = nullptr, *Vc = nullptr, *misc = nullptr;
    size_t off_n, off_part, off_ticket, off_cu, off_q, off_pos, off_tok, misc_bytes;
    uint64_t kc_counters[2] = {0, 0};   // last compression: tokens looked at, full rows read
    cudaStream_t st = nullptr;
    std::vector<int> n_host;
    uint64_t launches = 0;
};

namespace {

template <typename T> ExactCache<T> make_exact(const subgen_exact* h) {
    ExactCache<T> E;
    E.B = h->B; E.H = h->H; E.Hkv = h->Hkv; E.G = h->G; E.n_max = h->n_max;
    E.Kc = (T*)h->Kc; E.Vc = (T*)h->Vc;
    E.n_unit = (int*)(h->misc + h->off_n);
    E.part = (float*)(h->misc + h->off_part);
    E.ticket = (unsigned*)(h->misc + h->off_ticket);
    E.qnext = (unsigned*)(h->misc + h->off_q);
    E.pos = (int*)(h->misc + h->off_pos);
    E.tok = (int*)(h->misc + h->off_tok);
    return E;
}

template <typename T, int D>
int exact_append_td(subgen_exact* h, const void* K, const void* V, int n, const int* cu_dev, int total, int longest) {
    ExactCache<T> E = make_exact<T>(h);
    int bx = (int)(((size_t)longest * (D / Elem<T>::EPL) + 255) / 256);
    bx = bx < 1 ? 1 : (bx > 64 ? 64 : bx);
    exact_append_kernel<T, D><<<dim3(bx, h->U), 256, 0, h->st>>>(E, (const T*)K, (const T*)V, n, cu_dev, total);
    exact_advance_kernel<T><<<(h->U + 255) / 256, 256, 0, h->st>>>(E, h->U, n, cu_dev);
    CUDA_TRY(take_launch_error());
    h->launches += 2;
    return SUBGEN_OK;
}

int exact_append(subgen_exact* h, const void* K, const void* V, int n, const int* cu_dev, int total, int longest) {
    const bool f32 = h->dtype == SUBGEN_DTYPE_FP32;
    if (h->D == 64)
        return f32 ? exact_append_td<float, 64>(h, K, V, n, cu_dev, total, longest)
                   : exact_append_td<__nv_bfloat16, 64>(h, K, V, n, cu_dev, total, longest);
    return f32 ? exact_append_td<float, 128>(h, K, V, n, cu_dev, total, longest)
               : exact_append_td<__nv_bfloat16, 128>(h, K, V, n, cu_dev, total, longest);
}

template <typename T, int D>
int exact_step_td(subgen_exact* h, const void* q, const void* k, const void* v, void* out) {
    ExactCache<T> E = make_exact<T>(h);
    const dim3 grid(h->splits, h->U);
    switch (h->G) {
        case 1: exact_step_kernel<T, D, 1><<<grid, kQueryThreads, 0, h->st>>>(E, (const T*)q, (const T*)k, (const T*)v, (T*)out); break;
        case 2: exact_step_kernel<T, D, 2><<<grid, kQueryThreads, 0, h->st>>>(E, (const T*)q, (const T*)k, (const T*)v, (T*)out); break;
        case 4: exact_step_kernel<T, D, 4><<<grid, kQueryThreads, 0, h->st>>>(E, (const T*)q, (const T*)k, (const T*)v, (T*)out); break;
        default: exact_step_kernel<T, D, 8><<<grid, kQueryThreads, 0, h->st>>>(E, (const T*)q, (const T*)k, (const T*)v, (T*)out); break;
    }
    CUDA_TRY(take_launch_error());
    h->launches += 1;
    return SUBGEN_OK;
}

// bf16: append the step's token (k, v are [U, 1, d] in the dense layout), then the tensor-core scan.
template <int D>
int exact_step_mma(subgen_exact* h, const void* q, const void* k, const void* v, void* out) {
    typedef __nv_bfloat16 T;
    int rc = exact_append_td<T, D>(h, k, v, 1, nullptr, 0, 1);
    if (rc) return rc;
    ExactCache<T> E = make_exact<T>(h);
    const dim3 grid(h->splits, h->U);
    switch (h->G) {
        case 1: exact_mma_kernel<D, 1><<<grid, kQmThreads, 0, h->st>>>(E, (const T*)q, (T*)out); break;
        case 2: exact_mma_kernel<D, 2><<<grid, kQmThreads, 0, h->st>>>(E, (const T*)q, (T*)out); break;
        case 4: exact_mma_kernel<D, 4><<<grid, kQmThreads, 0, h->st>>>(E, (const T*)q, (T*)out); break;
        default: exact_mma_kernel<D, 8><<<grid, kQmThreads, 0, h->st>>>(E, (const T*)q, (T*)out); break;
    }
    CUDA_TRY(take_launch_error());
    h->launches += 1;
    return SUBGEN_OK;
}

}  // namespace

extern "C" {

subgen_exact_t* subgen_exact_create(int B, int H, int Hkv, int d, int n_max, int dtype, void* stream) {
    if (Hkv == 0) Hkv = H;
    if (B <= 0 || H <= 0 || Hkv <= 0 || H % Hkv || n_max <= 0 || (d != 64 && d != 128) ||
        (dtype != SUBGEN_DTYPE_FP32 && dtype != SUBGEN_DTYPE_BF16) || (long long)B * Hkv > 65535) {
        fail(SUBGEN_EINVAL, "subgen_exact_create: invalid argument");
        return nullptr;
    }
    const int G = H / Hkv;
    if (G != 1 && G != 2 && G != 4 && G != 8) { fail(SUBGEN_EINVAL, "subgen_exact_create: H / Hkv must be 1, 2, 4 or 8"); return nullptr; }
    if (check_device() != SUBGEN_OK) return nullptr;
    subgen_exact* h = new subgen_exact();
    h->B = B; h->H = H; h->Hkv = Hkv; h->G = G; h->D = d; h->n_max = n_max; h->dtype = dtype; h->U = B * Hkv;
    h->E = dtype == SUBGEN_DTYPE_FP32 ? 4 : 2;
    int sp = dtype == SUBGEN_DTYPE_BF16 ? (148 * 4) / h->U : (148 * 8 + h->U - 1) / h->U;   // bf16: one resident wave of 4 blocks/SM
    h->splits = sp < 1 ? 1 : (sp > 64 ? 64 : sp);
    h->st = (cudaStream_t)stream;
    const size_t cache = (size_t)h->U * n_max * d * h->E;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    h->off_n = take((size_t)h->U * 4);
    h->off_ticket = take((size_t)h->U * 4);
    h->off_q = take((size_t)h->U * 4);
    h->off_pos = take((size_t)h->U * 4);
    h->off_tok = take((size_t)h->U * n_max * 4);
    h->off_cu = take(((size_t)B + 1) * 4);
    h->off_part = take((size_t)h->U * h->splits * G * (d + 2) * 4);
    h->misc_bytes = off;
    if (cudaMalloc((void**)&h->Kc, cache) != cudaSuccess || cudaMalloc((void**)&h->Vc, cache) != cudaSuccess ||
        cudaMalloc((void**)&h->misc, h->misc_bytes) != cudaSuccess ||
        cudaMemsetAsync(h->misc, 0, h->misc_bytes, h->st) != cudaSuccess) {
        fail(SUBGEN_ENOMEM, "subgen_exact_create: allocating 2 x %zu bytes failed: %s", cache, cudaGetErrorString(cudaGetLastError()));
        cudaFree(h->Kc); cudaFree(h->Vc); cudaFree(h->misc);
        delete h;
        return nullptr;
    }
    h->n_host.assign(B, 0);
    return h;
}

void subgen_exact_destroy(subgen_exact_t* h) {
    if (!h) return;
    cudaStreamSynchronize(h->st);
    cudaFree(h->Kc); cudaFree(h->Vc); cudaFree(h->misc);
    delete h;
}

int subgen_exact_append(subgen_exact_t* h, const void* K, const void* V, int n) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_exact_append: handle is NULL");
    if (n < 0) return fail(SUBGEN_EINVAL, "subgen_exact_append: n must be >= 0");
    if (n == 0) return SUBGEN_OK;
    if (!K || !V) return fail(SUBGEN_EINVAL, "subgen_exact_append: K and V must not be NULL");
    for (int b = 0; b < h->B; ++b)
        if ((long long)h->n_host[b] + n > h->n_max) return fail(SUBGEN_ESTATE, "subgen_exact_append: cache capacity n_max exceeded");
    int rc = exact_append(h, K, V, n, nullptr, 0, n);
    if (rc) return rc;
    for (int b = 0; b < h->B; ++b) h->n_host[b] += n;
    return SUBGEN_OK;
}

int subgen_exact_append_varlen(subgen_exact_t* h, const void* K, const void* V, const int* cu) {
    if (!h || !cu) return fail(SUBGEN_EINVAL, "subgen_exact_append_varlen: NULL argument");
    if (cu[0] != 0) return fail(SUBGEN_EINVAL, "subgen_exact_append_varlen: cu_seqlens[0] must be 0");
    int longest = 0;
    for (int b = 0; b < h->B; ++b) {
        const int len = cu[b + 1] - cu[b];
        if (len < 0) return fail(SUBGEN_EINVAL, "subgen_exact_append_varlen: cu_seqlens must be non-decreasing");
        if ((long long)h->n_host[b] + len > h->n_max) return fail(SUBGEN_ESTATE, "subgen_exact_append_varlen: cache capacity n_max exceeded");
        longest = len > longest ? len : longest;
    }
    const int total = cu[h->B];
    if (total == 0) return SUBGEN_OK;
    if (!K || !V) return fail(SUBGEN_EINVAL, "subgen_exact_append_varlen: K and V must not be NULL");
    int* cu_dev = (int*)(h->misc + h->off_cu);
    CUDA_TRY(cudaMemcpyAsync(cu_dev, cu, sizeof(int) * (h->B + 1), cudaMemcpyHostToDevice, h->st));
    CUDA_TRY(cudaStreamSynchronize(h->st));
    int rc = exact_append(h, K, V, 0, cu_dev, total, longest);
    if (rc) return rc;
    for (int b = 0; b < h->B; ++b) h->n_host[b] += cu[b + 1] - cu[b];
    return SUBGEN_OK;
}

int subgen_exact_step(subgen_exact_t* h, const void* q, const void* k, const void* v, void* out) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_exact_step: handle is NULL");
    if (!q || !k || !v || !out) return fail(SUBGEN_EINVAL, "subgen_exact_step: q, k, v, out must not be NULL");
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15)
        return fail(SUBGEN_EINVAL, "subgen_exact_step: pointers must be 16-byte aligned");
    for (int b = 0; b < h->B; ++b)
        if (h->n_host[b] >= h->n_max) return fail(SUBGEN_ESTATE, "subgen_exact_step: cache capacity n_max exceeded");
    const bool f32 = h->dtype == SUBGEN_DTYPE_FP32;
    int rc;
    if (h->D == 64) rc = f32 ? exact_step_td<float, 64>(h, q, k, v, out) : exact_step_mma<64>(h, q, k, v, out);
    else rc = f32 ? exact_step_td<float, 128>(h, q, k, v, out) : exact_step_mma<128>(h, q, k, v, out);
    if (rc) return rc;
    for (int b = 0; b < h->B; ++b) h->n_host[b] += 1;
    return SUBGEN_OK;
}

int subgen_exact_bytes(subgen_exact_t* h, uint64_t* bytes) {
    if (!h || !bytes) return fail(SUBGEN_EINVAL, "subgen_exact_bytes: NULL argument");
    uint64_t rows = 0;
    for (int b = 0; b < h->B; ++b) rows += (uint64_t)h->n_host[b] * h->Hkv;
    *bytes = 2 * rows * (uint64_t)h->D * h->E;
    return SUBGEN_OK;
}

}  // extern "C"

namespace {

template <typename T, int D>
int kcenter_compress_td(subgen_exact* h, int k, int r, int k_iter, int keep_max, int n_old_max) {
    ExactCache<T> E = make_exact<T>(h);
    // one resident wave of 128-thread blocks, and slices short enough for the 16-bit survivor offsets
    int S = (148 * 8) / h->U;
    S = S < 1 ? 1 : (S > 64 ? 64 : S);
    const int s_min = (n_old_max + kKcSliceMax - 1) / kKcSliceMax;
    S = S < s_min ? s_min : S;
    const size_t smem = (size_t)((n_old_max + S - 1) / S) * sizeof(unsigned short);
    constexpr int HP = kKcHead / Elem<T>::EPL;
    const size_t b_dist = align_up((size_t)h->U * h->n_max * 8), b_cent = align_up((size_t)h->U * k * 4);
    const size_t b_part = align_up((size_t)h->U * S * sizeof(Best));
    const size_t b_rows = align_up((size_t)h->U * keep_max * D * sizeof(T)), b_tok = align_up((size_t)h->U * keep_max * 4);
    const size_t b_head = align_up((size_t)h->U * HP * h->n_max * sizeof(uint4)), b_cnt = align_up(16);
    char* scratch = nullptr;
    cudaError_t e = cudaMalloc((void**)&scratch, b_dist + b_cent + 2 * b_part + 2 * b_rows + b_tok + b_head + b_cnt);
    if (e != cudaSuccess) return fail(SUBGEN_ENOMEM, "subgen_exact_kcenter_compress: scratch allocation failed: %s", cudaGetErrorString(e));
    unsigned long long* dist = (unsigned long long*)scratch;
    int* centres = (int*)(scratch + b_dist);
    Best* part[2] = {(Best*)(scratch + b_dist + b_cent), (Best*)(scratch + b_dist + b_cent + b_part)};
    T* Kt = (T*)(scratch + b_dist + b_cent + 2 * b_part);
    T* Vt = (T*)(scratch + b_dist + b_cent + 2 * b_part + b_rows);
    int* tokt = (int*)(scratch + b_dist + b_cent + 2 * b_part + 2 * b_rows);
    uint4* head = (uint4*)(scratch + b_dist + b_cent + 2 * b_part + 2 * b_rows + b_tok);
    unsigned long long* counters = (unsigned long long*)(scratch + b_dist + b_cent + 2 * b_part + 2 * b_rows + b_tok + b_head);
    cudaMemsetAsync(counters, 0, 16, h->st);
    int gi = (h->n_max + 255) / 256;
    gi = gi > 32 ? 32 : gi;
    kcenter_init_kernel<T, D><<<dim3(gi, h->U), 256, 0, h->st>>>(E, r, head, dist);
    for (int t = 0; t < k_iter; ++t)
        launch_pdl_smem(kcenter_iter_kernel<T, D>, dim3(S, h->U), dim3(kKcThreads), smem, h->st, E, t, k, r, (const uint4*)head, dist, centres,
                        (const Best*)part[(t + 1) & 1], part[t & 1], counters);
    int gx = (int)(((size_t)keep_max * (D / Elem<T>::EPL) + 255) / 256);
    gx = gx < 1 ? 1 : (gx > 32 ? 32 : gx);
    kcenter_gather_kernel<T, D><<<dim3(gx, h->U), 256, 0, h->st>>>(E, k, r, centres, Kt, Vt, tokt, keep_max);
    kcenter_scatter_kernel<T, D><<<dim3(gx, h->U), 256, 0, h->st>>>(E, k, r, Kt, Vt, tokt, keep_max);
    kcenter_commit_kernel<T><<<(h->U + 255) / 256, 256, 0, h->st>>>(E, h->U, k, r);
    cudaError_t le = take_launch_error();
    cudaError_t se = cudaMemcpyAsync(h->kc_counters, counters, 16, cudaMemcpyDeviceToHost, h->st);
    if (se == cudaSuccess) se = cudaStreamSynchronize(h->st);
    cudaFree(scratch);
    if (le != cudaSuccess || se != cudaSuccess)
        return fail(SUBGEN_ECUDA, "subgen_exact_kcenter_compress: %s", cudaGetErrorString(le != cudaSuccess ? le : se));
    h->launches += (uint64_t)k_iter + 4;
    return SUBGEN_OK;
}

}  // namespace

extern "C" int subgen_exact_kcenter_compress(subgen_exact_t* h, int k, int r) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_exact_kcenter_compress: handle is NULL");
    if (k < 1 || r < 0) return fail(SUBGEN_EINVAL, "subgen_exact_kcenter_compress: k must be >= 1 and r >= 0");
    int k_iter = 0, keep_max = 0, n_old_max = 0;
    for (int b = 0; b < h->B; ++b) {
        const int n = h->n_host[b], n_old = n > r ? n - r : 0, kk = k < n_old ? k : n_old;
        n_old_max = n_old > n_old_max ? n_old : n_old_max;
        k_iter = kk > k_iter ? kk : k_iter;
        keep_max = kk + (n - n_old) > keep_max ? kk + (n - n_old) : keep_max;
    }
    if (keep_max == 0) return SUBGEN_OK;
    const bool f32 = h->dtype == SUBGEN_DTYPE_FP32;
    int rc;
    if (h->D == 64) rc = f32 ? kcenter_compress_td<float, 64>(h, k, r, k_iter, keep_max, n_old_max) : kcenter_compress_td<__nv_bfloat16, 64>(h, k, r, k_iter, keep_max, n_old_max);
    else rc = f32 ? kcenter_compress_td<float, 128>(h, k, r, k_iter, keep_max, n_old_max) : kcenter_compress_td<__nv_bfloat16, 128>(h, k, r, k_iter, keep_max, n_old_max);
    if (rc) return rc;
    for (int b = 0; b < h->B; ++b) {
        const int n = h->n_host[b], n_old = n > r ? n - r : 0;
        h->n_host[b] = (k < n_old ? k : n_old) + (n - n_old);
    }
    return SUBGEN_OK;
}

extern "C" int subgen_exact_kcenter_counters(const subgen_exact_t* h, uint64_t* tokens_looked_at, uint64_t* full_rows_read) {
    if (!h) return fail(SUBGEN_EINVAL, "subgen_exact_kcenter_counters: handle is NULL");
    if (tokens_looked_at) *tokens_looked_at = h->kc_counters[0];
    if (full_rows_read) *full_rows_read = h->kc_counters[1];
    return SUBGEN_OK;
}

extern "C" int subgen_exact_export_tokens(subgen_exact_t* h, int seq, int kvhead, int* n_out, int* tok) {
    if (!h || !n_out) return fail(SUBGEN_EINVAL, "subgen_exact_export_tokens: NULL argument");
    if (seq < 0 || seq >= h->B || kvhead < 0 || kvhead >= h->Hkv) return fail(SUBGEN_EINVAL, "subgen_exact_export_tokens: unit out of range");
    CUDA_TRY(cudaStreamSynchronize(h->st));
    const size_t u = (size_t)seq * h->Hkv + kvhead;
    *n_out = h->n_host[seq];
    if (tok && h->n_host[seq] > 0)
        CUDA_TRY(cudaMemcpy(tok, h->misc + h->off_tok + u * h->n_max * 4, (size_t)h->n_host[seq] * 4, cudaMemcpyDeviceToHost));
    return SUBGEN_OK;
}

extern "C" {

uint64_t subgen_exact_launch_count(const subgen_exact_t* h) { return h ? h->launches : 0; }

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Exact attention for callers that must not allocate: the split partials live in a fixed array that
// is part of the loaded module instead of in memory obtained from cudaMalloc.

#include <mutex>

namespace {

// One array per device that loads this library, held until the process exits. The name below is only
// meaningful to device code; host code must use the address cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_static_scratch[SUBGEN_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {nullptr};

// grid (splits, U): softmax(K q)^T V over the n rows of the caller's K, V [B, Hkv, n, D].
template <typename T, int D, int G>
__global__ void __launch_bounds__(kQueryThreads) attend_static_kernel(const T* __restrict__ q, const T* __restrict__ K,
                                                                      const T* __restrict__ V, T* __restrict__ out,
                                                                      int n, int H, int Hkv, float* part, unsigned* ticket) {
    constexpr int EPL = Elem<T>::EPL, LPR = D / EPL, RPW = 32 / LPR, STR = D + 2, UN = 2;
    __shared__ float sm[(kQueryThreads / 32) * G * STR];
    __shared__ int sm_last;
    const int u = blockIdx.y, splits = gridDim.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, lr = lane % LPR, sub = lane / LPR;
    const int b = u / Hkv, kvh = u % Hkv;
    const size_t qrow0 = (size_t)b * H + (size_t)kvh * G;
    const T* Ku = K + (size_t)u * n * D;
    const T* Vu = V + (size_t)u * n * D;
    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint4 r = *reinterpret_cast<const uint4*>(q + (qrow0 + g) * D + lr * EPL);
        Elem<T>::unpack(r, qf[g]);
    }
    Acc<G, EPL> A;
    A.init();
    const int gg = (blockIdx.x * (kQueryThreads / 32) + warp) * RPW + sub;
    const int GG = splits * (kQueryThreads / 32) * RPW;
    for (int jb = 0; jb < n; jb += GG * UN) {
        uint4 kraw[UN], vraw[UN];
        bool valid[UN];
        float wt_tau[UN], wt_z[UN];
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            const int idx = jb + i * GG + gg;
            valid[i] = idx < n;
            wt_tau[i] = 1.f; wt_z[i] = 1.f;
            kraw[i] = make_uint4(0, 0, 0, 0);
            vraw[i] = kraw[i];
            if (valid[i]) {
                kraw[i] = *reinterpret_cast<const uint4*>(Ku + (size_t)idx * D + lr * EPL);
                vraw[i] = *reinterpret_cast<const uint4*>(Vu + (size_t)idx * D + lr * EPL);
            }
        }
        float sc[UN][G];
        scores<T, D, G, UN>(kraw, qf, sc);
        fold<T, D, G, UN, true>(A, sc, valid, wt_tau, wt_z, vraw);
    }
    float* part_u = part + (size_t)u * splits * G * STR;
    block_partial<T, D, G>(A, sm, part_u + (size_t)blockIdx.x * G * STR);
    __threadfence();
    __syncthreads();
    if (splits > 1) {
        if (tid == 0) {
            __threadfence();
            sm_last = (atomicAdd(&ticket[u], 1u) == (unsigned)splits - 1u);
        }
        __syncthreads();
        if (!sm_last) return;
        __threadfence();
    }
    final_merge<T, D, G>(part_u, splits, out + qrow0 * D, false);
}

template <typename T, int D>
void launch_attend_static(int G, dim3 grid, cudaStream_t st, const void* q, const void* K, const void* V, void* out, int n,
                          int H, int Hkv, float* part, unsigned* ticket) {
    switch (G) {
        case 1: attend_static_kernel<T, D, 1><<<grid, kQueryThreads, 0, st>>>((const T*)q, (const T*)K, (const T*)V, (T*)out, n, H, Hkv, part, ticket); break;
        case 2: attend_static_kernel<T, D, 2><<<grid, kQueryThreads, 0, st>>>((const T*)q, (const T*)K, (const T*)V, (T*)out, n, H, Hkv, part, ticket); break;
        case 4: attend_static_kernel<T, D, 4><<<grid, kQueryThreads, 0, st>>>((const T*)q, (const T*)K, (const T*)V, (T*)out, n, H, Hkv, part, ticket); break;
        default: attend_static_kernel<T, D, 8><<<grid, kQueryThreads, 0, st>>>((const T*)q, (const T*)K, (const T*)V, (T*)out, n, H, Hkv, part, ticket); break;
    }
}

}  // namespace

extern "C" int subgen_exact_attention_noalloc(const void* q, const void* K, const void* V, void* out, int B, int H, int Hkv,
                                              int d, int n, int dtype, void* stream) {
    if (Hkv == 0) Hkv = H;
    if (!q || !K || !V || !out) return fail(SUBGEN_EINVAL, "subgen_exact_attention_noalloc: q, K, V, out must not be NULL");
    if (B <= 0 || H <= 0 || Hkv <= 0 || H % Hkv || n <= 0 || (d != 64 && d != 128) ||
        (dtype != SUBGEN_DTYPE_FP32 && dtype != SUBGEN_DTYPE_BF16) || (long long)B * Hkv > 65535)
        return fail(SUBGEN_EINVAL, "subgen_exact_attention_noalloc: invalid shape or dtype");
    const int G = H / Hkv;
    if (G != 1 && G != 2 && G != 4 && G != 8) return fail(SUBGEN_EINVAL, "subgen_exact_attention_noalloc: H / Hkv must be 1, 2, 4 or 8");
    if (((uintptr_t)q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)out) & 15)
        return fail(SUBGEN_EINVAL, "subgen_exact_attention_noalloc: pointers must be 16-byte aligned");
    const int U = B * Hkv;
    // layout of the fixed array: [tickets: U unsigned, rounded up to 256 bytes][partials: U*splits*G*(d+2) floats]
    const size_t ticket_bytes = align_up((size_t)U * sizeof(unsigned));
    const size_t per_split = (size_t)U * G * (d + 2) * sizeof(float);
    if (ticket_bytes + per_split > (size_t)SUBGEN_NOALLOC_SCRATCH_BYTES)
        return fail(SUBGEN_EINVAL,
                    "subgen_exact_attention_noalloc: B*Hkv=%d with H/Hkv=%d, d=%d needs %zu bytes of scratch, the fixed array has %zu",
                    U, G, d, ticket_bytes + per_split, (size_t)SUBGEN_NOALLOC_SCRATCH_BYTES);
    int splits = (148 * 8 + U - 1) / U;
    splits = splits < 1 ? 1 : (splits > 32 ? 32 : splits);
    const int by_rows = (n + 63) / 64;                      // no more blocks than 64-row pieces
    if (splits > by_rows) splits = by_rows;
    const size_t fit = ((size_t)SUBGEN_NOALLOC_SCRATCH_BYTES - ticket_bytes) / per_split;
    if ((size_t)splits > fit) splits = (int)fit;

    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(SUBGEN_EINVAL, "subgen_exact_attention_noalloc: device index %d not supported", dev);
    void* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {                           // first call on this device: resolve the array's device address
            void* p = nullptr;
            CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
            g_static_ptr[dev] = p;
        }
        base = g_static_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    unsigned* ticket = (unsigned*)base;
    float* part = (float*)((char*)base + ticket_bytes);
    CUDA_TRY(cudaMemsetAsync(ticket, 0, (size_t)U * sizeof(unsigned), st));   // the array keeps the last call's contents
    const dim3 grid(splits, U);
    const bool f32 = dtype == SUBGEN_DTYPE_FP32;
    if (d == 64) {
        if (f32) launch_attend_static<float, 64>(G, grid, st, q, K, V, out, n, H, Hkv, part, ticket);
        else launch_attend_static<__nv_bfloat16, 64>(G, grid, st, q, K, V, out, n, H, Hkv, part, ticket);
    } else {
        if (f32) launch_attend_static<float, 128>(G, grid, st, q, K, V, out, n, H, Hkv, part, ticket);
        else launch_attend_static<__nv_bfloat16, 128>(G, grid, st, q, K, V, out, n, H, Hkv, part, ticket);
    }
    CUDA_TRY(take_launch_error());
    return SUBGEN_OK;
}
