// Host side of the C ABI declared in include/stateflow.h: validation, workspace layout, kernel
// dispatch, the segment-chaining driver and the host-memory end-to-end wrapper.
#include "../../include/stateflow.h"

#include <algorithm>
#include <atomic>
#include <climits>
#include <cmath>
#include <mutex>
#include <new>
#include <vector>

#include "sf_common.cuh"
#include "sf_scan.cuh"
#include "sf_simt.cuh"
#include "sf_tc.cuh"

namespace {

using sf::SegParams;

std::atomic<long long> g_launches{0};

// Optional per-stage device timers (off by default): every kernel launch is bracketed by a pair of
// events on its own stream.
enum Stage { ST_AGG_KV = 0, ST_AGG_QDO, ST_SCAN, ST_FWD_OUT, ST_DQ, ST_DKDV, ST_DG, ST_COUNT };
struct TimedLaunch { cudaEvent_t a, b; int stage; };
std::mutex g_timing_mu;
bool g_timing_on = false;
std::vector<TimedLaunch> g_timed;

struct StageTimer {
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st;
    int stage;
    StageTimer(int stage_, cudaStream_t st_) : st(st_), stage(stage_) {
        if (!g_timing_on) return;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { cudaGetLastError(); a = b = nullptr; return; }
        cudaEventRecord(a, st);
    }
    ~StageTimer() {
        if (!a) return;
        cudaEventRecord(b, st);
        std::lock_guard<std::mutex> lk(g_timing_mu);
        g_timed.push_back({a, b, stage});
    }
};

constexpr int kDefaultChunksPerBlock = 16;
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// A chain call made by the host-buffer wrapper on one segment of its own (aligned) buffers: g and dg of a segment
// that starts at an odd token are only 4-byte aligned, exactly as for an inner segment of a chain.
thread_local bool tl_segment_of_chain = false;
struct SegmentOfChain {
    SegmentOfChain() { tl_segment_of_chain = true; }
    ~SegmentOfChain() { tl_segment_of_chain = false; }
};
inline bool chain_ptr_ok(const void* p, const void* g, const void* dg) {
    if (tl_segment_of_chain && (p == g || p == dg)) return (reinterpret_cast<uintptr_t>(p) & 3u) == 0;
    return aligned16(p);
}

enum class Path { Invalid, Unsupported, Simt, Tc };

Path classify(const sf_seg_desc_t* d) {
    if (!d) return Path::Invalid;
    if (d->B <= 0 || d->H <= 0 || d->d_k <= 0 || d->d_v <= 0 || d->chunk <= 0 || d->seg_len <= 0) return Path::Invalid;
    if (d->chunks_per_block < 0 || d->chunks_per_block > sf::simt::MAXR) return Path::Invalid;
    if (d->dtype != SF_BF16 && d->dtype != SF_F32) return Path::Invalid;
    if (d->tok_stride_qk < (long long)d->H * d->d_k || d->tok_stride_v < (long long)d->H * d->d_v || d->tok_stride_g < d->H)
        return Path::Invalid;
    if (d->B > 1 && (d->batch_stride_qk <= 0 || d->batch_stride_v <= 0 || d->batch_stride_g <= 0)) return Path::Invalid;
    if (d->H > 65535 || d->B > 65535) return Path::Invalid;
    const bool c_ok = d->chunk == 16 || d->chunk == 32 || d->chunk == 64;
    auto d_ok = [](int x) { return x == 32 || x == 64 || x == 128; };
    if (!c_ok || !d_ok(d->d_k) || !d_ok(d->d_v)) return Path::Unsupported;
    if ((long long)d->B * d->H > 65535LL) return Path::Invalid;              // grid.y of the scan kernels
    if (d->dtype == SF_BF16) {
        if (d->tok_stride_qk % 8 || d->tok_stride_v % 8 || d->batch_stride_qk % 8 || d->batch_stride_v % 8) return Path::Invalid;
        if (d->d_k == 128 && d->d_v == 128) {
            if (d->chunk != 64 || d->chunks_per_block > sf::tc::MAXR || 2LL * d->H > 65535LL) return Path::Unsupported;
            return Path::Tc;
        }
        if (d->d_k == 128 || d->d_v == 128) return Path::Unsupported;
        return d->d_k == d->d_v || (d->d_k == 32 && d->d_v == 64) ? Path::Simt : Path::Unsupported;
    }
    if (d->tok_stride_qk % 4 || d->tok_stride_v % 4 || d->batch_stride_qk % 4 || d->batch_stride_v % 4) return Path::Invalid;
    return d->d_k == d->d_v || (d->d_k == 32 && d->d_v == 64) ? Path::Simt : Path::Unsupported;
}

int sm_count() {
    static int table[sf::tc::MAX_DEVICES] = {};          // per device: a process may drive several
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= sf::tc::MAX_DEVICES) { cudaGetLastError(); return 148; }
    if (table[dev] == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) table[dev] = v;
        else { cudaGetLastError(); table[dev] = 148; }
    }
    return table[dev];
}

// Block length when the caller leaves it open: one CTA per (batch, head, block) and one CTA per SM, so a
// kernel takes waves * (chunks per block + a fixed per-CTA cost of about six chunk times).  Pick the
// length in [4, 64] that minimises this; ties go to the longer block (fewer block states in HBM).
int auto_chunks_per_block(int NC, long long bh) {
    const int sms = sm_count();
    int best = kDefaultChunksPerBlock;
    long long best_cost = -1;
    for (int r = 4; r <= 64; ++r) {
        const int reff = r < NC ? r : NC;
        const long long nb = (NC + reff - 1) / reff;
        const long long waves = (nb * bh + sms - 1) / sms;
        const long long cost = waves * (reff + 6);
        if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best = reff; }
        if (r >= NC) break;
    }
    return best;
}

// The same choice for a segment that runs inside a chain of several.  There the sweeps of neighbouring segments
// share the device (the chain driver sends them to different streams), so what counts for a short segment is the
// work per launch, not whole waves: measured (graph replays of whole chains), the fastest block length keeps
// blocks at least 8 chunks long and a launch at 40 CTAs or more (4096-token segments x 16 heads: 16-22 instead of 8
// chunks, 10 % faster; 512- to 2048-token segments x 40 heads: one block instead of two, 8-10 % faster).  Segments
// of more than 64 chunks keep the wave model.
int chain_chunks_per_block(int NC, long long bh) {
    if (NC > 64) return auto_chunks_per_block(NC, bh);
    long long nb = (40 + bh - 1) / bh;                       // blocks for 40 CTAs or more
    const long long by_len = NC / 8 > 0 ? NC / 8 : 1;        // blocks of at least 8 chunks
    if (nb > by_len) nb = by_len;
    const long long least = (NC + 63) / 64;                  // blocks of at most 64 chunks
    if (nb < least) nb = least;
    return (int)((NC + nb - 1) / nb);
}

// Descriptor of segment i of a chain: the caller's block length if given, else the chain model above.
sf_seg_desc_t chain_segment_desc(const sf_seg_desc_t* desc, int32_t seg_len, int32_t n_seg) {
    sf_seg_desc_t t = *desc;
    t.seg_len = seg_len;
    if (t.chunks_per_block == 0 && n_seg > 1 && t.chunk > 0)
        t.chunks_per_block = chain_chunks_per_block((seg_len + t.chunk - 1) / t.chunk, (long long)t.B * t.H);
    return t;
}

SegParams make_params(const sf_seg_desc_t* d, int cpb_override = 0) {
    SegParams p;
    p.B = d->B; p.H = d->H; p.L = d->seg_len; p.C = d->chunk;
    p.NC = (d->seg_len + d->chunk - 1) / d->chunk;      // the last chunk may be partial
    int r = cpb_override > 0 ? cpb_override : d->chunks_per_block;
    p.R = r > 0 ? r : auto_chunks_per_block(p.NC, (long long)d->B * d->H);
    p.NB = (p.NC + p.R - 1) / p.R;
    p.tqk = d->tok_stride_qk; p.tv = d->tok_stride_v; p.tg = d->tok_stride_g;
    p.bqk = d->batch_stride_qk; p.bv = d->batch_stride_v; p.bg = d->batch_stride_g;
    p.bslot = nullptr; p.bbase = nullptr; p.bstride = 0;
    return p;
}

// ---- workspace layout -------------------------------------------------------------------------
// forward           : [beta B*H*NB f32][UH B*H*NB*dk*dv f32]       UH: block aggregates, scanned in place
//                                                                   into block-entering states
// backward (saved)  : [GU B*H*NB*dk*dv][xq B*H*L][xk B*H*L]
// backward (replay) : backward (saved) ++ forward ++ [Sfin B*H*dk*dv]
struct FwdWs { float* beta; float* UH; size_t bytes; };
struct BwdWs { float* GU; float* xq; float* xk; size_t bytes; };

FwdWs fwd_ws(const sf_seg_desc_t* d, const SegParams& p, void* base) {
    FwdWs w;
    char* c = static_cast<char*>(base);
    size_t off = 0;
    const size_t bh = (size_t)p.B * p.H;
    w.beta = reinterpret_cast<float*>(c + off); off += align_up(bh * p.NB * sizeof(float));
    w.UH = reinterpret_cast<float*>(c + off);   off += align_up(bh * p.NB * (size_t)d->d_k * d->d_v * sizeof(float));
    w.bytes = off;
    return w;
}

BwdWs bwd_ws(const sf_seg_desc_t* d, const SegParams& p, void* base) {
    BwdWs w;
    char* c = static_cast<char*>(base);
    size_t off = 0;
    const size_t bh = (size_t)p.B * p.H;
    w.GU = reinterpret_cast<float*>(c + off); off += align_up(bh * p.NB * (size_t)d->d_k * d->d_v * sizeof(float));
    w.xq = reinterpret_cast<float*>(c + off); off += align_up(bh * p.L * sizeof(float));
    w.xk = reinterpret_cast<float*>(c + off); off += align_up(bh * p.L * sizeof(float));
    w.bytes = off;
    return w;
}

size_t state_bytes(const sf_seg_desc_t* d) { return align_up((size_t)d->B * d->H * d->d_k * d->d_v * sizeof(float)); }

inline sf_status_t check_launch() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SF_OK : SF_ERR_CUDA;
}

#define SF_TRY(expr) do { sf_status_t st__ = (expr); if (st__ != SF_OK) return st__; } while (0)

// ---- SIMT dispatch ------------------------------------------------------------------------------
template <typename K>
sf_status_t set_smem(K kernel, size_t bytes) {
    if (bytes > 48 * 1024) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
            cudaGetLastError();
            return SF_ERR_CUDA;
        }
    }
    return SF_OK;
}

enum class Role { Aggregate, FwdOut, BwdDq, BwdDkDv };

struct RoleArgs {
    const void *q, *k, *v, *dO;
    const float* g;
    int mode;                 // Aggregate: 0 forward (k,v), 1 backward (q,dO)
    float *U, *beta;          // Aggregate outputs
    const float* states;      // FwdOut/BwdDq: Hs ; BwdDkDv: Gs
    void *o, *dq, *dk, *dv;
    float *xq, *xk;
};

template <typename T, int DK, int DV>
sf_status_t launch_simt(Role role, const SegParams& p, const RoleArgs& a, cudaStream_t st) {
    using namespace sf::simt;
    dim3 grid(p.NB, p.H, p.B), block(NT);
    switch (role) {
        case Role::Aggregate: {
            auto kern = block_aggregate_kernel<T, DK, DV>;
            constexpr size_t sm = smem_aggregate<DK, DV>();
            SF_TRY(set_smem(kern, sm));
            const T* X = static_cast<const T*>(a.mode == 0 ? a.k : a.q);
            const T* Y = static_cast<const T*>(a.mode == 0 ? a.v : a.dO);
            kern<<<grid, block, sm, st>>>(p, X, Y, a.g, a.mode, a.U, a.beta);
            break;
        }
        case Role::FwdOut: {
            auto kern = fwd_out_kernel<T, DK, DV>;
            constexpr size_t sm = smem_fwd_out<DK, DV>();
            SF_TRY(set_smem(kern, sm));
            kern<<<grid, block, sm, st>>>(p, static_cast<const T*>(a.q), static_cast<const T*>(a.k),
                                          static_cast<const T*>(a.v), a.g, a.states, static_cast<T*>(a.o));
            break;
        }
        case Role::BwdDq: {
            auto kern = bwd_dq_kernel<T, DK, DV>;
            constexpr size_t sm = smem_bwd_dq<DK, DV>();
            SF_TRY(set_smem(kern, sm));
            kern<<<grid, block, sm, st>>>(p, static_cast<const T*>(a.q), static_cast<const T*>(a.k),
                                          static_cast<const T*>(a.v), a.g, static_cast<const T*>(a.dO), a.states,
                                          static_cast<T*>(a.dq), a.xq);
            break;
        }
        case Role::BwdDkDv: {
            auto kern = bwd_dkdv_kernel<T, DK, DV>;
            constexpr size_t sm = smem_bwd_dkdv<DK, DV>();
            SF_TRY(set_smem(kern, sm));
            kern<<<grid, block, sm, st>>>(p, static_cast<const T*>(a.q), static_cast<const T*>(a.k),
                                          static_cast<const T*>(a.v), a.g, static_cast<const T*>(a.dO), a.states,
                                          static_cast<T*>(a.dk), static_cast<T*>(a.dv), a.xk);
            break;
        }
    }
    return check_launch();
}

template <typename T>
sf_status_t launch_simt_d(Role role, const sf_seg_desc_t* d, const SegParams& p, const RoleArgs& a, cudaStream_t st) {
    if (d->d_k == 32 && d->d_v == 32) return launch_simt<T, 32, 32>(role, p, a, st);
    if (d->d_k == 64 && d->d_v == 64) return launch_simt<T, 64, 64>(role, p, a, st);
    if (d->d_k == 32 && d->d_v == 64) return launch_simt<T, 32, 64>(role, p, a, st);
    if constexpr (sizeof(T) == 4) {
        if (d->d_k == 128 && d->d_v == 128) return launch_simt<T, 128, 128>(role, p, a, st);
    }
    return SF_ERR_UNSUPPORTED;
}

sf_status_t launch_role(Path path, Role role, const sf_seg_desc_t* d, const SegParams& p, const RoleArgs& a, cudaStream_t st) {
    const int stage = role == Role::Aggregate ? (a.mode == 0 ? ST_AGG_KV : ST_AGG_QDO)
                    : role == Role::FwdOut ? ST_FWD_OUT : role == Role::BwdDq ? ST_DQ : ST_DKDV;
    StageTimer timer(stage, st);
    if (path == Path::Tc) {
        long long n = 0;
        sf_status_t s = sf::tc::launch(static_cast<int>(role), d, p, a.q, a.k, a.v, a.dO, a.g, a.mode, a.U, a.beta, a.states,
                                       a.o, a.dq, a.dk, a.dv, a.xq, a.xk, st, &n);
        g_launches.fetch_add(n, std::memory_order_relaxed);
        return s;
    }
    if (d->dtype == SF_F32) return launch_simt_d<float>(role, d, p, a, st);
    return launch_simt_d<__nv_bfloat16>(role, d, p, a, st);
}

sf_status_t launch_scan(const sf_seg_desc_t* d, const SegParams& p, int reverse, const float* ld, const float* U,
                        const float* init, float* states, float* fin, cudaStream_t st) {
    const int m = d->d_k * d->d_v;
    StageTimer timer(ST_SCAN, st);
    dim3 grid((m / 4 + sf::SCAN_NT - 1) / sf::SCAN_NT, p.B * p.H);
    sf::state_scan_kernel<<<grid, sf::SCAN_NT, 0, st>>>(p.NB, m, reverse, ld, U, init, states, fin);
    return check_launch();
}

// Scan of a group of consecutive segments in one launch (the chaining driver's way to shorten the serial chain of
// small scan kernels).  `grp` lists the segments in visiting order.
sf_status_t launch_scan_group(const sf_seg_desc_t* d, int BH, const sf::ScanGroup& grp, int reverse, const float* init,
                              cudaStream_t st) {
    const int m = d->d_k * d->d_v;
    StageTimer timer(ST_SCAN, st);
    dim3 grid((m / 4 + sf::SCAN_NT - 1) / sf::SCAN_NT, BH);
    sf::state_scan_group_kernel<<<grid, sf::SCAN_NT, 0, st>>>(grp, m, reverse, init);
    return check_launch();
}

// Schedule of the chaining driver (sf_tuning_t; process-wide, read at every chain call).
constexpr int kMaxSweepStreams = 4, kMaxAggStreams = 4;
const sf_tuning_t kDefaultTuning = {4, 4, 4096, 74, 0, 0};
std::mutex g_tuning_mu;
sf_tuning_t g_tuning = kDefaultTuning;
sf_tuning_t current_tuning() {
    std::lock_guard<std::mutex> lk(g_tuning_mu);
    return g_tuning;
}

// Segments i, i+dir, ... that the chaining driver scans together: up to SCAN_GROUP_MAX short segments of at most
// scan_group_tokens tokens in total (one long segment is a group of its own).
int scan_group_size(const int32_t* seg_lens, int n_seg, int i, int dir, long long kScanGroupTokens) {
    int count = 1;
    long long tokens = seg_lens[i];
    for (int k = i + dir; k >= 0 && k < n_seg && count < sf::SCAN_GROUP_MAX; k += dir) {
        if (tokens + seg_lens[k] > kScanGroupTokens) break;
        tokens += seg_lens[k];
        ++count;
    }
    return count;
}

// ---- one segment -------------------------------------------------------------------------------
struct FwdPtrs { const void *q, *k, *v; const float* g; const float* S_in; void* o; float* S_out; };

// Stage split used by the chaining driver: `pre` needs no boundary state, `post` does.
sf_status_t fwd_pre(Path path, const sf_seg_desc_t* d, const SegParams& p, const FwdPtrs& x, const FwdWs& w, cudaStream_t st) {
    RoleArgs a{};
    a.k = x.k; a.v = x.v; a.g = x.g; a.mode = 0; a.U = w.UH; a.beta = w.beta;
    return launch_role(path, Role::Aggregate, d, p, a, st);
}
sf_status_t fwd_scan(const sf_seg_desc_t* d, const SegParams& p, const FwdPtrs& x, const FwdWs& w, cudaStream_t st) {
    return launch_scan(d, p, 0, w.beta, w.UH, x.S_in, w.UH, x.S_out, st);
}
sf_status_t fwd_out(Path path, const sf_seg_desc_t* d, const SegParams& p, const FwdPtrs& x, const FwdWs& w, cudaStream_t st) {
    RoleArgs a{};
    a.q = x.q; a.k = x.k; a.v = x.v; a.g = x.g; a.states = w.UH; a.o = x.o;
    return launch_role(path, Role::FwdOut, d, p, a, st);
}

struct BwdPtrs {
    const void *q, *k, *v; const float* g; const float* S_in; const void* dO; const float* dS_out;
    void *dq, *dk, *dv; float* dg; float* dS_in;
};

sf_status_t bwd_pre(Path path, const sf_seg_desc_t* d, const SegParams& p, const BwdPtrs& x, const BwdWs& w, float* beta_out,
                    cudaStream_t st) {
    RoleArgs a{};
    a.q = x.q; a.dO = x.dO; a.g = x.g; a.mode = 1; a.U = w.GU; a.beta = beta_out;
    return launch_role(path, Role::Aggregate, d, p, a, st);
}
sf_status_t bwd_scan(const sf_seg_desc_t* d, const SegParams& p, const BwdPtrs& x, const BwdWs& w, const float* beta, cudaStream_t st) {
    return launch_scan(d, p, 1, beta, w.GU, x.dS_out, w.GU, x.dS_in, st);
}
sf_status_t bwd_dq(Path path, const sf_seg_desc_t* d, const SegParams& p, const BwdPtrs& x, const BwdWs& w, const float* Hs, cudaStream_t st) {
    RoleArgs a{};
    a.q = x.q; a.k = x.k; a.v = x.v; a.dO = x.dO; a.g = x.g; a.states = Hs; a.dq = x.dq; a.xq = w.xq;
    return launch_role(path, Role::BwdDq, d, p, a, st);
}
sf_status_t bwd_dkdv(Path path, const sf_seg_desc_t* d, const SegParams& p, const BwdPtrs& x, const BwdWs& w, cudaStream_t st) {
    RoleArgs a{};
    a.q = x.q; a.k = x.k; a.v = x.v; a.dO = x.dO; a.g = x.g; a.states = w.GU; a.dk = x.dk; a.dv = x.dv; a.xk = w.xk;
    return launch_role(path, Role::BwdDkDv, d, p, a, st);
}
sf_status_t bwd_dg(const sf_seg_desc_t* d, const SegParams& p, const BwdPtrs& x, const BwdWs& w, const float* Hs, cudaStream_t st) {
    StageTimer timer(ST_DG, st);
    dim3 grid(p.NB, p.H, p.B);
    sf::dg_epilogue_kernel<<<grid, sf::DG_NT, 0, st>>>(p, d->d_k * d->d_v, w.xq, w.xk, Hs, w.GU, x.dS_in, x.dg);
    return check_launch();
}

sf_status_t validate_fwd(const sf_seg_desc_t* d, const FwdPtrs& x, const void* ws, size_t ws_bytes, Path* path) {
    *path = classify(d);
    if (*path == Path::Invalid) return SF_ERR_INVALID_ARG;
    if (*path == Path::Unsupported) return SF_ERR_UNSUPPORTED;
    if (!x.q || !x.k || !x.v || !x.g || !x.o || !x.S_out) return SF_ERR_INVALID_ARG;
    if (x.S_in == x.S_out) return SF_ERR_INVALID_ARG;
    const void* ptrs[] = {x.q, x.k, x.v, x.g, x.S_in, x.o, x.S_out};
    for (const void* ptr : ptrs) if (ptr && !aligned16(ptr)) return SF_ERR_INVALID_ARG;
    if (!ws || ws_bytes < sf_workspace_bytes(d, 0)) return SF_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) % kAlign) return SF_ERR_INVALID_ARG;
    return SF_OK;
}

sf_status_t validate_bwd(const sf_seg_desc_t* d, const BwdPtrs& x, const void* saved, const void* ws, size_t ws_bytes, Path* path) {
    *path = classify(d);
    if (*path == Path::Invalid) return SF_ERR_INVALID_ARG;
    if (*path == Path::Unsupported) return SF_ERR_UNSUPPORTED;
    if (!x.q || !x.k || !x.v || !x.g || !x.dO || !x.dq || !x.dk || !x.dv || !x.dg || !x.dS_in) return SF_ERR_INVALID_ARG;
    if (x.dS_out == x.dS_in) return SF_ERR_INVALID_ARG;
    const void* ptrs[] = {x.q, x.k, x.v, x.g, x.S_in, x.dO, x.dS_out, x.dq, x.dk, x.dv, x.dg, x.dS_in, saved};
    for (const void* ptr : ptrs) if (ptr && !aligned16(ptr)) return SF_ERR_INVALID_ARG;
    if (!ws || ws_bytes < sf_workspace_bytes(d, saved ? 1 : 2)) return SF_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) % kAlign) return SF_ERR_INVALID_ARG;
    if (saved && saved == ws) return SF_ERR_INVALID_ARG;
    if (saved && reinterpret_cast<uintptr_t>(saved) % kAlign) return SF_ERR_INVALID_ARG;
    return SF_OK;
}

// Side streams and events of the chaining driver (host objects only; created once per process).
// Sweeps of consecutive segments go to different streams: a short segment's sweep does not fill the device.
constexpr int kSweepStreams = kMaxSweepStreams;       // streams that exist; a tuning may use fewer
// The aggregates of different segments are independent of everything: they go round-robin to their own streams
// (with short segments one stream of small aggregate kernels is the longest chain of the step).
constexpr int kAggStreams = kMaxAggStreams;
// ... unless a segment's aggregate kernel fills half the device by itself: those stay in order on one stream
inline int agg_stream_index(const SegParams& p, int i, const sf_tuning_t& tu) {
    return (long long)p.B * p.H * p.NB >= tu.agg_inorder_ctas ? 0 : i % tu.agg_streams;
}
struct ChainRes {
    cudaStream_t side[1 + 2 * kSweepStreams] = {};   // 0: unused; then two groups of sweep streams, used round-robin by segment
    cudaStream_t agg[kAggStreams] = {};
    cudaStream_t copy[2] = {};              // host-buffer wrapper: second upload stream, download stream
    cudaEvent_t ev[64] = {};
    std::vector<cudaEvent_t> pool;          // extra events of the backward driver, grown on demand
    bool ok = false;
    int device = -1;
};
std::mutex g_chain_mu;
ChainRes g_chain[sf::tc::MAX_DEVICES];      // one set of side streams and events per device, created on first use there

sf_status_t chain_resources(ChainRes** out) {
    std::lock_guard<std::mutex> lk(g_chain_mu);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= sf::tc::MAX_DEVICES) { cudaGetLastError(); return SF_ERR_CUDA; }
    ChainRes& r = g_chain[dev];
    if (!r.ok) {
        for (auto& s : r.side)
            if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess) return SF_ERR_CUDA;
        for (auto& s : r.agg)
            if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess) return SF_ERR_CUDA;
        for (auto& s : r.copy)
            if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess) return SF_ERR_CUDA;
        for (auto& e : r.ev)
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return SF_ERR_CUDA;
        r.ok = true;
        r.device = dev;
    }
    *out = &r;
    return SF_OK;
}

sf_status_t chain_events(ChainRes* res, size_t n) {
    std::lock_guard<std::mutex> lk(g_chain_mu);
    while (res->pool.size() < n) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return SF_ERR_CUDA; }
        res->pool.push_back(e);
    }
    return SF_OK;
}

#define SF_CUDA(expr) do { if ((expr) != cudaSuccess) { cudaGetLastError(); return SF_ERR_CUDA; } } while (0)

struct SeqPtr {
    // byte pointer arithmetic over a [B,T,H,d] tensor along T
    static const void* at(const void* base, long long tok, long long stride, size_t esz) {
        return base ? static_cast<const char*>(base) + tok * stride * (long long)esz : nullptr;
    }
    static void* at(void* base, long long tok, long long stride, size_t esz) {
        return base ? static_cast<char*>(base) + tok * stride * (long long)esz : nullptr;
    }
};

sf_status_t validate_chain(const sf_seg_desc_t* d, const int32_t* seg_lens, int32_t n_seg, long long* T_out) {
    if (!d || !seg_lens || n_seg <= 0 || n_seg > 1 << 20) return SF_ERR_INVALID_ARG;
    long long T = 0;
    for (int i = 0; i < n_seg; ++i) {
        if (seg_lens[i] <= 0 || d->chunk <= 0) return SF_ERR_INVALID_ARG;
        T += seg_lens[i];
    }
    sf_seg_desc_t t = *d;
    t.seg_len = seg_lens[0];
    Path p = classify(&t);
    if (p == Path::Invalid) return SF_ERR_INVALID_ARG;
    if (p == Path::Unsupported) return SF_ERR_UNSUPPORTED;
    if (T_out) *T_out = T;
    return SF_OK;
}

// ---- merged launches (sf_tuning_t.merge_launches) ------------------------------------------------------------------
// When the segments are whole chunks (tensor-core path) or, on the CUDA-core path, every segment but the last is a whole
// number of blocks of one common length R, the chain is ONE segment that spans the sequence: each stage then runs once over the whole chain (one aggregate launch,
// one scan, one sweep, ...) instead of once per segment, with the same blocks, the same kernels and the same arithmetic
// (results are bit-identical).  The boundary states S_bounds[i] are the states entering the first block of each segment.
// Returns the descriptor of that segment, or false if the chain does not have this shape.
// `free_grid`: on the tensor-core path the forward sweep itself writes the state entering a segment's first chunk
// (SegParams::bslot), so the blocks need not respect the segment boundaries: any block length, segments of whole chunks.
bool merged_desc(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, long long T, sf_seg_desc_t* out,
                 bool* free_grid = nullptr) {
    if (free_grid) *free_grid = false;
    if (n_seg < 2 || T > 0x7fffffffLL) return false;
    const int C = desc->chunk;
    for (int i = 0; i + 1 < n_seg; ++i)
        if (seg_lens[i] % C) return false;
    sf_seg_desc_t t = *desc;
    t.seg_len = (int32_t)T;
    {
        sf_seg_desc_t f = t;                             // block length: the caller's, else the library's model for one long segment
        const Path path = classify(&f);
        if (path == Path::Tc) {
            if (make_params(&f).NB > 65535) return false;
            f.chunks_per_block = make_params(&f).R;
            *out = f;
            if (free_grid) *free_grid = true;
            return true;
        }
    }
    int R = desc->chunks_per_block;
    if (R == 0) {
        // the longest block length (at most 64 chunks) that divides the chunk count of every segment but the last
        for (R = 64; R >= 1; --R) {
            bool ok = true;
            for (int i = 0; i + 1 < n_seg && ok; ++i) ok = (seg_lens[i] / C) % R == 0;
            if (ok) break;
        }
        if (R < 4) return false;
    } else {
        for (int i = 0; i + 1 < n_seg; ++i)
            if ((seg_lens[i] / C) % R) return false;
    }
    t.chunks_per_block = R;
    const Path path = classify(&t);
    if (path == Path::Invalid || path == Path::Unsupported) return false;
    if (make_params(&t).NB > 65535) return false;
    *out = t;
    return true;
}

size_t merged_slot_bytes(const sf_seg_desc_t* vd) { return align_up((size_t)make_params(vd).NC * sizeof(int)); }

sf_status_t chain_fwd_merged(const sf_seg_desc_t* vd, bool free_grid, const int32_t* seg_lens, int32_t n_seg, const FwdPtrs& x,
                             float* S_bounds, void* workspace, cudaStream_t st) {
    const Path path = classify(vd);
    SegParams p = make_params(vd);
    const FwdWs w = fwd_ws(vd, p, workspace);
    const size_t m = (size_t)vd->d_k * vd->d_v, sN = (size_t)vd->B * vd->H * m;
    if (free_grid) {
        // slot[c] = i for the first chunk c of segment i >= 1, else -1; read by the forward sweep
        int* slot = reinterpret_cast<int*>(static_cast<char*>(workspace) + w.bytes);
        SF_CUDA(cudaMemsetAsync(slot, 0xFF, (size_t)p.NC * sizeof(int), st));
        long long chunk = 0;
        for (int i0 = 1; i0 < n_seg; i0 += sf::MARK_MAX) {
            sf::SegStarts s{};
            s.first = i0;
            s.count = n_seg - i0 < sf::MARK_MAX ? n_seg - i0 : sf::MARK_MAX;
            for (int k = 0; k < s.count; ++k) {
                chunk += seg_lens[i0 + k - 1] / vd->chunk;
                s.chunk[k] = (int)chunk;
            }
            sf::mark_bounds_kernel<<<1, sf::MARK_MAX, 0, st>>>(slot, s);
            SF_TRY(check_launch());
        }
        p.bslot = slot;
        p.bbase = S_bounds;
        p.bstride = (long long)sN;
    }
    SF_TRY(fwd_pre(path, vd, p, x, w, st));
    SF_TRY(fwd_scan(vd, p, x, w, st));
    if (!free_grid) {
        // S_bounds[i] = state entering the first block of segment i (a strided copy: one state per batch x head)
        long long blk = 0;
        for (int i = 1; i < n_seg; ++i) {
            blk += (seg_lens[i - 1] / vd->chunk) / p.R;
            SF_CUDA(cudaMemcpy2DAsync(S_bounds + (size_t)i * sN, m * sizeof(float), w.UH + (size_t)blk * m, (size_t)p.NB * m * sizeof(float),
                                      m * sizeof(float), (size_t)vd->B * vd->H, cudaMemcpyDeviceToDevice, st));
        }
    }
    return fwd_out(path, vd, p, x, w, st);
}

sf_status_t chain_bwd_merged(const sf_seg_desc_t* vd, const BwdPtrs& x, const void* fwd_workspace, void* workspace, bool overlap,
                             cudaStream_t st) {
    const Path path = classify(vd);
    const SegParams p = make_params(vd);
    const BwdWs w = bwd_ws(vd, p, workspace);
    FwdWs fw;
    if (fwd_workspace) {
        fw = fwd_ws(vd, p, const_cast<void*>(fwd_workspace));
    } else {
        char* base = static_cast<char*>(workspace) + w.bytes;
        fw = fwd_ws(vd, p, base);
        float* sfin = reinterpret_cast<float*>(base + fw.bytes);
        FwdPtrs fx{x.q, x.k, x.v, x.g, x.S_in, nullptr, sfin};
        SF_TRY(fwd_pre(path, vd, p, fx, fw, st));
        SF_TRY(fwd_scan(vd, p, fx, fw, st));
    }
    // the dq sweep needs only the forward states: with overlap it runs on a side stream beside the backward aggregate and
    // the reverse scan (whose dependent steps leave most of the device idle)
    ChainRes* res = nullptr;
    if (overlap) {
        SF_TRY(chain_resources(&res));
        SF_CUDA(cudaEventRecord(res->ev[5], st));
        SF_CUDA(cudaStreamWaitEvent(res->side[1], res->ev[5], 0));
        SF_TRY(bwd_dq(path, vd, p, x, w, fw.UH, res->side[1]));
        SF_CUDA(cudaEventRecord(res->ev[6], res->side[1]));
    }
    SF_TRY(bwd_pre(path, vd, p, x, w, nullptr, st));
    SF_TRY(bwd_scan(vd, p, x, w, fw.beta, st));
    if (!overlap) SF_TRY(bwd_dq(path, vd, p, x, w, fw.UH, st));
    SF_TRY(bwd_dkdv(path, vd, p, x, w, st));
    if (overlap) SF_CUDA(cudaStreamWaitEvent(st, res->ev[6], 0));
    return bwd_dg(vd, p, x, w, fw.UH, st);
}

}  // namespace

// Scratch of sf_segment_fwd_static: part of the library image, one copy per GPU that loads it.  In host
// code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[SF_STATIC_SCRATCH_BYTES];

// ================================================================================================
extern "C" {

const char* sf_status_string(sf_status_t s) {
    switch (s) {
        case SF_OK: return "ok";
        case SF_ERR_INVALID_ARG: return "invalid argument";
        case SF_ERR_UNSUPPORTED: return "unsupported (dtype, d_k, d_v, chunk) combination";
        case SF_ERR_WORKSPACE: return "workspace missing or too small";
        case SF_ERR_CUDA: return "CUDA call or kernel launch failed";
        case SF_ERR_TIMEOUT: return "bounded device-side wait ran out";
    }
    return "unknown status";
}

int32_t sf_num_blocks(const sf_seg_desc_t* desc) {
    Path p = classify(desc);
    if (p == Path::Invalid || p == Path::Unsupported) return 0;
    return make_params(desc).NB;
}

size_t sf_workspace_bytes(const sf_seg_desc_t* desc, int backward) {
    Path path = classify(desc);
    if (path == Path::Invalid || path == Path::Unsupported) return 0;
    const SegParams p = make_params(desc);
    const size_t f = fwd_ws(desc, p, nullptr).bytes;
    if (backward == 0) return f;
    const size_t b = bwd_ws(desc, p, nullptr).bytes;
    if (backward == 1) return b;
    return b + f + state_bytes(desc);
}

sf_status_t sf_segment_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                           const float* S_in, void* o, float* S_out, void* workspace, size_t workspace_bytes,
                           sf_stream_t stream) {
    FwdPtrs x{q, k, v, g, S_in, o, S_out};
    Path path;
    SF_TRY(validate_fwd(desc, x, workspace, workspace_bytes, &path));
    const SegParams p = make_params(desc);
    const FwdWs w = fwd_ws(desc, p, workspace);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    SF_TRY(fwd_pre(path, desc, p, x, w, st));
    SF_TRY(fwd_scan(desc, p, x, w, st));
    SF_TRY(fwd_out(path, desc, p, x, w, st));
    return SF_OK;
}

sf_status_t sf_segment_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                           const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv, float* dg,
                           float* dS_in, const void* fwd_saved, void* workspace, size_t workspace_bytes, sf_stream_t stream) {
    BwdPtrs x{q, k, v, g, S_in, dO, dS_out, dq, dk, dv, dg, dS_in};
    Path path;
    SF_TRY(validate_bwd(desc, x, fwd_saved, workspace, workspace_bytes, &path));
    const SegParams p = make_params(desc);
    const BwdWs w = bwd_ws(desc, p, workspace);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    FwdWs fw;
    if (fwd_saved) {
        fw = fwd_ws(desc, p, const_cast<void*>(fwd_saved));
    } else {
        // SR: replay the block-entering states from S_in
        char* base = static_cast<char*>(workspace) + w.bytes;
        fw = fwd_ws(desc, p, base);
        float* sfin = reinterpret_cast<float*>(base + fw.bytes);
        FwdPtrs fx{q, k, v, g, S_in, nullptr, sfin};
        SF_TRY(fwd_pre(path, desc, p, fx, fw, st));
        SF_TRY(fwd_scan(desc, p, fx, fw, st));
    }
    SF_TRY(bwd_pre(path, desc, p, x, w, nullptr, st));
    SF_TRY(bwd_scan(desc, p, x, w, fw.beta, st));
    SF_TRY(bwd_dq(path, desc, p, x, w, fw.UH, st));
    SF_TRY(bwd_dkdv(path, desc, p, x, w, st));
    SF_TRY(bwd_dg(desc, p, x, w, fw.UH, st));
    return SF_OK;
}

sf_status_t sf_segment_fwd_static(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                  const float* S_in, void* o, float* S_out, sf_stream_t stream) {
    const Path path = classify(desc);
    if (path == Path::Invalid) return SF_ERR_INVALID_ARG;
    if (path == Path::Unsupported) return SF_ERR_UNSUPPORTED;
    if (sf_workspace_bytes(desc, 0) > SF_STATIC_SCRATCH_BYTES) return SF_ERR_WORKSPACE;
    // device address of the scratch array, looked up once per device with that device current
    constexpr int kMaxDevices = 64;
    static void* scratch_of_device[kMaxDevices] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return SF_ERR_CUDA; }
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lk(mu);
        if (!scratch_of_device[dev]) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) { cudaGetLastError(); return SF_ERR_CUDA; }
            scratch_of_device[dev] = ptr;
        }
        scratch = scratch_of_device[dev];
    }
    return sf_segment_fwd(desc, q, k, v, g, S_in, o, S_out, scratch, SF_STATIC_SCRATCH_BYTES, stream);
}

sf_status_t sf_state_scan(const sf_seg_desc_t* desc, int32_t chunks_per_block, int32_t reverse, const float* log_decay,
                          const float* U, const float* S_boundary_in, float* states, float* S_boundary_out,
                          sf_stream_t stream) {
    Path path = classify(desc);
    if (path == Path::Invalid) return SF_ERR_INVALID_ARG;
    if (path == Path::Unsupported) return SF_ERR_UNSUPPORTED;
    if (chunks_per_block < 0 || chunks_per_block > sf::simt::MAXR) return SF_ERR_INVALID_ARG;
    if (!log_decay || !U || !states || !S_boundary_out || S_boundary_in == S_boundary_out) return SF_ERR_INVALID_ARG;
    if (!aligned16(U) || !aligned16(states) || !aligned16(S_boundary_out) || (S_boundary_in && !aligned16(S_boundary_in)))
        return SF_ERR_INVALID_ARG;
    const SegParams p = make_params(desc, chunks_per_block);
    return launch_scan(desc, p, reverse != 0, log_decay, U, S_boundary_in, states, S_boundary_out,
                       reinterpret_cast<cudaStream_t>(stream));
}

size_t sf_chain_workspace_bytes(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, int backward) {
    if (validate_chain(desc, seg_lens, n_seg, nullptr) != SF_OK) return 0;
    size_t total = 0, mx = 0;
    for (int i = 0; i < n_seg; ++i) {
        sf_seg_desc_t t = chain_segment_desc(desc, seg_lens[i], n_seg);
        const size_t b = sf_workspace_bytes(&t, backward);
        total += b;
        mx = b > mx ? b : mx;
    }
    // forward keeps every segment's block states for the backward; the backward gives every segment its own
    // workspace and boundary-gradient buffer so that the stages of different segments can run concurrently
    (void)mx;
    size_t need = backward == 0 ? total : total + (size_t)n_seg * state_bytes(desc);
    // enough for the merged-launch mode as well (its common block length may be shorter than the segments' own)
    long long T = 0;
    for (int i = 0; i < n_seg; ++i) T += seg_lens[i];
    sf_seg_desc_t vd;
    if (merged_desc(desc, seg_lens, n_seg, T, &vd)) {
        const size_t mb = sf_workspace_bytes(&vd, backward) + (backward == 0 ? merged_slot_bytes(&vd) : 0);
        need = mb > need ? mb : need;
    }
    return need;
}

sf_status_t sf_chain_fwd(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, const void* q, const void* k,
                         const void* v, const float* g, const float* S_init, void* o, float* S_bounds, void* workspace,
                         size_t workspace_bytes, int32_t overlap, sf_stream_t stream) {
    long long T = 0;
    SF_TRY(validate_chain(desc, seg_lens, n_seg, &T));
    if (!q || !k || !v || !g || !o || !S_bounds) return SF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < sf_chain_workspace_bytes(desc, seg_lens, n_seg, 0)) return SF_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return SF_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, g, S_init, o, S_bounds};
    for (const void* ptr : ptrs) if (ptr && !chain_ptr_ok(ptr, g, nullptr)) return SF_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t esz = desc->dtype == SF_BF16 ? 2 : 4;
    const size_t sN = (size_t)desc->B * desc->H * desc->d_k * desc->d_v;

    // S_bounds[0] = S_init (or zero)
    if (S_init == S_bounds) {}              // the state is in place already
    else if (S_init) SF_CUDA(cudaMemcpyAsync(S_bounds, S_init, sN * sizeof(float), cudaMemcpyDeviceToDevice, st));
    else             SF_CUDA(cudaMemsetAsync(S_bounds, 0, sN * sizeof(float), st));

    const sf_tuning_t tu = current_tuning();
    {
        sf_seg_desc_t vd;
        bool free_grid = false;
        if (tu.merge_launches && merged_desc(desc, seg_lens, n_seg, T, &vd, &free_grid) &&
            sf_workspace_bytes(&vd, 0) + merged_slot_bytes(&vd) <= workspace_bytes) {
            FwdPtrs x{q, k, v, g, S_bounds, o, S_bounds + (size_t)n_seg * sN};
            return chain_fwd_merged(&vd, free_grid, seg_lens, n_seg, x, S_bounds, workspace, st);
        }
    }
    ChainRes* res = nullptr;
    if (overlap) SF_TRY(chain_resources(&res));
    // overlap schedule (the forward wavefront of Section 3.4, Eq. 17, across segments):
    //   side stream 0   : Pre(0) Pre(1) Pre(2) ...        (block aggregates need no boundary state)
    //   main stream     : [wait Pre(i)] ST(i)             (only the scans carry the state from segment to segment)
    //   side streams 1..: [wait ST(i)] Out(i)             (round-robin, so that the sweeps of short neighbouring
    //                                                      segments, which do not fill the device, run side by side)
    if (overlap) {
        SF_TRY(chain_events(res, 3 * (size_t)n_seg + 2 + kSweepStreams + kAggStreams));
        SF_CUDA(cudaEventRecord(res->ev[0], st));
        for (int s = 0; s <= kSweepStreams; ++s) SF_CUDA(cudaStreamWaitEvent(res->side[s], res->ev[0], 0));
        for (int s = 0; s < kAggStreams; ++s) SF_CUDA(cudaStreamWaitEvent(res->agg[s], res->ev[0], 0));
    }
    struct Seg { sf_seg_desc_t t; Path path; SegParams p; FwdWs w; FwdPtrs x; };
    std::vector<Seg> segs(n_seg);
    {
        size_t ws_off = 0;
        long long tok = 0;
        for (int i = 0; i < n_seg; ++i) {
            Seg& sg = segs[i];
            sg.t = chain_segment_desc(desc, seg_lens[i], n_seg);
            sg.path = classify(&sg.t);
            sg.p = make_params(&sg.t);
            sg.w = fwd_ws(&sg.t, sg.p, static_cast<char*>(workspace) + ws_off);
            ws_off += sg.w.bytes;
            sg.x = FwdPtrs{SeqPtr::at(q, tok, sg.t.tok_stride_qk, esz), SeqPtr::at(k, tok, sg.t.tok_stride_qk, esz),
                           SeqPtr::at(v, tok, sg.t.tok_stride_v, esz),
                           static_cast<const float*>(SeqPtr::at(g, tok, sg.t.tok_stride_g, sizeof(float))),
                           S_bounds + (size_t)i * sN, SeqPtr::at(o, tok, sg.t.tok_stride_v, esz), S_bounds + (size_t)(i + 1) * sN};
            tok += seg_lens[i];
        }
    }
    if (!overlap) {
        for (int i = 0; i < n_seg; ++i) {
            const Seg& sg = segs[i];
            SF_TRY(fwd_pre(sg.path, &sg.t, sg.p, sg.x, sg.w, st));
            SF_TRY(fwd_scan(&sg.t, sg.p, sg.x, sg.w, st));
            SF_TRY(fwd_out(sg.path, &sg.t, sg.p, sg.x, sg.w, st));
        }
    } else {
        for (int i = 0; i < n_seg;) {
            // short neighbouring segments are scanned in one launch (the state is carried in registers from one to
            // the next); their aggregates go first, their sweeps after
            const int cnt = scan_group_size(seg_lens, n_seg, i, +1, tu.scan_group_tokens);
            sf::ScanGroup grp{};
            grp.count = cnt;
            for (int k = 0; k < cnt; ++k) {
                const Seg& sg = segs[i + k];
                cudaStream_t s_agg = res->agg[agg_stream_index(sg.p, i + k, tu)];
                cudaEvent_t e = res->pool[(size_t)n_seg + (i + k)];
                // agg_ahead: the aggregate of segment j starts only when the sweep of segment j - agg_ahead is done
                // (a segment of an earlier group: its sweep has been enqueued already)
                const int jw = i + k - tu.agg_ahead;
                if (tu.agg_ahead > 0 && jw >= 0 && jw < i) SF_CUDA(cudaStreamWaitEvent(s_agg, res->pool[2 * (size_t)n_seg + jw], 0));
                SF_TRY(fwd_pre(sg.path, &sg.t, sg.p, sg.x, sg.w, s_agg));
                SF_CUDA(cudaEventRecord(e, s_agg));
                SF_CUDA(cudaStreamWaitEvent(st, e, 0));
                grp.seg[k] = sf::ScanSeg{sg.w.beta, sg.w.UH, sg.x.S_out, sg.p.NB};
            }
            SF_TRY(launch_scan_group(desc, desc->B * desc->H, grp, 0, segs[i].x.S_in, st));
            SF_CUDA(cudaEventRecord(res->pool[i], st));
            for (int k = 0; k < cnt; ++k) {
                const Seg& sg = segs[i + k];
                cudaStream_t s_out = res->side[1 + ((i + k) % tu.sweep_streams)];
                SF_CUDA(cudaStreamWaitEvent(s_out, res->pool[i], 0));
                SF_TRY(fwd_out(sg.path, &sg.t, sg.p, sg.x, sg.w, s_out));
                SF_CUDA(cudaEventRecord(res->pool[2 * (size_t)n_seg + (i + k)], s_out));
            }
            i += cnt;
        }
    }
    if (overlap) {
        // join the sweep streams back into the caller's stream
        for (int s = 1; s <= kSweepStreams; ++s) {
            cudaEvent_t e = res->pool[3 * (size_t)n_seg + s];
            SF_CUDA(cudaEventRecord(e, res->side[s]));
            SF_CUDA(cudaStreamWaitEvent(st, e, 0));
        }
        for (int s = 0; s < kAggStreams; ++s) {
            cudaEvent_t e = res->pool[3 * (size_t)n_seg + 1 + kSweepStreams + s];
            SF_CUDA(cudaEventRecord(e, res->agg[s]));
            SF_CUDA(cudaStreamWaitEvent(st, e, 0));
        }
    }
    return SF_OK;
}

sf_status_t sf_chain_bwd(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, const void* q, const void* k,
                         const void* v, const float* g, const float* S_bounds, const void* dO, const float* dS_final,
                         void* dq, void* dk, void* dv, float* dg, float* dS_init, const void* fwd_workspace, void* workspace,
                         size_t workspace_bytes, int32_t overlap, sf_stream_t stream) {
    long long T = 0;
    SF_TRY(validate_chain(desc, seg_lens, n_seg, &T));
    if (!q || !k || !v || !g || !S_bounds || !dO || !dq || !dk || !dv || !dg || !dS_init) return SF_ERR_INVALID_ARG;
    const int mode = fwd_workspace ? 1 : 2;
    const size_t need = sf_chain_workspace_bytes(desc, seg_lens, n_seg, mode);
    const size_t sB = state_bytes(desc);
    if (!workspace || workspace_bytes < need) return SF_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return SF_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, g, S_bounds, dO, dS_final, dq, dk, dv, dg, dS_init, fwd_workspace};
    for (const void* ptr : ptrs) if (ptr && !chain_ptr_ok(ptr, g, dg)) return SF_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t esz = desc->dtype == SF_BF16 ? 2 : 4;
    const size_t sN = (size_t)desc->B * desc->H * desc->d_k * desc->d_v;

    {
        sf_seg_desc_t vd;
        if (current_tuning().merge_launches && merged_desc(desc, seg_lens, n_seg, T, &vd) &&
            sf_workspace_bytes(&vd, mode) <= workspace_bytes && (!fwd_workspace || sf_workspace_bytes(&vd, 0) <= sf_chain_workspace_bytes(desc, seg_lens, n_seg, 0))) {
            BwdPtrs x{q, k, v, g, S_bounds, dO, dS_final, dq, dk, dv, dg, dS_init};
            return chain_bwd_merged(&vd, x, fwd_workspace, workspace, overlap != 0, st);
        }
    }
    // layout: [dS buffers: one state per segment][segment workspaces in order]
    char* base = static_cast<char*>(workspace);
    char* seg_base = base + (size_t)n_seg * sB;

    // overlap schedule (Section 3.4, Eq. 18, across segments): only the reverse scans carry the boundary
    // gradient from segment to segment.  The backward aggregates need no boundary gradient (their own streams,
    // ahead of everything), the scans chain on the main stream, and the two sweeps of a segment need only
    // its own scan: dq sweeps queue on one group of side streams, dk/dv sweeps and the dg epilogue on another
    // (round-robin by segment, so that neighbouring short segments share the device).
    const bool ov = overlap != 0 && fwd_workspace != nullptr;
    const sf_tuning_t tu = current_tuning();
    ChainRes* res = nullptr;
    if (ov) {
        SF_TRY(chain_resources(&res));
        SF_TRY(chain_events(res, 4 * (size_t)n_seg + 2 + 2 * kSweepStreams + kAggStreams));
        cudaEvent_t e0 = res->pool[4 * (size_t)n_seg];
        SF_CUDA(cudaEventRecord(e0, st));
        for (int s = 0; s <= 2 * kSweepStreams; ++s) SF_CUDA(cudaStreamWaitEvent(res->side[s], e0, 0));
        for (int s = 0; s < kAggStreams; ++s) SF_CUDA(cudaStreamWaitEvent(res->agg[s], e0, 0));
    }

    // per-segment offsets
    std::vector<size_t> fwd_off(n_seg), bwd_off(n_seg);
    std::vector<long long> tok0(n_seg);
    {
        size_t fo = 0, bo = 0;
        long long t = 0;
        for (int i = 0; i < n_seg; ++i) {
            sf_seg_desc_t d1 = chain_segment_desc(desc, seg_lens[i], n_seg);
            fwd_off[i] = fo; bwd_off[i] = bo; tok0[i] = t;
            fo += sf_workspace_bytes(&d1, 0);
            bo += sf_workspace_bytes(&d1, mode);
            t += seg_lens[i];
        }
    }
    auto seg_ptrs = [&](int i, const sf_seg_desc_t& t, const float* dS_next, float* dS_here) {
        const long long tok = tok0[i];
        return BwdPtrs{SeqPtr::at(q, tok, t.tok_stride_qk, esz), SeqPtr::at(k, tok, t.tok_stride_qk, esz),
                       SeqPtr::at(v, tok, t.tok_stride_v, esz),
                       static_cast<const float*>(SeqPtr::at(g, tok, t.tok_stride_g, sizeof(float))),
                       S_bounds + (size_t)i * sN, SeqPtr::at(dO, tok, t.tok_stride_v, esz), dS_next,
                       SeqPtr::at(dq, tok, t.tok_stride_qk, esz), SeqPtr::at(dk, tok, t.tok_stride_qk, esz),
                       SeqPtr::at(dv, tok, t.tok_stride_v, esz),
                       static_cast<float*>(SeqPtr::at(dg, tok, t.tok_stride_g, sizeof(float))), dS_here};
    };
    auto dS_buf = [&](int i) { return i == 0 ? dS_init : reinterpret_cast<float*>(base + (size_t)i * sB); };

    // backward aggregate of segment idx on its aggregate stream; with agg_ahead it first waits for the dk/dv sweep of
    // segment idx + agg_ahead (visited earlier; only called once that sweep has been enqueued)
    auto enqueue_agg = [&](int idx, bool throttled) -> sf_status_t {
        sf_seg_desc_t t = chain_segment_desc(desc, seg_lens[idx], n_seg);
        const Path path = classify(&t);
        const SegParams p = make_params(&t);
        const BwdWs w = bwd_ws(&t, p, seg_base + bwd_off[idx]);
        BwdPtrs x = seg_ptrs(idx, t, nullptr, nullptr);
        cudaStream_t s_agg = res->agg[agg_stream_index(p, idx, tu)];
        if (throttled) SF_CUDA(cudaStreamWaitEvent(s_agg, res->pool[4 * (size_t)(idx + tu.agg_ahead) + 3], 0));
        SF_TRY(bwd_pre(path, &t, p, x, w, nullptr, s_agg));
        SF_CUDA(cudaEventRecord(res->pool[4 * (size_t)idx], s_agg));
        return SF_OK;
    };
    if (ov && tu.agg_ahead == 0) {
        // no limit: all backward aggregates first, in the order the scans will need them
        for (int i = n_seg - 1; i >= 0; --i) SF_TRY(enqueue_agg(i, false));
    }
    const float* dS_next = dS_final;
    if (ov) {
        // (ov implies the forward workspace is given)  Groups of short neighbouring segments, visited in descending
        // order, share one reverse scan; each segment's sweeps start when its group's scan is done.
        for (int i = n_seg - 1; i >= 0;) {
            const int cnt = scan_group_size(seg_lens, n_seg, i, -1, tu.scan_group_tokens);
            struct Seg { sf_seg_desc_t t; Path path; SegParams p; BwdWs w; BwdPtrs x; FwdWs fw; };
            Seg sg[sf::SCAN_GROUP_MAX];
            sf::ScanGroup grp{};
            grp.count = cnt;
            const float* group_init = dS_next;
            for (int k = 0; k < cnt; ++k) {
                const int idx = i - k;
                Seg& s = sg[k];
                s.t = chain_segment_desc(desc, seg_lens[idx], n_seg);
                s.path = classify(&s.t);
                s.p = make_params(&s.t);
                s.w = bwd_ws(&s.t, s.p, seg_base + bwd_off[idx]);
                float* dS_here = dS_buf(idx);
                s.x = seg_ptrs(idx, s.t, dS_next, dS_here);
                s.fw = fwd_ws(&s.t, s.p, const_cast<char*>(static_cast<const char*>(fwd_workspace)) + fwd_off[idx]);
                grp.seg[k] = sf::ScanSeg{s.fw.beta, s.w.GU, dS_here, s.p.NB};
                dS_next = dS_here;
            }
            if (tu.agg_ahead > 0)
                for (int k = 0; k < cnt; ++k) SF_TRY(enqueue_agg(i - k, i - k + tu.agg_ahead <= n_seg - 1 && i - k + tu.agg_ahead > i));
            for (int k = 0; k < cnt; ++k) SF_CUDA(cudaStreamWaitEvent(st, res->pool[4 * (size_t)(i - k)], 0));
            SF_TRY(launch_scan_group(desc, desc->B * desc->H, grp, 1, group_init, st));
            cudaEvent_t e_scan = res->pool[4 * (size_t)i + 1];
            SF_CUDA(cudaEventRecord(e_scan, st));
            for (int k = 0; k < cnt; ++k) {
                const int idx = i - k;
                const Seg& s = sg[k];
                cudaEvent_t e_dq = res->pool[4 * (size_t)idx + 2];
                // the sweeps of neighbouring segments go round-robin to different streams
                cudaStream_t s_dq = res->side[1 + (idx % tu.sweep_streams)], s_kv = res->side[1 + kSweepStreams + (idx % tu.sweep_streams)];
                SF_CUDA(cudaStreamWaitEvent(s_dq, e_scan, 0));
                SF_CUDA(cudaStreamWaitEvent(s_kv, e_scan, 0));
                SF_TRY(bwd_dq(s.path, &s.t, s.p, s.x, s.w, s.fw.UH, s_dq));
                SF_CUDA(cudaEventRecord(e_dq, s_dq));
                SF_TRY(bwd_dkdv(s.path, &s.t, s.p, s.x, s.w, s_kv));
                SF_CUDA(cudaStreamWaitEvent(s_kv, e_dq, 0));
                SF_TRY(bwd_dg(&s.t, s.p, s.x, s.w, s.fw.UH, s_kv));
                SF_CUDA(cudaEventRecord(res->pool[4 * (size_t)idx + 3], s_kv));
            }
            i -= cnt;
        }
    } else {
        for (int i = n_seg - 1; i >= 0; --i) {
            sf_seg_desc_t t = chain_segment_desc(desc, seg_lens[i], n_seg);
            const Path path = classify(&t);
            const SegParams p = make_params(&t);
            char* wsi = seg_base + bwd_off[i];
            const BwdWs w = bwd_ws(&t, p, wsi);
            float* dS_here = dS_buf(i);
            BwdPtrs x = seg_ptrs(i, t, dS_next, dS_here);
            FwdWs fw;
            if (fwd_workspace) {
                fw = fwd_ws(&t, p, const_cast<char*>(static_cast<const char*>(fwd_workspace)) + fwd_off[i]);
            } else {
                char* fbase = wsi + w.bytes;
                fw = fwd_ws(&t, p, fbase);
                float* sfin = reinterpret_cast<float*>(fbase + fw.bytes);
                FwdPtrs fx{x.q, x.k, x.v, x.g, x.S_in, nullptr, sfin};
                SF_TRY(fwd_pre(path, &t, p, fx, fw, st));
                SF_TRY(fwd_scan(&t, p, fx, fw, st));
            }
            SF_TRY(bwd_pre(path, &t, p, x, w, nullptr, st));
            SF_TRY(bwd_scan(&t, p, x, w, fw.beta, st));
            SF_TRY(bwd_dq(path, &t, p, x, w, fw.UH, st));
            SF_TRY(bwd_dkdv(path, &t, p, x, w, st));
            SF_TRY(bwd_dg(&t, p, x, w, fw.UH, st));
            dS_next = dS_here;
        }
    }
    if (ov) {
        // join the side streams back into the caller's stream
        for (int s = 1; s <= 2 * kSweepStreams; ++s) {
            cudaEvent_t e = res->pool[4 * (size_t)n_seg + s];
            SF_CUDA(cudaEventRecord(e, res->side[s]));
            SF_CUDA(cudaStreamWaitEvent(st, e, 0));
        }
        for (int s = 0; s < kAggStreams; ++s) {
            cudaEvent_t e = res->pool[4 * (size_t)n_seg + 1 + 2 * kSweepStreams + s];
            SF_CUDA(cudaEventRecord(e, res->agg[s]));
            SF_CUDA(cudaStreamWaitEvent(st, e, 0));
        }
    }
    return SF_OK;
}

struct sf_chain_graph {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    long long kernels = 0;
};

sf_status_t sf_chain_graph_create(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, const void* q,
                                  const void* k, const void* v, const float* g, const float* S_init, void* o,
                                  float* S_bounds, void* fwd_workspace, size_t fwd_workspace_bytes, const void* dO,
                                  const float* dS_final, void* dq, void* dk, void* dv, float* dg, float* dS_init,
                                  void* bwd_workspace, size_t bwd_workspace_bytes, int32_t overlap, sf_stream_t stream,
                                  sf_chain_graph_t** out) {
    if (!out) return SF_ERR_INVALID_ARG;
    *out = nullptr;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (st == nullptr || st == cudaStreamLegacy) return SF_ERR_INVALID_ARG;
    {
        std::lock_guard<std::mutex> lk(g_timing_mu);
        if (g_timing_on) return SF_ERR_UNSUPPORTED;        // timing events do not belong in a graph
    }
    auto run = [&]() -> sf_status_t {
        SF_TRY(sf_chain_fwd(desc, seg_lens, n_seg, q, k, v, g, S_init, o, S_bounds, fwd_workspace, fwd_workspace_bytes,
                            overlap, stream));
        if (dO)
            SF_TRY(sf_chain_bwd(desc, seg_lens, n_seg, q, k, v, g, S_bounds, dO, dS_final, dq, dk, dv, dg, dS_init,
                                fwd_workspace, bwd_workspace, bwd_workspace_bytes, overlap, stream));
        return SF_OK;
    };
    // A plain pass first: it validates every argument and creates the per-process host objects (kernel attributes,
    // side streams, events) outside the capture.
    SF_TRY(run());
    const long long before = g_launches.load();
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return SF_ERR_CUDA; }
    const sf_status_t rs = run();
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(st, &graph);
    if (rs != SF_OK || ce != cudaSuccess || !graph) {
        cudaGetLastError();
        if (graph) cudaGraphDestroy(graph);
        return rs != SF_OK ? rs : SF_ERR_CUDA;
    }
    sf_chain_graph* h = new (std::nothrow) sf_chain_graph;
    if (!h) { cudaGraphDestroy(graph); return SF_ERR_CUDA; }
    h->graph = graph;
    h->kernels = g_launches.load() - before;
    if (cudaGraphInstantiate(&h->exec, graph, 0) != cudaSuccess) {
        cudaGetLastError();
        cudaGraphDestroy(graph);
        delete h;
        return SF_ERR_CUDA;
    }
    *out = h;
    return SF_OK;
}

sf_status_t sf_chain_graph_launch(sf_chain_graph_t* graph, sf_stream_t stream) {
    if (!graph || !graph->exec) return SF_ERR_INVALID_ARG;
    if (cudaGraphLaunch(graph->exec, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) { cudaGetLastError(); return SF_ERR_CUDA; }
    g_launches.fetch_add(graph->kernels, std::memory_order_relaxed);
    return SF_OK;
}

int64_t sf_chain_graph_kernels(const sf_chain_graph_t* graph) { return graph ? graph->kernels : 0; }

void sf_chain_graph_destroy(sf_chain_graph_t* graph) {
    if (!graph) return;
    if (graph->exec) cudaGraphExecDestroy(graph->exec);
    if (graph->graph) cudaGraphDestroy(graph->graph);
    delete graph;
}

sf_status_t sf_chain_autotune(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, const void* q,
                              const void* k, const void* v, const float* g, const float* S_init, void* o, float* S_bounds,
                              void* fwd_workspace, size_t fwd_workspace_bytes, const void* dO, const float* dS_final,
                              void* dq, void* dk, void* dv, float* dg, float* dS_init, void* bwd_workspace,
                              size_t bwd_workspace_bytes, const int32_t* candidates, int32_t n_cand, int32_t reps,
                              int32_t overlap, sf_stream_t stream, int32_t* best, float* ms) {
    if (!desc || !candidates || n_cand < 1 || reps < 1 || !best) return SF_ERR_INVALID_ARG;
    SF_TRY(validate_chain(desc, seg_lens, n_seg, nullptr));
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        cudaGetLastError();
        if (e0) cudaEventDestroy(e0);
        return SF_ERR_CUDA;
    }
    float best_ms = -1.f;
    sf_status_t result = SF_ERR_WORKSPACE;
    for (int c = 0; c < n_cand; ++c) {
        if (ms) ms[c] = -1.f;
        sf_seg_desc_t d = *desc;
        d.chunks_per_block = candidates[c];
        const size_t need_f = sf_chain_workspace_bytes(&d, seg_lens, n_seg, 0);
        const size_t need_b = dO ? sf_chain_workspace_bytes(&d, seg_lens, n_seg, 1) : 0;
        if (need_f == 0 || need_f > fwd_workspace_bytes || need_b > bwd_workspace_bytes) continue;
        // On a stream that can be captured the candidate is timed as a graph replay (what a tuned caller will most
        // likely run, and free of the host's launch cost, which hides the differences for short segments);
        // on the legacy default stream it is launched directly.
        sf_chain_graph_t* graph = nullptr;
        auto run = [&]() -> sf_status_t {
            if (graph) return sf_chain_graph_launch(graph, stream);
            SF_TRY(sf_chain_fwd(&d, seg_lens, n_seg, q, k, v, g, S_init, o, S_bounds, fwd_workspace, fwd_workspace_bytes,
                                overlap, stream));
            if (dO)
                SF_TRY(sf_chain_bwd(&d, seg_lens, n_seg, q, k, v, g, S_bounds, dO, dS_final, dq, dk, dv, dg, dS_init,
                                    fwd_workspace, bwd_workspace, bwd_workspace_bytes, overlap, stream));
            return SF_OK;
        };
        sf_status_t rs;
        if (st != nullptr && st != cudaStreamLegacy) {
            rs = sf_chain_graph_create(&d, seg_lens, n_seg, q, k, v, g, S_init, o, S_bounds, fwd_workspace,
                                       fwd_workspace_bytes, dO, dS_final, dq, dk, dv, dg, dS_init, bwd_workspace,
                                       bwd_workspace_bytes, overlap, stream, &graph);       // runs the chain once itself
            if (rs == SF_OK) rs = run();
        } else {
            rs = run();                                           // untimed: first-use costs of this shape
        }
        if (rs == SF_ERR_UNSUPPORTED || rs == SF_ERR_INVALID_ARG) {  // this value is not available for this shape
            if (result != SF_OK) result = rs;
            sf_chain_graph_destroy(graph);
            continue;
        }
        bool ok = rs == SF_OK && cudaEventRecord(e0, st) == cudaSuccess;
        for (int r = 0; ok && r < reps; ++r) ok = (rs = run()) == SF_OK;
        float t = 0.f;
        ok = ok && cudaEventRecord(e1, st) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess &&
             cudaEventElapsedTime(&t, e0, e1) == cudaSuccess;
        sf_chain_graph_destroy(graph);
        if (!ok) {
            cudaGetLastError();
            result = rs != SF_OK ? rs : SF_ERR_CUDA;
            break;
        }
        t /= (float)reps;
        if (ms) ms[c] = t;
        if (best_ms < 0.f || t < best_ms) { best_ms = t; *best = candidates[c]; }
        result = SF_OK;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return result;
}

sf_status_t sf_chain_autotune_schedule(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, const void* q,
                                       const void* k, const void* v, const float* g, const float* S_init, void* o,
                                       float* S_bounds, void* fwd_workspace, size_t fwd_workspace_bytes, const void* dO,
                                       const float* dS_final, void* dq, void* dk, void* dv, float* dg, float* dS_init,
                                       void* bwd_workspace, size_t bwd_workspace_bytes, int32_t reps, float margin,
                                       sf_stream_t stream, sf_tuning_t* chosen, float* chosen_ms, float* default_ms) {
    if (!desc || reps < 1 || !(margin >= 0.f) || !chosen) return SF_ERR_INVALID_ARG;
    // a small set of valid schedules, the default first
    std::vector<sf_tuning_t> grid;
    grid.push_back(kDefaultTuning);
    for (int ahead : {0, 1, 2})
        for (int sweeps : {2, 4})
            for (int inorder : {1, 74}) {
                sf_tuning_t t = kDefaultTuning;
                t.agg_ahead = ahead; t.sweep_streams = sweeps; t.agg_inorder_ctas = inorder;
                if (ahead == 0 && sweeps == 4 && inorder == 74) continue;       // the default itself
                grid.push_back(t);
            }
    {
        sf_tuning_t t = kDefaultTuning;
        t.merge_launches = 1;                                                    // one launch per stage over the whole chain
        grid.push_back(t);
    }
    const sf_tuning_t before = current_tuning();
    const int32_t cand = desc->chunks_per_block;
    float best_ms = -1.f, def_ms = -1.f;
    sf_tuning_t best = kDefaultTuning;
    sf_status_t result = SF_OK;
    for (size_t i = 0; i < grid.size(); ++i) {
        if (sf_set_tuning(&grid[i]) != SF_OK) continue;
        int32_t b = 0;
        float ms = -1.f;
        const sf_status_t st = sf_chain_autotune(desc, seg_lens, n_seg, q, k, v, g, S_init, o, S_bounds, fwd_workspace,
                                                 fwd_workspace_bytes, dO, dS_final, dq, dk, dv, dg, dS_init, bwd_workspace,
                                                 bwd_workspace_bytes, &cand, 1, reps, 1, stream, &b, &ms);
        if (st != SF_OK) { result = st; break; }
        if (i == 0) def_ms = ms;
        if (best_ms < 0.f || ms < best_ms) { best_ms = ms; best = grid[i]; }
    }
    if (result != SF_OK) { sf_set_tuning(&before); return result; }
    // the default stays unless something beats it by more than the margin (differences below that are noise)
    if (def_ms > 0.f && def_ms <= (1.f + margin) * best_ms) { best = kDefaultTuning; best_ms = def_ms; }
    sf_set_tuning(&best);
    *chosen = best;
    if (chosen_ms) *chosen_ms = best_ms;
    if (default_ms) *default_ms = def_ms;
    return SF_OK;
}

sf_status_t sf_partition_hybrid(int64_t T, int32_t N, double w_tok, double w_soft, double alpha, int32_t multiple,
                                int32_t* seg_lens) {
    if (T < 1 || N < 1 || multiple < 1 || !seg_lens) return SF_ERR_INVALID_ARG;
    if (!(w_tok >= 0.0) || !(w_soft >= 0.0) || (w_tok == 0.0 && w_soft == 0.0) || !std::isfinite(alpha) ||
        !std::isfinite(w_tok) || !std::isfinite(w_soft))
        return SF_ERR_INVALID_ARG;
    if ((int64_t)N * multiple > T || T > INT32_MAX) return SF_ERR_INVALID_ARG;
    // Equal Cost_i (Eq. 10) means the cost accumulated over the prefix [0, c), acc(c) = w_tok*c + w_soft*c^2/2
    // (Cost_i = acc(c_{i+1}) - acc(c_i) by Eq. 9), grows by the same amount per segment: acc(c_i) = (i/N) acc(T).
    // The positive root of that quadratic, in the form that stays exact as w_soft -> 0:
    //     c_i = 2 K_i / (w_tok + sqrt(w_tok^2 + 2 w_soft K_i)),   K_i = (i/N) acc(T)
    const double Td = (double)T, accT = w_tok * Td + 0.5 * w_soft * Td * Td;
    std::vector<long long> r(N + 1);
    r[0] = 0;
    r[N] = T;
    for (int i = 1; i < N; ++i) {
        const double K = accT * ((double)i / (double)N);
        const double hybrid = 2.0 * K / (w_tok + std::sqrt(w_tok * w_tok + 2.0 * w_soft * K));
        const double c = (1.0 - alpha) * (Td * (double)i / (double)N) + alpha * hybrid;              // Eq. 11
        r[i] = (long long)std::floor(c / (double)multiple + 0.5) * (long long)multiple;
    }
    for (int i = 1; i < N; ++i) r[i] = std::max(r[i], r[i - 1] + multiple);
    for (int i = N - 1; i >= 1; --i) r[i] = std::min(r[i], r[i + 1] - multiple);
    if (N > 1 && r[1] < multiple) return SF_ERR_INVALID_ARG;
    for (int i = 0; i < N; ++i) seg_lens[i] = (int32_t)(r[i + 1] - r[i]);
    return SF_OK;
}

namespace {
// Device-buffer plan of the host wrapper: per-segment forward workspaces (kept for the backward), one backward
// workspace (the segments' backward passes run one after the other on the caller's stream).
struct E2ePlan { std::vector<size_t> wf; size_t wf_total = 0, wb = 0; };
E2ePlan e2e_plan(const sf_seg_desc_t* d, const int32_t* seg_lens, int32_t n_seg) {
    E2ePlan pl;
    pl.wf.resize(n_seg);
    for (int i = 0; i < n_seg; ++i) {
        pl.wf[i] = align_up(sf_chain_workspace_bytes(d, seg_lens + i, 1, 0));
        pl.wf_total += pl.wf[i];
        pl.wb = std::max(pl.wb, align_up(sf_chain_workspace_bytes(d, seg_lens + i, 1, 1)));
    }
    return pl;
}
}  // namespace

size_t sf_e2e_device_bytes(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg) {
    long long T = 0;
    if (validate_chain(desc, seg_lens, n_seg, &T) != SF_OK) return 0;
    const size_t esz = desc->dtype == SF_BF16 ? 2 : 4;
    const size_t nqk = align_up((size_t)desc->B * T * desc->H * desc->d_k * esz);
    const size_t nv = align_up((size_t)desc->B * T * desc->H * desc->d_v * esz);
    const size_t ng = align_up((size_t)desc->B * T * desc->H * sizeof(float));
    const size_t sB = state_bytes(desc);
    const E2ePlan pl = e2e_plan(desc, seg_lens, n_seg);
    return 4 * nqk + 4 * nv + 2 * ng + (size_t)(n_seg + 1) * sB + 3 * sB + pl.wf_total + pl.wb;
}

sf_status_t sf_chain_fwd_bwd_host(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg, const void* q,
                                  const void* k, const void* v, const float* g, const float* S_init, const void* dO,
                                  const float* dS_final, void* o, float* S_final, void* dq, void* dk, void* dv, float* dg,
                                  float* dS_init, void* dev, size_t dev_bytes, sf_stream_t stream) {
    long long T = 0;
    SF_TRY(validate_chain(desc, seg_lens, n_seg, &T));
    if (!q || !k || !v || !g || !dO || !o || !dq || !dk || !dv || !dg || !dS_init) return SF_ERR_INVALID_ARG;
    if (!dev || dev_bytes < sf_e2e_device_bytes(desc, seg_lens, n_seg)) return SF_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(dev) % kAlign) return SF_ERR_INVALID_ARG;
    // the wrapper works on a densely packed device copy
    sf_seg_desc_t d = *desc;
    if (d.tok_stride_qk != (long long)d.H * d.d_k || d.tok_stride_v != (long long)d.H * d.d_v || d.tok_stride_g != d.H)
        return SF_ERR_INVALID_ARG;
    if (d.B > 1 && (d.batch_stride_qk != T * d.tok_stride_qk || d.batch_stride_v != T * d.tok_stride_v ||
                    d.batch_stride_g != T * d.tok_stride_g))
        return SF_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t esz = d.dtype == SF_BF16 ? 2 : 4;
    const size_t rqk = (size_t)d.H * d.d_k * esz, rv = (size_t)d.H * d.d_v * esz, rg = (size_t)d.H * sizeof(float);   // bytes per token
    const size_t bqk = (size_t)d.B * T * rqk, bv = (size_t)d.B * T * rv, bg = (size_t)d.B * T * rg;
    const size_t nqk = align_up(bqk), nv = align_up(bv), ng = align_up(bg), sB = state_bytes(&d);
    const size_t sN = (size_t)d.B * d.H * d.d_k * d.d_v, sbytes = sN * sizeof(float);
    const E2ePlan pl = e2e_plan(&d, seg_lens, n_seg);
    char* c = static_cast<char*>(dev);
    auto take = [&](size_t n) { char* r = c; c += n; return r; };
    char *dq_ = take(nqk), *dk_ = take(nqk), *q_ = take(nqk), *k_ = take(nqk);
    char *v_ = take(nv), *dO_ = take(nv), *o_ = take(nv), *dv_ = take(nv);
    char *g_ = take(ng), *dg_ = take(ng);
    float* bounds = reinterpret_cast<float*>(take((size_t)(n_seg + 1) * sB));      // indexed densely (sN floats apart)
    float* dsfin = reinterpret_cast<float*>(take(sB));
    float* dsbuf[2] = {reinterpret_cast<float*>(take(sB)), nullptr};
    dsbuf[1] = reinterpret_cast<float*>(take(sB));
    char* wsf = take(pl.wf_total);
    char* wsb = take(pl.wb);

    // The chain is pipelined segment by segment against the copies, so that both PCIe directions carry data for most
    // of the call (a step moves far more bytes over PCIe than the kernels take time for):
    //   upload stream   : q, k, v, g of segment 0, 1, ... n-1, then dO of segment n-1, n-2, ... 0
    //   caller's stream : [wait inputs(i)] forward(i) ...          then [wait dO(i)] backward(i) for i = n-1 ... 0
    //   download stream : [wait forward(i)] o(i) ...               then [wait backward(i)] dq, dk, dv, dg of segment i
    // Segment i is one time slice of every [B, T, H, d] tensor: B rows of len*H*d elements, T*H*d apart.
    ChainRes* res = nullptr;
    SF_TRY(chain_resources(&res));
    cudaStream_t up = res->copy[0], down = res->copy[1];
    std::vector<cudaEvent_t> ev(4 * (size_t)n_seg + 2, nullptr);
    struct EventGuard {
        std::vector<cudaEvent_t>& e;
        ~EventGuard() { for (cudaEvent_t x : e) if (x) cudaEventDestroy(x); }
    } guard{ev};
    for (auto& e : ev) SF_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    cudaEvent_t* e_in = ev.data();                   // inputs of segment i on the device
    cudaEvent_t* e_dO = ev.data() + n_seg;           // dO of segment i on the device
    cudaEvent_t* e_f = ev.data() + 2 * (size_t)n_seg;   // forward of segment i done
    cudaEvent_t* e_b = ev.data() + 3 * (size_t)n_seg;   // backward of segment i done
    cudaEvent_t e_start = ev[4 * (size_t)n_seg], e_end = ev[4 * (size_t)n_seg + 1];
    auto slice = [&](void* dst, const void* src, size_t row, long long tok, long long len, cudaMemcpyKind kind, cudaStream_t s) {
        const size_t pitch = (size_t)T * row;        // one plain copy per batch row (a 2-D copy would cap the pitch at 2 GB)
        for (int b = 0; b < d.B; ++b) {
            const size_t off = (size_t)b * pitch + (size_t)tok * row;
            const cudaError_t e = cudaMemcpyAsync(static_cast<char*>(dst) + off, static_cast<const char*>(src) + off, (size_t)len * row, kind, s);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    };
    std::vector<long long> tok0(n_seg + 1, 0);
    for (int i = 0; i < n_seg; ++i) tok0[i + 1] = tok0[i] + seg_lens[i];

    SegmentOfChain sub_calls;
    SF_CUDA(cudaEventRecord(e_start, st));
    SF_CUDA(cudaStreamWaitEvent(up, e_start, 0));
    SF_CUDA(cudaStreamWaitEvent(down, e_start, 0));
    if (S_init) SF_CUDA(cudaMemcpyAsync(bounds, S_init, sbytes, cudaMemcpyHostToDevice, up));
    else        SF_CUDA(cudaMemsetAsync(bounds, 0, sbytes, up));
    for (int i = 0; i < n_seg; ++i) {
        SF_CUDA(slice(q_, q, rqk, tok0[i], seg_lens[i], cudaMemcpyHostToDevice, up));
        SF_CUDA(slice(k_, k, rqk, tok0[i], seg_lens[i], cudaMemcpyHostToDevice, up));
        SF_CUDA(slice(v_, v, rv, tok0[i], seg_lens[i], cudaMemcpyHostToDevice, up));
        SF_CUDA(slice(g_, g, rg, tok0[i], seg_lens[i], cudaMemcpyHostToDevice, up));
        SF_CUDA(cudaEventRecord(e_in[i], up));
    }
    if (dS_final) SF_CUDA(cudaMemcpyAsync(dsfin, dS_final, sbytes, cudaMemcpyHostToDevice, up));
    for (int i = n_seg - 1; i >= 0; --i) {
        SF_CUDA(slice(dO_, dO, rv, tok0[i], seg_lens[i], cudaMemcpyHostToDevice, up));
        SF_CUDA(cudaEventRecord(e_dO[i], up));
    }
    // forward, segment by segment as the inputs arrive; the boundary state of segment i is already in bounds[i]
    {
        size_t off = 0;
        for (int i = 0; i < n_seg; ++i) {
            float* b_i = bounds + (size_t)i * sN;
            SF_CUDA(cudaStreamWaitEvent(st, e_in[i], 0));
            SF_TRY(sf_chain_fwd(&d, seg_lens + i, 1, q_ + tok0[i] * rqk, k_ + tok0[i] * rqk, v_ + tok0[i] * rv,
                                reinterpret_cast<float*>(g_ + tok0[i] * rg), b_i, o_ + tok0[i] * rv, b_i, wsf + off, pl.wf[i], 0, stream));
            SF_CUDA(cudaEventRecord(e_f[i], st));
            SF_CUDA(cudaStreamWaitEvent(down, e_f[i], 0));
            SF_CUDA(slice(o, o_, rv, tok0[i], seg_lens[i], cudaMemcpyDeviceToHost, down));
            off += pl.wf[i];
        }
        if (S_final) SF_CUDA(cudaMemcpyAsync(S_final, bounds + (size_t)n_seg * sN, sbytes, cudaMemcpyDeviceToHost, down));
    }
    // backward, last segment first as its dO arrives; dS ping-pongs between two buffers
    {
        size_t off = pl.wf_total;
        const float* ds_out = dS_final ? dsfin : nullptr;
        for (int i = n_seg - 1; i >= 0; --i) {
            off -= pl.wf[i];
            float* ds_in = dsbuf[i & 1];
            SF_CUDA(cudaStreamWaitEvent(st, e_dO[i], 0));
            SF_TRY(sf_chain_bwd(&d, seg_lens + i, 1, q_ + tok0[i] * rqk, k_ + tok0[i] * rqk, v_ + tok0[i] * rv,
                                reinterpret_cast<float*>(g_ + tok0[i] * rg), bounds + (size_t)i * sN, dO_ + tok0[i] * rv, ds_out,
                                dq_ + tok0[i] * rqk, dk_ + tok0[i] * rqk, dv_ + tok0[i] * rv, reinterpret_cast<float*>(dg_ + tok0[i] * rg),
                                ds_in, wsf + off, wsb, pl.wb, 0, stream));
            SF_CUDA(cudaEventRecord(e_b[i], st));
            SF_CUDA(cudaStreamWaitEvent(down, e_b[i], 0));
            SF_CUDA(slice(dq, dq_, rqk, tok0[i], seg_lens[i], cudaMemcpyDeviceToHost, down));
            SF_CUDA(slice(dk, dk_, rqk, tok0[i], seg_lens[i], cudaMemcpyDeviceToHost, down));
            SF_CUDA(slice(dv, dv_, rv, tok0[i], seg_lens[i], cudaMemcpyDeviceToHost, down));
            SF_CUDA(slice(dg, dg_, rg, tok0[i], seg_lens[i], cudaMemcpyDeviceToHost, down));
            ds_out = ds_in;
        }
        SF_CUDA(cudaMemcpyAsync(dS_init, dsbuf[0], sbytes, cudaMemcpyDeviceToHost, down));
    }
    SF_CUDA(cudaEventRecord(e_end, down));
    SF_CUDA(cudaStreamWaitEvent(st, e_end, 0));
    SF_CUDA(cudaStreamSynchronize(st));
    return SF_OK;
}

sf_status_t sf_set_tuning(const sf_tuning_t* t) {
    std::lock_guard<std::mutex> lk(g_tuning_mu);
    if (!t) { g_tuning = kDefaultTuning; return SF_OK; }
    if (t->sweep_streams < 1 || t->sweep_streams > kMaxSweepStreams || t->agg_streams < 1 || t->agg_streams > kMaxAggStreams ||
        t->scan_group_tokens < 0 || t->agg_inorder_ctas < 1 || t->agg_ahead < 0 || t->merge_launches < 0 || t->merge_launches > 1)
        return SF_ERR_INVALID_ARG;
    g_tuning = *t;
    return SF_OK;
}

void sf_get_tuning(sf_tuning_t* t) {
    if (t) *t = current_tuning();
}

int32_t sf_device_status(void) { return sf::tc::read_device_status(); }

sf_status_t sf_device_check(void) {
    const int v = sf::tc::read_device_status();
    return v < 0 ? SF_ERR_CUDA : (v == 0 ? SF_OK : SF_ERR_TIMEOUT);
}

sf_status_t sf_selftest_bounded_wait(int64_t limit_cycles, sf_stream_t stream) {
    if (limit_cycles < 1 || limit_cycles > 100000000LL) return SF_ERR_INVALID_ARG;     // at most a few hundredths of a second
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    SF_TRY(sf::tc::launch_wait_selftest(limit_cycles, st));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return SF_ERR_CUDA; }
    return sf_device_check();
}
void sf_device_status_clear(void) { sf::tc::clear_device_status(); }
int64_t sf_launch_count(void) { return g_launches.load(); }

void sf_stage_timing(int32_t enable) {
    std::lock_guard<std::mutex> lk(g_timing_mu);
    g_timing_on = enable != 0;
}

int32_t sf_stage_timing_read(float* ms, int64_t* launches, int32_t n) {
    cudaDeviceSynchronize();
    std::lock_guard<std::mutex> lk(g_timing_mu);
    for (int i = 0; i < n; ++i) { ms[i] = 0.f; launches[i] = 0; }
    for (auto& t : g_timed) {
        float e = 0.f;
        if (cudaEventElapsedTime(&e, t.a, t.b) == cudaSuccess && t.stage < n) { ms[t.stage] += e; launches[t.stage] += 1; }
        else cudaGetLastError();
        cudaEventDestroy(t.a);
        cudaEventDestroy(t.b);
    }
    g_timed.clear();
    return ST_COUNT;
}

}  // extern "C"

// Launches made by the library's other translation units count too.
namespace sf { void note_launches(long long n) { g_launches.fetch_add(n, std::memory_order_relaxed); } }
