// C ABI of the extension operators: diagonal decay, gated delta rule, short convolution with a carried tail.
// Argument checks happen before any launch; nothing here allocates, synchronises or falls back to the host.
#include <type_traits>
#include "../../include/stateflow.h"
#include "sf_recurrent.cuh"
#include "sf_delta_chunk.cuh"
#include "sf_channel_chunk.cuh"

namespace sf { void note_launches(long long n); }

namespace {

using sf::rec::RecParams;

bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }
bool aligned2(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 1u) == 0; }

sf_status_t check_desc(const sf_seg_desc_t* d, bool wide_keys = false) {
    if (!d) return SF_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->seg_len <= 0 || d->d_k <= 0 || d->d_v <= 0) return SF_ERR_INVALID_ARG;
    if (d->B > 65535) return SF_ERR_INVALID_ARG;                                       // grid.y
    if (d->tok_stride_qk < (long long)d->H * d->d_k || d->tok_stride_v < (long long)d->H * d->d_v || d->tok_stride_g < d->H)
        return SF_ERR_INVALID_ARG;
    if (d->B > 1 && (d->batch_stride_qk <= 0 || d->batch_stride_v <= 0 || d->batch_stride_g <= 0)) return SF_ERR_INVALID_ARG;
    if (d->dtype != SF_F32 && d->dtype != SF_BF16) return SF_ERR_INVALID_ARG;
    const bool k_ok = d->d_k == 32 || d->d_k == 64 || (wide_keys && d->d_k == 128);
    const bool v_ok = d->d_v == 32 || d->d_v == 64 || d->d_v == 128;
    return k_ok && v_ok ? SF_OK : SF_ERR_UNSUPPORTED;
}

RecParams make_params(const sf_seg_desc_t* d) {
    RecParams p;
    p.B = d->B; p.H = d->H; p.L = d->seg_len;
    p.tqk = d->tok_stride_qk; p.tv = d->tok_stride_v; p.tg = d->tok_stride_g;
    p.bqk = d->batch_stride_qk; p.bv = d->batch_stride_v; p.bg = d->batch_stride_g;
    return p;
}

size_t ws_bytes(const sf_seg_desc_t* d) {
    return (size_t)d->B * d->H * (size_t)sf::rec::ws_states(d->seg_len) * d->d_k * d->d_v * sizeof(float);
}

sf_status_t launched(int n = 1) {
    sf::note_launches(n);
    return cudaGetLastError() == cudaSuccess ? SF_OK : SF_ERR_CUDA;
}

template <int VAR, typename T>
sf_status_t rec_fwd_t(const sf_seg_desc_t* d, const RecParams& p, const void* q, const void* k, const void* v, const float* g,
                      const float* beta, const float* S_in, void* o, float* S_out, cudaStream_t st) {
    const dim3 grid(d->H, d->B);
    const T *tq = static_cast<const T*>(q), *tk = static_cast<const T*>(k), *tv = static_cast<const T*>(v);
    T* to = static_cast<T*>(o);
#define SF_REC_FWD(DK, DV)                                                                                         \
    if (d->d_k == DK && d->d_v == DV) {                                                                            \
        sf::rec::rec_fwd_kernel<T, DK, DV, VAR><<<grid, DV, 0, st>>>(p, tq, tk, tv, g, beta, S_in, to, S_out);     \
        return launched();                                                                                         \
    }
    SF_REC_FWD(32, 32) SF_REC_FWD(32, 64) SF_REC_FWD(32, 128) SF_REC_FWD(64, 32) SF_REC_FWD(64, 64) SF_REC_FWD(64, 128)
#undef SF_REC_FWD
    return SF_ERR_UNSUPPORTED;
}

template <int VAR>
sf_status_t rec_fwd(const sf_seg_desc_t* d, const void* q, const void* k, const void* v, const float* g, const float* beta,
                    const float* S_in, void* o, float* S_out, cudaStream_t st) {
    const sf_status_t c = check_desc(d);
    if (c != SF_OK) return c;
    if (!q || !k || !v || !g || !o || !S_out || (VAR == sf::rec::DELTA && !beta)) return SF_ERR_INVALID_ARG;
    if (S_in == S_out) return SF_ERR_INVALID_ARG;
    const bool f32 = d->dtype == SF_F32;
    auto al = [&](const void* x) { return f32 ? aligned4(x) : aligned2(x); };
    if (!al(q) || !al(k) || !al(v) || !al(o) || !aligned4(g) || !aligned4(S_out)) return SF_ERR_INVALID_ARG;
    const RecParams p = make_params(d);
    return f32 ? rec_fwd_t<VAR, float>(d, p, q, k, v, g, beta, S_in, o, S_out, st)
               : rec_fwd_t<VAR, __nv_bfloat16>(d, p, q, k, v, g, beta, S_in, o, S_out, st);
}

template <int VAR, typename T>
sf_status_t rec_bwd_t(const sf_seg_desc_t* d, const RecParams& p, const void* q, const void* k, const void* v, const float* g,
                      const float* beta, const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv,
                      float* dg, float* dbeta, float* dS_in, float* w, cudaStream_t st) {
    const dim3 grid(d->H, d->B);
    const T *tq = static_cast<const T*>(q), *tk = static_cast<const T*>(k), *tv = static_cast<const T*>(v),
            *tdo = static_cast<const T*>(dO);
    T *tdq = static_cast<T*>(dq), *tdk = static_cast<T*>(dk), *tdv = static_cast<T*>(dv);
#define SF_REC_BWD(DK, DV)                                                                                         \
    if (d->d_k == DK && d->d_v == DV) {                                                                            \
        sf::rec::rec_bwd_kernel<T, DK, DV, VAR><<<grid, DV, 0, st>>>(p, tq, tk, tv, g, beta, S_in, tdo, dS_out, tdq, tdk, \
                                                                     tdv, dg, dbeta, dS_in, w);                    \
        return launched();                                                                                         \
    }
    SF_REC_BWD(32, 32) SF_REC_BWD(32, 64) SF_REC_BWD(32, 128) SF_REC_BWD(64, 32) SF_REC_BWD(64, 64) SF_REC_BWD(64, 128)
#undef SF_REC_BWD
    return SF_ERR_UNSUPPORTED;
}

template <int VAR>
sf_status_t rec_bwd(const sf_seg_desc_t* d, const void* q, const void* k, const void* v, const float* g, const float* beta,
                    const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv, float* dg,
                    float* dbeta, float* dS_in, void* ws, size_t bytes, cudaStream_t st) {
    const sf_status_t c = check_desc(d);
    if (c != SF_OK) return c;
    if (!q || !k || !v || !g || !dO || !dq || !dk || !dv || !dg || !dS_in) return SF_ERR_INVALID_ARG;
    if (VAR == sf::rec::DELTA && (!beta || !dbeta)) return SF_ERR_INVALID_ARG;
    if (dS_in == dS_out) return SF_ERR_INVALID_ARG;
    if (!ws || bytes < ws_bytes(d) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return SF_ERR_WORKSPACE;
    const RecParams p = make_params(d);
    float* w = static_cast<float*>(ws);
    return d->dtype == SF_F32
        ? rec_bwd_t<VAR, float>(d, p, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, w, st)
        : rec_bwd_t<VAR, __nv_bfloat16>(d, p, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, w, st);
}

sf_status_t check_conv(int32_t B, int32_t L, int32_t C, int32_t W) {
    if (B <= 0 || L <= 0 || C <= 0 || W < 1) return SF_ERR_INVALID_ARG;
    if (W > sf::rec::CONV_MAXW || B > 65535) return SF_ERR_UNSUPPORTED;       // B is a grid dimension
    return SF_OK;
}

// Launch shape of the row-walking convolution kernels over `rows` rows: V channels per thread (4 when the channel
// count and every pointer allow 16-byte accesses).
bool conv_vec4(int C, std::initializer_list<const void*> ptrs) {
    if (C % 4) return false;
    for (const void* p : ptrs) if (p && (reinterpret_cast<uintptr_t>(p) & 15u)) return false;
    return true;
}
// Calls f with the convolution width as a compile-time constant (1 .. CONV_MAXW, checked before).
template <class F>
void conv_width_switch(int W, F&& f) {
    switch (W) {
        case 1: f(std::integral_constant<int, 1>{}); break;
        case 2: f(std::integral_constant<int, 2>{}); break;
        case 3: f(std::integral_constant<int, 3>{}); break;
        case 4: f(std::integral_constant<int, 4>{}); break;
        case 5: f(std::integral_constant<int, 5>{}); break;
        case 6: f(std::integral_constant<int, 6>{}); break;
        case 7: f(std::integral_constant<int, 7>{}); break;
        default: f(std::integral_constant<int, 8>{}); break;
    }
}
dim3 conv_grid(int B, long long rows, int C, int V) {
    const int groups = (C + V - 1) / V;
    return dim3((unsigned)((groups + 31) / 32), (unsigned)((rows + 8LL * sf::rec::CONV_TS - 1) / (8LL * sf::rec::CONV_TS)), (unsigned)B);
}

// ---- chunkwise delta rule ----------------------------------------------------------------------------------------
constexpr size_t kMaxSmem = 227 * 1024;       // dynamic shared memory a CTA can opt into on this architecture

// `delta`: the delta-rule kernels, else the diagonal-decay ones; the shape is supported if every kernel's tiles fit
sf_status_t check_chunked(const sf_seg_desc_t* d, bool delta) {
    const sf_status_t c = check_desc(d, true);
    if (c != SF_OK) return c;
    if (d->chunk <= 0) return SF_ERR_INVALID_ARG;
    if (d->chunk != 16 && d->chunk != 32) return SF_ERR_UNSUPPORTED;
    if (d->H > 65535) return SF_ERR_INVALID_ARG;
    const size_t need = delta ? sf::gdn::smem_max(d->chunk, d->d_k, d->d_v) : sf::dcc::smem_max(d->chunk, d->d_k, d->d_v);
    return need <= kMaxSmem ? SF_OK : SF_ERR_UNSUPPORTED;
}

sf::gdn::Params chunked_params(const sf_seg_desc_t* d) {
    sf::gdn::Params p;
    p.B = d->B; p.H = d->H; p.L = d->seg_len; p.C = d->chunk; p.NC = (d->seg_len + d->chunk - 1) / d->chunk;
    p.dk = d->d_k; p.dv = d->d_v;
    p.tqk = d->tok_stride_qk; p.tv = d->tok_stride_v; p.tg = d->tok_stride_g;
    p.bqk = d->batch_stride_qk; p.bv = d->batch_stride_v; p.bg = d->batch_stride_g;
    return p;
}

size_t chunked_ws_bytes(const sf_seg_desc_t* d, bool backward) {
    return (size_t)d->B * d->H * sf::gdn::ws_floats(chunked_params(d), backward) * sizeof(float);
}

template <typename K>
bool opt_in(K kern, size_t bytes) {
    if (bytes <= 48 * 1024) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) { cudaGetLastError(); return false; }
    return true;
}

// The sequential state pass (forward or reverse) of the chunkwise delta rule: two levels (maps composed over blocks of GR
// chunks, a pass over the blocks, the chunks of all blocks in parallel) when the segment has more chunks than one block and
// the composing kernel's tiles fit into shared memory, else one pass over the chunks.  Returns the number of launches.
int delta_state_pass(const sf::gdn::Params& p, bool reverse, const float* init, float* fin, float* ws, int backward, cudaStream_t st) {
    using namespace sf::gdn;
    const dim3 cols(p.dv / DVS, p.H, p.B);
    const size_t s2 = smem_chain(p.dk), sc = smem_compose(p.dk, p.dv);
    const int NB = (p.NC + GR - 1) / GR;
    const bool wide = p.dk > 64;
    auto chain = [&](dim3 grid, int mode, const float* i0, float* f0) {
        if (wide) chain_kernel<128><<<grid, NT, s2, st>>>(p, mode, i0, f0, ws, backward);
        else      chain_kernel<64><<<grid, NT, s2, st>>>(p, mode, i0, f0, ws, backward);
    };
    if (p.NC > GR && sc <= kMaxSmem && (long long)p.B * p.H <= 65535) {
        compose_kernel<<<dim3(NB, p.H, p.B), NT, sc, st>>>(p, reverse ? 1 : 0, ws, backward);
        chain(cols, reverse ? BLOCKS_REV : BLOCKS_FWD, init, fin);
        chain(dim3(p.dv / DVS, NB, p.B * p.H), reverse ? INBLOCK_REV : INBLOCK_FWD, nullptr, nullptr);
        return 3;
    }
    chain(cols, reverse ? CHUNKS_REV : CHUNKS_FWD, init, fin);
    return 1;
}

// Pre + ST (+ Out when o != NULL); the backward calls it with o == NULL to rebuild the chunk states.
template <typename T>
sf_status_t chunked_forward(const sf_seg_desc_t* d, const sf::gdn::Params& p, const void* q, const void* k, const void* v,
                            const float* g, const float* beta, const float* S_in, void* o, float* S_out, float* ws, int backward,
                            cudaStream_t st) {
    using namespace sf::gdn;
    const T *tq = static_cast<const T*>(q), *tk = static_cast<const T*>(k), *tv = static_cast<const T*>(v);
    const dim3 chunks(p.NC, p.H, p.B), cols(p.dv / DVS, p.H, p.B);
    const size_t s1 = smem_pre(p.C, p.dk, p.dv), s2 = smem_chain(p.dk), s3 = smem_out(p.C, p.dk, p.dv);
    const size_t sc = smem_compose(p.dk, p.dv);
    if (!opt_in(pre_kernel<T>, s1) || !opt_in(chain_kernel<64>, s2) || !opt_in(chain_kernel<128>, s2) || !opt_in(out_kernel<T>, s3) ||
        (sc <= kMaxSmem && !opt_in(compose_kernel, sc)))
        return SF_ERR_CUDA;
    pre_kernel<T><<<chunks, NT, s1, st>>>(p, tq, tk, tv, g, beta, ws, backward);
    int n = 1 + delta_state_pass(p, false, S_in, S_out, ws, backward, st);
    if (o) { out_kernel<T><<<chunks, NT, s3, st>>>(p, tq, tk, g, static_cast<T*>(o), ws, backward); ++n; }
    return launched(n);
}

template <typename T>
sf_status_t chunked_backward(const sf_seg_desc_t* d, const sf::gdn::Params& p, const void* q, const void* k, const void* v,
                             const float* g, const float* beta, const float* S_in, const void* dO, const float* dS_out, void* dq,
                             void* dk, void* dv, float* dg, float* dbeta, float* dS_in, float* ws, cudaStream_t st) {
    using namespace sf::gdn;
    const sf_status_t f = chunked_forward<T>(d, p, q, k, v, g, beta, S_in, nullptr, nullptr, ws, 1, st);
    if (f != SF_OK) return f;
    const T *tq = static_cast<const T*>(q), *tk = static_cast<const T*>(k), *tv = static_cast<const T*>(v), *tdo = static_cast<const T*>(dO);
    const dim3 chunks(p.NC, p.H, p.B), cols(p.dv / DVS, p.H, p.B);
    const size_t s1 = smem_bwd_pre(p.C, p.dk, p.dv), s2 = smem_chain(p.dk), s3 = smem_bwd_out(p.C, p.dk, p.dv);
    if (!opt_in(bwd_pre_kernel<T>, s1) || !opt_in(chain_kernel<64>, s2) || !opt_in(chain_kernel<128>, s2) || !opt_in(bwd_out_kernel<T>, s3))
        return SF_ERR_CUDA;
    bwd_pre_kernel<T><<<chunks, NT, s1, st>>>(p, tq, tk, g, beta, tdo, ws);
    const int ns = delta_state_pass(p, true, dS_out, dS_in, ws, 1, st);
    bwd_out_kernel<T><<<chunks, NT, s3, st>>>(p, tq, tk, tv, g, beta, tdo, static_cast<T*>(dq), static_cast<T*>(dk), static_cast<T*>(dv),
                                              dg, dbeta, ws);
    return launched(2 + ns);
}

// ---- chunkwise diagonal decay ----------------------------------------------------------------------------------------
sf::dcc::Params channel_params(const sf_seg_desc_t* d) {
    const sf::gdn::Params g = chunked_params(d);
    sf::dcc::Params p;
    p.B = g.B; p.H = g.H; p.L = g.L; p.C = g.C; p.NC = g.NC; p.dk = g.dk; p.dv = g.dv;
    p.tqk = g.tqk; p.tv = g.tv; p.tg = g.tg; p.bqk = g.bqk; p.bv = g.bv; p.bg = g.bg;
    return p;
}

size_t channel_chunked_ws_bytes(const sf_seg_desc_t* d, bool backward) {
    return (size_t)d->B * d->H * sf::dcc::ws_floats(channel_params(d), backward) * sizeof(float);
}

template <typename T>
sf_status_t channel_chunked_run(const sf::dcc::Params& p, const void* q, const void* k, const void* v, const float* g,
                                const float* S_in, void* o, float* S_out, const void* dO, const float* dS_out, void* dq, void* dk,
                                void* dv, float* dg, float* dS_in, float* ws, cudaStream_t st) {
    using namespace sf::dcc;
    const bool backward = dO != nullptr;
    const T *tq = static_cast<const T*>(q), *tk = static_cast<const T*>(k), *tv = static_cast<const T*>(v), *tdo = static_cast<const T*>(dO);
    const dim3 chunks(p.NC, p.H, p.B), elems((p.dk * p.dv + NT - 1) / NT, p.H, p.B);
    const size_t s1 = smem_pre(p.C, p.dk, p.dv), s2 = smem_out(p.C, p.dk, p.dv), s3 = smem_bwd_out(p.C, p.dk, p.dv);
    if (!opt_in(pre_kernel<T>, s1) || !opt_in(out_kernel<T>, s2) || !opt_in(bwd_out_kernel<T>, s3)) return SF_ERR_CUDA;
    pre_kernel<T><<<chunks, NT, s1, st>>>(p, tq, tk, tv, g, tdo, ws, backward);
    chain_kernel<<<elems, NT, 0, st>>>(p, 0, S_in, S_out, ws, backward);
    if (!backward) {
        out_kernel<T><<<chunks, NT, s2, st>>>(p, tq, tk, tv, g, static_cast<T*>(o), ws, 0);
        return launched(3);
    }
    chain_kernel<<<elems, NT, 0, st>>>(p, 1, dS_out, dS_in, ws, 1);
    bwd_out_kernel<T><<<chunks, NT, s3, st>>>(p, tq, tk, tv, g, tdo, static_cast<T*>(dq), static_cast<T*>(dk), static_cast<T*>(dv), dg, ws);
    return launched(4);
}

}  // namespace

extern "C" {

size_t sf_recurrent_workspace_bytes(const sf_seg_desc_t* desc) {
    return check_desc(desc) == SF_OK ? ws_bytes(desc) : 0;
}

sf_status_t sf_channel_segment_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, void* o, float* S_out, sf_stream_t stream) {
    return rec_fwd<sf::rec::CHANNEL>(desc, q, k, v, g, nullptr, S_in, o, S_out, reinterpret_cast<cudaStream_t>(stream));
}

sf_status_t sf_channel_segment_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv,
                                   float* dg, float* dS_in, void* workspace, size_t workspace_bytes, sf_stream_t stream) {
    return rec_bwd<sf::rec::CHANNEL>(desc, q, k, v, g, nullptr, S_in, dO, dS_out, dq, dk, dv, dg, nullptr, dS_in, workspace,
                                     workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

sf_status_t sf_delta_segment_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, void* o, float* S_out, sf_stream_t stream) {
    return rec_fwd<sf::rec::DELTA>(desc, q, k, v, g, beta, S_in, o, S_out, reinterpret_cast<cudaStream_t>(stream));
}

sf_status_t sf_delta_segment_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk,
                                 void* dv, float* dg, float* dbeta, float* dS_in, void* workspace, size_t workspace_bytes,
                                 sf_stream_t stream) {
    return rec_bwd<sf::rec::DELTA>(desc, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, workspace,
                                   workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

size_t sf_channel_chunked_workspace_bytes(const sf_seg_desc_t* desc, int backward) {
    return check_chunked(desc, false) == SF_OK ? channel_chunked_ws_bytes(desc, backward != 0) : 0;
}

sf_status_t sf_channel_chunked_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, void* o, float* S_out, void* workspace, size_t workspace_bytes,
                                   sf_stream_t stream) {
    const sf_status_t c = check_chunked(desc, false);
    if (c != SF_OK) return c;
    if (!q || !k || !v || !g || !o || !S_out || S_in == S_out) return SF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < channel_chunked_ws_bytes(desc, false) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return SF_ERR_WORKSPACE;
    const sf::dcc::Params p = channel_params(desc);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    float* ws = static_cast<float*>(workspace);
    return desc->dtype == SF_F32
        ? channel_chunked_run<float>(p, q, k, v, g, S_in, o, S_out, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, ws, st)
        : channel_chunked_run<__nv_bfloat16>(p, q, k, v, g, S_in, o, S_out, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, ws, st);
}

sf_status_t sf_channel_chunked_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv,
                                   float* dg, float* dS_in, void* workspace, size_t workspace_bytes, sf_stream_t stream) {
    const sf_status_t c = check_chunked(desc, false);
    if (c != SF_OK) return c;
    if (!q || !k || !v || !g || !dO || !dq || !dk || !dv || !dg || !dS_in || dS_in == dS_out) return SF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < channel_chunked_ws_bytes(desc, true) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return SF_ERR_WORKSPACE;
    const sf::dcc::Params p = channel_params(desc);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    float* ws = static_cast<float*>(workspace);
    return desc->dtype == SF_F32
        ? channel_chunked_run<float>(p, q, k, v, g, S_in, nullptr, nullptr, dO, dS_out, dq, dk, dv, dg, dS_in, ws, st)
        : channel_chunked_run<__nv_bfloat16>(p, q, k, v, g, S_in, nullptr, nullptr, dO, dS_out, dq, dk, dv, dg, dS_in, ws, st);
}

size_t sf_delta_chunked_workspace_bytes(const sf_seg_desc_t* desc, int backward) {
    return check_chunked(desc, true) == SF_OK ? chunked_ws_bytes(desc, backward != 0) : 0;
}

sf_status_t sf_delta_chunked_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, void* o, float* S_out, void* workspace, size_t workspace_bytes,
                                 sf_stream_t stream) {
    const sf_status_t c = check_chunked(desc, true);
    if (c != SF_OK) return c;
    if (!q || !k || !v || !g || !beta || !o || !S_out || S_in == S_out) return SF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < chunked_ws_bytes(desc, false) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return SF_ERR_WORKSPACE;
    const sf::gdn::Params p = chunked_params(desc);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    float* ws = static_cast<float*>(workspace);
    return desc->dtype == SF_F32 ? chunked_forward<float>(desc, p, q, k, v, g, beta, S_in, o, S_out, ws, 0, st)
                                 : chunked_forward<__nv_bfloat16>(desc, p, q, k, v, g, beta, S_in, o, S_out, ws, 0, st);
}

sf_status_t sf_delta_chunked_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk,
                                 void* dv, float* dg, float* dbeta, float* dS_in, void* workspace, size_t workspace_bytes,
                                 sf_stream_t stream) {
    const sf_status_t c = check_chunked(desc, true);
    if (c != SF_OK) return c;
    if (!q || !k || !v || !g || !beta || !dO || !dq || !dk || !dv || !dg || !dbeta || !dS_in || dS_in == dS_out) return SF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < chunked_ws_bytes(desc, true) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return SF_ERR_WORKSPACE;
    const sf::gdn::Params p = chunked_params(desc);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    float* ws = static_cast<float*>(workspace);
    return desc->dtype == SF_F32
        ? chunked_backward<float>(desc, p, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, ws, st)
        : chunked_backward<__nv_bfloat16>(desc, p, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, ws, st);
}

sf_status_t sf_conv_segment_fwd(int32_t B, int32_t L, int32_t C, int32_t W, const float* x, const float* w, const float* tail_in,
                                float* y, float* tail_out, sf_stream_t stream) {
    const sf_status_t c = check_conv(B, L, C, W);
    if (c != SF_OK) return c;
    if (!x || !w || !y || (W > 1 && !tail_out) || (tail_in && tail_in == tail_out)) return SF_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const bool v4 = conv_vec4(C, {x, w, tail_in, y, tail_out});
    const dim3 grid = conv_grid(B, L, C, v4 ? 4 : 1), block(32, 8);
    conv_width_switch(W, [&](auto wc) {
        constexpr int Wc = decltype(wc)::value;
        if (v4) sf::rec::conv_fwd_kernel<4, Wc><<<grid, block, 0, st>>>(B, L, C, x, w, tail_in, y, tail_out);
        else    sf::rec::conv_fwd_kernel<1, Wc><<<grid, block, 0, st>>>(B, L, C, x, w, tail_in, y, tail_out);
    });
    return launched();
}

sf_status_t sf_conv_segment_bwd(int32_t B, int32_t L, int32_t C, int32_t W, const float* x, const float* w, const float* tail_in,
                                const float* dy, const float* dtail_out, float* dx, float* dw, float* dtail_in,
                                sf_stream_t stream) {
    const sf_status_t c = check_conv(B, L, C, W);
    if (c != SF_OK) return c;
    if (!x || !w || !dy || !dx || !dw || (W > 1 && !dtail_in) || (dtail_out && dtail_out == dtail_in)) return SF_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const long long rows = (long long)L + W - 1;
    const bool v4 = conv_vec4(C, {w, dy, dtail_out, dx, dtail_in});
    const dim3 grid = conv_grid(B, rows, C, v4 ? 4 : 1), block(32, 8);
    conv_width_switch(W, [&](auto wc) {
        constexpr int Wc = decltype(wc)::value;
        if (v4) sf::rec::conv_bwd_input_kernel<4, Wc><<<grid, block, 0, st>>>(B, L, C, w, dy, dtail_out, dx, dtail_in);
        else    sf::rec::conv_bwd_input_kernel<1, Wc><<<grid, block, 0, st>>>(B, L, C, w, dy, dtail_out, dx, dtail_in);
    });
    if (cudaGetLastError() != cudaSuccess) return SF_ERR_CUDA;
    conv_width_switch(W, [&](auto wc) {
        sf::rec::conv_bwd_weight_kernel<decltype(wc)::value><<<dim3((C + sf::rec::CONV_WC - 1) / sf::rec::CONV_WC),
                                                                 dim3(sf::rec::CONV_WC, sf::rec::CONV_WT), 0, st>>>(B, L, C, x, tail_in, dy, dw);
    });
    return launched(2);
}

}  // extern "C"
