/*
 * stateflow.h - C ABI of the B200 (sm_100a) segment kernels for the chunkwise
 * gated linear recurrence
 *
 *     S_t = exp(g_t) * S_{t-1} + k_t^T v_t ,      o_t = q_t S_t
 *
 * (paper Eq. 1 with the scalar-identity transition of Section 2.1), run over one
 * sequence segment with an incoming boundary state S_in and an outgoing S_out
 * (paper Eq. 4-5), and its backward, which takes dO and the downstream
 * boundary-state gradient dS_out and returns dq, dk, dv, dg and dS_in (paper
 * Eq. 6-7).  A "segment" is the paper's sequence chunk C_i, the scheduling unit;
 * a "chunk" is its kernel-level chunk of T_C tokens (Section 3.1, last paragraph).
 *
 * Conventions for every entry point
 *  - All data pointers are DEVICE pointers unless a comment says "host".  The
 *    caller owns every buffer, including the workspace; the library allocates no
 *    device memory (the one exception is documented at its declaration).
 *  - Work is enqueued on the given stream and the call returns without
 *    synchronising.  Outputs are valid once the stream reaches that point; all
 *    buffers must stay alive and unmodified until then.
 *  - Layout (row-major, strides in ELEMENTS of the tensor's type):
 *      q, k, dq, dk : [B, T, H, d_k]       v, o, dO, dv : [B, T, H, d_v]
 *      g, dg        : [B, T, H]  float32   (log-decay, g <= 0 expected, not checked)
 *      states       : [B, H, d_k, d_v] float32, contiguous
 *    A segment is a view: the pointer addresses its first token, consecutive
 *    tokens are tok_stride_* apart, batches batch_stride_* apart, head h starts
 *    h*d (resp. h) elements after the token base.  Passing the strides of the
 *    full sequence lets segments be chained without copies.
 *  - q, k, v, dO and o, dq, dk, dv have type desc->dtype; g, dg and all states
 *    are float32.  Arithmetic accumulates in float32.
 *  - Validation happens on the host before anything is launched.  A call that
 *    returns an error has enqueued nothing.  The library never throws, aborts,
 *    prints or traps the device.
 *  - Pointers must be 16-byte aligned; for SF_BF16 the token and batch strides
 *    must be multiples of 8 elements (16 bytes).
 *  - Devices and threads: the library's own host state (kernel attributes, the
 *    status word's address, the chain driver's side streams and events) is kept
 *    per device and created on first use with that device current, so one process
 *    may drive several devices.  On ONE device, calls that use the chain driver's
 *    side streams (sf_chain_* with overlap != 0, graphs recorded from them, the
 *    tuner) must not run concurrently from several host threads: they share those
 *    streams and events.  Everything else may be called from any thread.
 */
#ifndef STATEFLOW_H
#define STATEFLOW_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque here so that the header needs no CUDA include; pass a cudaStream_t. */
typedef struct CUstream_st* sf_stream_t;

typedef enum {
    SF_OK = 0,
    SF_ERR_INVALID_ARG = 1,   /* NULL where required, bad shape, misalignment, aliasing */
    SF_ERR_UNSUPPORTED = 2,   /* (dtype, d_k, d_v, chunk) outside the supported set */
    SF_ERR_WORKSPACE = 3,     /* workspace NULL or smaller than sf_workspace_bytes() */
    SF_ERR_CUDA = 4,          /* a CUDA runtime/driver call or a launch failed (cudaGetLastError, no sync) */
    SF_ERR_TIMEOUT = 5        /* a bounded device-side wait ran out (see sf_device_status) */
} sf_status_t;

typedef enum { SF_BF16 = 0, SF_F32 = 1 } sf_dtype_t;

/*
 * Shape of one segment.  Supported sets:
 *   SF_F32  : d_k, d_v in {32, 64, 128}, chunk in {16, 32, 64}          (CUDA-core kernels)
 *   SF_BF16 : d_k = d_v = 128, chunk = 64                               (tcgen05 / TMEM / TMA kernels)
 *             d_k, d_v in {32, 64}, chunk in {16, 32, 64}               (CUDA-core kernels)
 * seg_len is any positive number of tokens.  The paper rounds boundaries to multiples of 128 (Section 3.2), so
 * its workloads never leave a partial chunk; when seg_len is not a multiple of chunk the last chunk simply has
 * fewer tokens (its missing rows count as zero keys, values and gradients with log-decay 0, and are never
 * written).  chunks_per_block sets how many chunks form one block, the only granularity
 * whose states are written to the workspace (at most 64); 0 lets the library
 * pick the length in [4, 32] that fills the device's SMs best for this shape.  Heads are independent.
 */
typedef struct {
    int32_t B, H, d_k, d_v;
    int32_t seg_len, chunk;
    int32_t dtype;                 /* sf_dtype_t */
    int32_t chunks_per_block;      /* 0 = default */
    int64_t tok_stride_qk, tok_stride_v, tok_stride_g;
    int64_t batch_stride_qk, batch_stride_v, batch_stride_g;
} sf_seg_desc_t;

const char* sf_status_string(sf_status_t s);

/* Number of blocks of the segment: ceil(ceil(seg_len / chunk) / chunks_per_block), with the library's own choice
   of chunks_per_block when the descriptor leaves it 0.  0 on an invalid descriptor. */
int32_t sf_num_blocks(const sf_seg_desc_t* desc);

/*
 * Bytes of workspace a call needs (host function; 0 on an invalid descriptor).
 *   backward == 0 : sf_segment_fwd
 *   backward == 1 : sf_segment_bwd given the forward's workspace as fwd_saved
 *   backward == 2 : sf_segment_bwd with fwd_saved == NULL (block states are replayed)
 * The workspace must be 256-byte aligned.
 */
size_t sf_workspace_bytes(const sf_seg_desc_t* desc, int backward);

/*
 * Forward of one segment, (C_out, S_out) = Fwd(C_in, S_in) (paper Eq. 4) with C_in = (q, k, v, g),
 * C_out = o.  Internally the three stages of paper Eq. 2: block aggregates (Pre), state scan over
 * blocks (ST), chunk outputs (Out).
 *   S_in  : nullable, NULL means the zero state (the paper's S_0 = 0)
 *   S_out : required, must not alias S_in
 *   workspace : sf_workspace_bytes(desc, 0) bytes; after the call it holds the block-entering
 *               states, which sf_segment_bwd can reuse (fwd_saved) as long as it is left unchanged
 */
sf_status_t sf_segment_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v,
                           const float* g, const float* S_in, void* o, float* S_out,
                           void* workspace, size_t workspace_bytes, sf_stream_t stream);

/*
 * Backward of one segment, (dC_in, dS_in) = Bwd(C_in, S_in, dC_out, dS_out) (paper Eq. 6) with
 * dC_out = dO and dC_in = (dq, dk, dv, dg).  Stages: state replay (SR, skipped when fwd_saved is
 * given), backward block aggregates and reverse state scan (STB), output gradient (OG -> dq),
 * preparation gradient (PG -> dk, dv), and the log-decay gradient dg assembled from both
 * (Section 3.4, backward pass).
 *   S_in      : the state the forward of this segment started from (nullable = zero)
 *   dS_out    : nullable, NULL means zero
 *   dS_in     : required, must not alias dS_out
 *   fwd_saved : nullable; the workspace sf_segment_fwd filled for this same segment and descriptor
 *   workspace : sf_workspace_bytes(desc, fwd_saved ? 1 : 2) bytes, distinct from fwd_saved
 */
sf_status_t sf_segment_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v,
                           const float* g, const float* S_in, const void* dO, const float* dS_out,
                           void* dq, void* dk, void* dv, float* dg, float* dS_in,
                           const void* fwd_saved, void* workspace, size_t workspace_bytes,
                           sf_stream_t stream);

/*
 * sf_segment_fwd for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * Some callers have no way to hand over a workspace: code running inside a CUDA-graph capture or
 * under a memory pool that forbids new allocations, plug-ins that receive only their input and
 * output pointers from a host framework, and real-time loops that must not touch the allocator.
 * For them the block aggregates and block-entering states live in a scratch array that is part of
 * the library image itself (SF_STATIC_SCRATCH_BYTES bytes, held by every GPU that loads the library
 * until the process exits).  The call allocates nothing: no cudaMalloc, no cudaFree, no allocating
 * library routine.  Inputs and outputs are still the caller's, exactly as for sf_segment_fwd.
 *
 *  - Limit: sf_workspace_bytes(desc, 0) must not exceed SF_STATIC_SCRATCH_BYTES, i.e. roughly
 *    B * H * sf_num_blocks(desc) <= 255 for d_k = d_v = 128; larger shapes get SF_ERR_WORKSPACE and
 *    nothing is launched.
 *  - The first call on each device looks up the device address of the scratch array (once per
 *    device, with that device current).  Make that first call before any stream capture begins.
 *  - All calls share the one array and it keeps whatever the previous call left in it.  The forward
 *    pass overwrites every scratch element it later reads, so nothing has to be cleared; but two
 *    calls whose kernels overlap on the GPU (different streams, no ordering between them) race on
 *    it.  Order such calls yourself.
 *  - The scratch content cannot be passed to sf_segment_bwd as fwd_saved once another call has run;
 *    use fwd_saved == NULL (state replay) for the backward of such a segment.
 */
#define SF_STATIC_SCRATCH_BYTES (16u << 20)
sf_status_t sf_segment_fwd_static(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v,
                                  const float* g, const float* S_in, void* o, float* S_out,
                                  sf_stream_t stream);

/*
 * The ST stage alone (paper Eq. 2, second line; Eq. 5 / Eq. 7 across boundaries): the first-order
 * linear recurrence over the n = sf_num_blocks(desc) blocks of a segment, element-wise over
 * B*H*d_k*d_v lanes.  B, H, d_k, d_v, seg_len, chunk come from desc; chunks_per_block overrides
 * desc->chunks_per_block when > 0.
 *   forward (reverse == 0): X_0 = S_boundary_in; states[j] = X_j (state ENTERING block j);
 *                           X_{j+1} = exp(log_decay[j]) X_j + U[j];  S_boundary_out = X_n
 *   reverse (reverse != 0): X_n = S_boundary_in; states[j] = X_{j+1} (gradient LEAVING block j);
 *                           X_j = exp(log_decay[j]) X_{j+1} + U[j];  S_boundary_out = X_0
 *   log_decay [B,H,n] float32 block totals of g;  U, states [B,H,n,d_k,d_v] float32 (states may
 *   alias U);  S_boundary_in nullable = zero;  S_boundary_out required, must not alias the input.
 */
sf_status_t sf_state_scan(const sf_seg_desc_t* desc, int32_t chunks_per_block, int32_t reverse,
                          const float* log_decay, const float* U, const float* S_boundary_in,
                          float* states, float* S_boundary_out, sf_stream_t stream);

/*
 * Segment-chaining driver (paper Eq. 5 and Eq. 7; the single-device part of the partial order of
 * Eq. 8: F_{i-1} before F_i, F_i before B_i, B_{i+1} before B_i).  seg_lens is a HOST array of
 * n_seg segment lengths (each positive; desc->seg_len is ignored);
 * q, k, v, g, o, ... address token 0 of the whole sequence of T = sum(seg_lens) tokens.
 *
 * sf_chain_fwd runs Fwd on segments 0..n_seg-1 with S_{i+1}^in = S_i^out.
 *   S_init   : nullable = zero; may be S_bounds itself (the initial state is then taken as already in S_bounds[0])
 *   S_bounds : [n_seg+1][B,H,d_k,d_v] float32; on return S_bounds[i] = S_i^in and
 *              S_bounds[n_seg] = the final state.  Kept by the caller for sf_chain_bwd.
 *   workspace: sf_chain_workspace_bytes(..., 0) bytes; holds every segment's saved block states.
 * sf_chain_bwd runs Bwd on segments n_seg-1..0 with dS_i^out = dS_{i+1}^in.
 *   dS_final : nullable = zero;   dS_init : required, receives dS_0^in
 *   fwd_workspace : the workspace sf_chain_fwd filled, or NULL to replay block states
 *   workspace: sf_chain_workspace_bytes(..., fwd_workspace ? 1 : 2) bytes
 * overlap != 0 lets the driver run state-independent stages on internal side streams concurrently
 * with the state scans (the split-and-overlap idea of Section 3.4, Eq. 17-18).  Only the scans carry
 * the state from segment to segment, so they alone chain on `stream`: forward, the block aggregates
 * run ahead on side streams and each segment's sweep starts on another as soon as its own scan is
 * done; backward (with fwd_workspace given), all aggregates run ahead, and each segment's dq sweep and
 * dk/dv sweep (+ dg) start on further streams after its own reverse scan.  Aggregates and sweeps of
 * consecutive short segments go to different streams (round-robin), so they share the device, and
 * up to 8 neighbouring segments of at most 4096 tokens in total are scanned by one kernel that carries
 * the state from one to the next in registers.
 * The result is bit-identical to overlap == 0.  The side streams are joined back
 * into `stream` before the call returns, so later work on `stream` sees all outputs.
 */
size_t sf_chain_workspace_bytes(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                                int backward);

sf_status_t sf_chain_fwd(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                         const void* q, const void* k, const void* v, const float* g,
                         const float* S_init, void* o, float* S_bounds,
                         void* workspace, size_t workspace_bytes, int32_t overlap, sf_stream_t stream);

sf_status_t sf_chain_bwd(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                         const void* q, const void* k, const void* v, const float* g,
                         const float* S_bounds, const void* dO, const float* dS_final,
                         void* dq, void* dk, void* dv, float* dg, float* dS_init,
                         const void* fwd_workspace, void* workspace, size_t workspace_bytes,
                         int32_t overlap, sf_stream_t stream);

/*
 * The same chain as one CUDA graph.  The paper's timings include inter-chunk state propagation and
 * kernel-launch overhead (Section 4.4); with short segments the chain is a long list of small kernels
 * and the host cannot launch them as fast as the device finishes them.  sf_chain_graph_create runs
 * sf_chain_fwd (and, if dO is not NULL, sf_chain_bwd with the forward workspace) once on `stream` as
 * it stands, then records the same calls, side streams included, into a graph; sf_chain_graph_launch
 * replays it.  Arguments are those of sf_chain_fwd / sf_chain_bwd; every pointer is baked into the
 * graph, so the buffers must stay alive, at the same addresses, until sf_chain_graph_destroy.
 *   stream : a stream that can be captured (not the legacy default stream, SF_ERR_INVALID_ARG)
 *   *out   : receives the handle (host object owned by the library); NULL on error
 * Results are bit-identical to the direct calls.  Errors: those of the direct calls, SF_ERR_UNSUPPORTED
 * while stage timing is enabled, SF_ERR_CUDA if capture or instantiation fails.
 * sf_chain_graph_kernels: kernels (of this library) per replay.  The paper has no counterpart.
 */
typedef struct sf_chain_graph sf_chain_graph_t;

sf_status_t sf_chain_graph_create(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                                  const void* q, const void* k, const void* v, const float* g,
                                  const float* S_init, void* o, float* S_bounds,
                                  void* fwd_workspace, size_t fwd_workspace_bytes,
                                  const void* dO, const float* dS_final,
                                  void* dq, void* dk, void* dv, float* dg, float* dS_init,
                                  void* bwd_workspace, size_t bwd_workspace_bytes,
                                  int32_t overlap, sf_stream_t stream, sf_chain_graph_t** out);
sf_status_t sf_chain_graph_launch(sf_chain_graph_t* graph, sf_stream_t stream);
int64_t sf_chain_graph_kernels(const sf_chain_graph_t* graph);
void sf_chain_graph_destroy(sf_chain_graph_t* graph);

/*
 * Schedule of the chaining driver (the paper picks "tile sizes, split points and overlap schedules" per operator
 * shape by profiling a small set of valid choices, Section 3.4 last paragraph and Section 4.4 / Table 3).  Process-wide;
 * read at every sf_chain_* call (and so frozen into a graph when it is recorded).  Results do not depend on it
 * (merge_launches: up to rounding, see there).
 *   sweep_streams     1..4  side streams the sweeps of consecutive segments rotate over (per kind of sweep)
 *   agg_streams       1..4  side streams the block-aggregate kernels of small segments rotate over
 *   scan_group_tokens >= 0  neighbouring segments of at most this many tokens in total share one scan launch
 *   agg_inorder_ctas  >= 1  an aggregate launch of at least this many CTAs stays in order on the first aggregate stream
 *   agg_ahead         >= 0  how many segments the aggregate kernels may run ahead of the sweeps (0 = no limit);
 *                           a small value keeps what the aggregates read close to the sweeps that read it again
 *   merge_launches    0 / 1 1: the chain runs as ONE segment spanning the sequence, every stage once (one aggregate launch,
 *                           one scan, one sweep, ...) instead of once per segment.  Tensor-core path: whenever all segments
 *                           but the last are whole chunks; the blocks then ignore the segment boundaries (block length =
 *                           chunks_per_block, else the library's choice for the whole sequence) and the forward sweep
 *                           itself writes the state entering each segment to S_bounds.  CUDA-core path: when every segment
 *                           but the last is a whole number of blocks of one common length.  Other chains run segment by
 *                           segment as with 0.  Same kernels; where the blocks coincide with the segments' own the
 *                           results are bit-identical, else equal to rounding.  The forward workspace is laid out
 *                           differently, so a backward that reuses it must run under the same value as its forward.
 * The block length is part of the descriptor (chunks_per_block); forward and backward share it because the backward
 * starts its blocks from the block states the forward saved.
 * sf_set_tuning(NULL) restores the defaults {4, 4, 4096, 74, 0, 0}; out-of-range values give SF_ERR_INVALID_ARG and change
 * nothing.  Host functions.
 */
typedef struct {
    int32_t sweep_streams;
    int32_t agg_streams;
    int32_t scan_group_tokens;
    int32_t agg_inorder_ctas;
    int32_t agg_ahead;
    int32_t merge_launches;
} sf_tuning_t;
sf_status_t sf_set_tuning(const sf_tuning_t* tuning);
void sf_get_tuning(sf_tuning_t* tuning);

/*
 * Profile-guided choice of the block length (the paper tunes its kernels' tile sizes and overlap schedules
 * "for each operator shape" by profiling, Section 3.4 end and Section 4.4; here the one tunable of that kind is
 * chunks_per_block).  Runs the chain (sf_chain_fwd, and sf_chain_bwd with the forward workspace if dO is not
 * NULL) once untimed and `reps` times timed (CUDA events on `stream`) for every candidate value and reports
 * the fastest.  On a stream that can be captured each candidate is timed as replays of its CUDA graph
 * (sf_chain_graph_create; free of the host's launch cost, which hides the differences between candidates when
 * segments are short); on the legacy default stream it is launched directly.  Arguments are those of sf_chain_graph_create, plus
 *   candidates : HOST array of n_cand values for desc->chunks_per_block (0 = the library's own model)
 *   best       : receives the fastest candidate (write it into desc->chunks_per_block for later calls)
 *   ms         : nullable HOST array of n_cand mean times in milliseconds; -1 for a candidate that was skipped
 *                because the given workspaces are too small for it (size them for the smallest nonzero
 *                candidate, which has the most blocks) or that the descriptor rejects
 * The outputs hold the result of the last run.  The call synchronises `stream`.  Errors: those of the chain
 * calls for argument problems common to all candidates; SF_ERR_WORKSPACE if no candidate fits.
 */
sf_status_t sf_chain_autotune(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                              const void* q, const void* k, const void* v, const float* g,
                              const float* S_init, void* o, float* S_bounds,
                              void* fwd_workspace, size_t fwd_workspace_bytes,
                              const void* dO, const float* dS_final,
                              void* dq, void* dk, void* dv, float* dg, float* dS_init,
                              void* bwd_workspace, size_t bwd_workspace_bytes,
                              const int32_t* candidates, int32_t n_cand, int32_t reps, int32_t overlap,
                              sf_stream_t stream, int32_t* best, float* ms);

/*
 * Profile-guided choice of the driver's schedule (Section 3.4 last paragraph, Section 4.4 / Table 3: the paper's overlap
 * schedules are picked per shape from measurements).  Times the chain (as sf_chain_autotune does, with the descriptor's
 * block length) under a small built-in set of valid sf_tuning_t values - how far the aggregates may run ahead (0, 1,
 * 2 segments), 2 or 4 sweep streams, aggregates in order or spread over their streams - and installs the fastest with
 * sf_set_tuning, except that the default stays unless it is beaten by more than `margin` (e.g. 0.02) over `reps`
 * repetitions.  chosen / chosen_ms / default_ms (the last two nullable, HOST) report the outcome.  Needs the same
 * buffers as sf_chain_graph_create; synchronises `stream`.
 */
sf_status_t sf_chain_autotune_schedule(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                                       const void* q, const void* k, const void* v, const float* g, const float* S_init,
                                       void* o, float* S_bounds, void* fwd_workspace, size_t fwd_workspace_bytes,
                                       const void* dO, const float* dS_final, void* dq, void* dk, void* dv, float* dg,
                                       float* dS_init, void* bwd_workspace, size_t bwd_workspace_bytes, int32_t reps,
                                       float margin, sf_stream_t stream, sf_tuning_t* chosen, float* chosen_ms,
                                       float* default_ms);

/*
 * Hybrid-aware sequence chunking (paper Section 3.2, Eq. 9-11): the segment lengths to hand to the chain
 * driver.  Host code only; no CUDA call.  With boundaries 0 = c_0 < ... < c_N = T and s_i = c_{i+1} - c_i,
 *     Cost_i = w_tok * s_i + w_soft * (c_i * s_i + s_i^2 / 2)                                       (Eq. 9)
 * (w_tok = L_lin*C_lin + C_dense: token-wise work; w_soft = L_soft*C_soft: work per query-key pair of the
 * softmax layers).  The FLOP-balanced boundaries c_i^hybrid make all Cost_i equal (Eq. 10); the candidate is
 *     c_i(alpha) = (1 - alpha) * i*T/N + alpha * c_i^hybrid                                          (Eq. 11)
 * rounded to the closest multiple of `multiple` (the paper uses 128; a tie goes up; c_N stays T).  After
 * rounding, boundaries are pushed apart (forward, then backward) so that every segment keeps at least one
 * multiple.  alpha = 0 or w_soft = 0 give equal lengths; alpha > 1 exaggerates the imbalance.
 *   seg_lens : HOST array of N entries, written on success
 * Errors (SF_ERR_INVALID_ARG): T < 1, N < 1, multiple < 1, negative or both-zero weights, non-finite alpha,
 * seg_lens NULL, or T too short for N segments of one multiple each.
 */
sf_status_t sf_partition_hybrid(int64_t T, int32_t N, double w_tok, double w_soft, double alpha,
                                int32_t multiple, int32_t* seg_lens);

/*
 * Host-memory convenience wrappers around the chain driver (the "end-to-end" path): every data
 * pointer is a HOST pointer (pinned memory recommended).  The call copies the inputs to the device
 * buffers in `dev` (caller-allocated device scratch, sf_e2e_device_bytes() bytes, 256-byte
 * aligned), runs sf_chain_fwd + sf_chain_bwd and copies o, dq, dk, dv, dg, the final state and
 * dS_init back, then synchronises `stream`; everything is ordered after earlier work on `stream` and is complete
 * when the call returns.  The chain is pipelined segment by segment against the copies on two copy streams of the
 * library: inputs are uploaded in segment order (dO afterwards, last segment first), a segment's forward runs as soon
 * as its inputs are there and its o goes back while later inputs still arrive; a segment's backward runs as soon as
 * its dO is there and its gradients go back while earlier segments' dO still arrive.  Both PCIe directions are busy
 * for most of the call (needs pinned host memory to take effect).  Each segment runs as a one-segment chain, in
 * order, on `stream`.  Uses the chain driver's per-device streams: the threading rule of
 * sf_chain_* with overlap != 0 applies.  Section 3.1, Eq. 4-7.
 */
size_t sf_e2e_device_bytes(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg);

sf_status_t sf_chain_fwd_bwd_host(const sf_seg_desc_t* desc, const int32_t* seg_lens, int32_t n_seg,
                                  const void* q, const void* k, const void* v, const float* g,
                                  const float* S_init, const void* dO, const float* dS_final,
                                  void* o, float* S_final, void* dq, void* dk, void* dv, float* dg,
                                  float* dS_init, void* dev, size_t dev_bytes, sf_stream_t stream);

/*
 * Device-side status word of the kernels launched by this library on the current device (host
 * function; it copies one word from the device, which waits for prior work).  0 means no bounded
 * wait has run out since sf_device_status_clear().  Kernels never spin without a limit; when a
 * limit is hit they record a code here, stop waiting and return normally, leaving their outputs
 * undefined.  No counterpart in the paper.
 *
 * Codes: 0 none; 1 a wait for tile data (TMA) ran out; 2 a wait for a tensor-core result or for another warp's
 * hand-off ran out; 3 the wait of sf_selftest_bounded_wait ran out (as it must); -1 the word could not be read.
 * sf_device_check() maps the word to a status: SF_OK, SF_ERR_TIMEOUT (any code > 0) or SF_ERR_CUDA.
 */
int32_t sf_device_status(void);
void sf_device_status_clear(void);
sf_status_t sf_device_check(void);

/*
 * Exercises the bounded wait without touching any product kernel: a one-warp kernel waits on a barrier that nothing
 * ever completes, gives up after `limit_cycles` clock cycles (1 .. 1e8: at most a few hundredths of a second),
 * records code 3 in the status word and returns normally; the call waits for it and returns what sf_device_check()
 * then says, i.e. SF_ERR_TIMEOUT when the mechanism works.  The context stays usable; call sf_device_status_clear()
 * afterwards.  No counterpart in the paper.
 */
sf_status_t sf_selftest_bounded_wait(int64_t limit_cycles, sf_stream_t stream);

/* Number of kernels this library has launched in this process (host counter). No paper counterpart. */
int64_t sf_launch_count(void);

/*
 * Per-stage device timers for profiling (host functions; no paper counterpart, the stages themselves
 * are those of Eq. 2 and Section 3.4).  While enabled, every kernel launch is bracketed by two CUDA
 * events on its own stream, which costs a little throughput, so leave it off when timing whole steps.
 * sf_stage_timing_read synchronises the device, adds up the elapsed time and launch count of each
 * stage since the last read into ms[0..n) / launches[0..n), forgets them and returns the number of
 * stages: 0 block aggregate of (k, v), 1 block aggregate of (q, dO), 2 state scan, 3 forward output
 * pass, 4 dq pass, 5 dk/dv pass, 6 log-decay gradient.
 */
void sf_stage_timing(int32_t enable);
int32_t sf_stage_timing_read(float* ms, int64_t* launches, int32_t n);

/*
 * ---- Extensions of the segment operator to further transition families --------------------------------------------
 * Paper Section 2.1 lets the transition F_t be diagonal or scalar-plus-low-rank besides the scalar decay that the
 * entry points above implement; Section 3.1 (footnote on auxiliary boundary states) lets a short-convolution state
 * travel with S across the segment boundary.  The calls below are those three operators with the same segment
 * semantics (Eq. 4-7): a forward maps the incoming boundary state to the outgoing one, a backward maps the gradient
 * of the outgoing boundary state to that of the incoming one, so segments chain exactly as with sf_segment_*.
 * They are CUDA-core kernels that walk the tokens in order (one CTA per batch x head) with float32 arithmetic:
 * deterministic, and not tuned.  All pointers are DEVICE pointers; q, k, v, dO and o, dq, dk, dv have the descriptor's
 * dtype (float32 or bf16; bf16 only rounds what is stored), log-decays, beta, their gradients and the states are
 * float32.  Nothing is allocated and the calls do not synchronise.
 *
 * Descriptor: d_k in {32, 64}, d_v in {32, 64, 128}; chunk and chunks_per_block are ignored.
 * q, k (and the per-channel g / dg of the diagonal family) use tok_stride_qk / batch_stride_qk, v, o, dO, dv use the
 * _v strides, the per-head scalars g, beta, dg, dbeta of the delta rule use the _g strides; element (b, t, h, i) sits
 * at b*batch_stride + t*tok_stride + h*d + i.  States are [B, H, d_k, d_v] dense.
 * Errors as above: SF_ERR_INVALID_ARG (NULL where required, bad shape, an input state aliasing an output state),
 * SF_ERR_UNSUPPORTED (shape or dtype outside the set), SF_ERR_WORKSPACE, SF_ERR_CUDA.
 */

/* Workspace of the two backward calls: one state per 16 tokens plus 16 states, per batch x head (0 on a bad descriptor).
   256-byte aligned. */
size_t sf_recurrent_workspace_bytes(const sf_seg_desc_t* desc);

/*
 * Diagonal transition (Section 2.1): one log-decay per key channel, g [B, T, H, d_k] laid out like q.
 *   S_t = diag(exp(g_t)) S_{t-1} + k_t^T v_t ,  o_t = q_t S_t
 * S_in nullable (zero state); S_out required.  Backward: dS_out nullable (zero), dg has the layout of g.
 */
sf_status_t sf_channel_segment_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, void* o, float* S_out, sf_stream_t stream);
sf_status_t sf_channel_segment_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv,
                                   float* dg, float* dS_in, void* workspace, size_t workspace_bytes, sf_stream_t stream);

/*
 * Gated delta rule (scalar decay plus a rank-one correction; Section 2.1, Eq. 2 with a non-empty V_new), with
 * a_t = exp(g_t), g and beta [B, T, H] laid out like the g of sf_segment_fwd:
 *   u_t = k_t S_{t-1} ;  w_t = beta_t (v_t - a_t u_t) ;  S_t = a_t S_{t-1} + k_t^T w_t ;  o_t = q_t S_t
 * i.e. S_t = a_t (I - beta_t k_t^T k_t) S_{t-1} + beta_t k_t^T v_t.  Keys are used as given (normalise them upstream).
 */
sf_status_t sf_delta_segment_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, void* o, float* S_out, sf_stream_t stream);
sf_status_t sf_delta_segment_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk,
                                 void* dv, float* dg, float* dbeta, float* dS_in, void* workspace, size_t workspace_bytes,
                                 sf_stream_t stream);

/*
 * The diagonal-decay operator in its chunkwise form (Section 2.2, Eq. 2 with an empty V_new): per chunk the decay-weighted
 * scores A[t,s] = sum_i q_t[i] k_s[i] exp(b_t[i] - b_s[i]) and the affine state map H' = diag(gam_n) H + (om*K)^T V are
 * built for all chunks in parallel, the state is carried from chunk to chunk element by element, and the outputs (and,
 * in the backward, every gradient, with dg anchored per chunk) are again formed for all chunks in parallel.  Same
 * arguments, layouts and results (to rounding) as sf_channel_segment_fwd/bwd.  desc->chunk in {16, 32}, d_k, d_v in
 * {32, 64, 128} as far as the kernels' tiles fit into shared memory (128-wide heads need chunk 16; otherwise
 * SF_ERR_UNSUPPORTED), float32 or bf16 storage, float32 arithmetic on CUDA cores.  Workspace:
 * sf_channel_chunked_workspace_bytes(desc, backward) bytes, 256-byte aligned.
 */
size_t sf_channel_chunked_workspace_bytes(const sf_seg_desc_t* desc, int backward);
sf_status_t sf_channel_chunked_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, void* o, float* S_out, void* workspace, size_t workspace_bytes,
                                   sf_stream_t stream);
sf_status_t sf_channel_chunked_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                   const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk, void* dv,
                                   float* dg, float* dS_in, void* workspace, size_t workspace_bytes, sf_stream_t stream);

/*
 * The same gated delta rule in its chunkwise form (Section 2.2, Eq. 2 with V_new): per chunk the unit-lower-triangular
 * system (I + L) W = beta*V - beta*gam*(K H) is solved by substitution (UT transform), Pre builds its state-free parts for
 * all chunks in parallel (including each chunk's affine state map), ST carries the state from chunk to chunk, Out forms
 * V_new = W and the outputs of all chunks in parallel; the backward mirrors it (transposed solve, reverse state pass, chunk-parallel gradients).
 * Same arguments, layouts and results (to rounding) as sf_delta_segment_fwd/bwd.  desc->chunk in {16, 32},
 * d_k, d_v in {32, 64, 128} as far as the kernels' tiles fit into shared memory (128-wide heads need chunk 16; otherwise
 * SF_ERR_UNSUPPORTED), float32 or bf16 storage, float32 arithmetic on CUDA cores.  Workspace:
 * sf_delta_chunked_workspace_bytes(desc, backward) bytes, 256-byte aligned (U and Wk per token, the chunk's state map
 * and one state per chunk; the backward rebuilds them and adds Z0 per token, Theta, one state gradient and two
 * chunk x chunk matrices per chunk).
 */
size_t sf_delta_chunked_workspace_bytes(const sf_seg_desc_t* desc, int backward);
sf_status_t sf_delta_chunked_fwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, void* o, float* S_out, void* workspace, size_t workspace_bytes,
                                 sf_stream_t stream);
sf_status_t sf_delta_chunked_bwd(const sf_seg_desc_t* desc, const void* q, const void* k, const void* v, const float* g,
                                 const float* beta, const float* S_in, const void* dO, const float* dS_out, void* dq, void* dk,
                                 void* dv, float* dg, float* dbeta, float* dS_in, void* workspace, size_t workspace_bytes,
                                 sf_stream_t stream);

/*
 * Causal depthwise convolution of width W (1..8) over the tokens of a segment, dense float32:
 *   x, y [B, L, C] ; w [W, C], w[j] multiplies the input j tokens back ; tails [B, W-1, C]
 *   ext = [tail_in ; x] ,  y_t = sum_j w[j] * ext[W-1+t-j] ,  tail_out = the last W-1 rows of ext
 * tail_in NULL means zeros (start of the sequence); tail_out is the boundary state handed to the next segment and
 * is required when W > 1 (L may be shorter than W-1: old tail rows then move up).  Backward: dtail_out nullable;
 * dw is overwritten with this segment's contribution (the caller adds the segments' dw), summed in a fixed order in
 * double precision.  Channels are processed four at a time with 16-byte accesses when C is a multiple of 4 and every
 * pointer is 16-byte aligned, one at a time otherwise (same results).  Errors: non-positive B, L, C or W < 1 or a missing
 * required pointer SF_ERR_INVALID_ARG; W > 8 or B > 65535 SF_ERR_UNSUPPORTED; nothing is launched then.
 */
sf_status_t sf_conv_segment_fwd(int32_t B, int32_t L, int32_t C, int32_t W, const float* x, const float* w, const float* tail_in,
                                float* y, float* tail_out, sf_stream_t stream);
sf_status_t sf_conv_segment_bwd(int32_t B, int32_t L, int32_t C, int32_t W, const float* x, const float* w, const float* tail_in,
                                const float* dy, const float* dtail_out, float* dx, float* dw, float* dtail_in,
                                sf_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* STATEFLOW_H */
