/*
 * kata.h -- C ABI of the KATA forward pass for NVIDIA B200 (sm_100a).
 *
 * KATA is causal linear attention whose feature map is the rank-one PSD lift of the
 * l2-normalised query/key, psi(u) = u_hat u_hat^T, so that the attention weight is
 * <psi(q_t), psi(k_i)> = (q_hat_t . k_hat_i)^2, with the normalised readout
 *
 *     o_t = sum_{i<=t} w_ti v_i / sum_{i<=t} w_ti            (paper Eq. (2), "linearized form")
 *
 * whose denominator acts as the parameter-free convex output gate of Proposition 1
 * ("Output-level gating").  o_t = 0 where the denominator is 0.  There is no temperature,
 * no epsilon in the normalisation (a zero row has a zero feature) and the causal mask
 * includes the diagonal.
 *
 * Problem statement (Algorithm 1, Require/Return): per head Q,K in R^{T x d_k},
 * V in R^{T x d_v}, chunk size C; returns O in R^{T x d_v}.  Batch and heads are independent.
 *
 * Conventions common to every entry point
 *   - q, k: [B,H,T,d_k]; v, out: [B,H,T,d_v]; row-major, contiguous, 16-byte aligned,
 *     DEVICE pointers (except in kata_fwd_host), element type opts->dtype (fp32 or bf16).
 *   - All accumulation, the running state (S,Z) and the normaliser are fp32; out is rounded
 *     to the element type (round-to-nearest-even).  On the bf16 tensor-core kernels the OPERANDS of the matrix
 *     products are bf16: the chunked forms read the running state through a bf16 copy taken once per tile of 128
 *     tokens (S and Z are accumulated in fp32, but psi(q)^T S and psi(q)^T Z see them rounded), the intra-tile
 *     weights (q.k)^2 are rounded to bf16 before they multiply the values, and the key scale 1/||k||^2 is rounded to
 *     bf16 (the chunked forms multiply it into the values, v/||k||^2 rounded again; the quadratic form into the
 *     weights, rounded again, whose row sum is then the normaliser).  The convex weights of the output gate therefore sum to 1 only to
 *     about 2^-8, and a normaliser that is tiny against its terms (a query nearly orthogonal to every key before it)
 *     can come out <= 0 from the rounded operands, in which case out = 0 as for an exact zero.  All of it stays
 *     inside the 2e-2 tolerance of the bf16 tests.
 *   - The caller owns every buffer.  The library allocates no device or host memory, frees nothing and never
 *     synchronises; all work is enqueued on opts->stream.  q,k,v are read-only; out and the
 *     workspace are fully overwritten (no pre-zeroing needed).  A call on device pointers may therefore be
 *     captured into a CUDA graph and replayed (same pointers, same workspace).  One exception to "allocates nothing":
 *     kata_fwd_host on its piecewise route creates, once per device and for the life of the process, two CUDA
 *     streams and seven events, and takes a process-wide mutex for the duration of the call (see there).
 *   - Supported shapes: d_k, d_v in {16,32,64}; C = 64 (the chunked/scan forms), and C = 128 for
 *     feature_order 1 with bf16, d_k = d_v = 64 (the chunk size of the paper's scan benchmark; tensor-core
 *     path, no s_pre/z_pre); T >= 1 (any; the last chunk is zero-padded as in Algorithm 1 and truncated on
 *     output); B,H >= 1.  A kernel takes at most 65535 heads (B * H) at a time: kata_fwd_quadratic,
 *     kata_fwd_chunked and kata_chunk_state_scan run more heads than that in slabs of 65535, one after the
 *     other on the stream and in the same workspace (kata_workspace_bytes gives the largest slab's need), as
 *     long as no state pointer is set; the other entry points, and these with state pointers, return
 *     KATA_ERR_UNSUPPORTED_SHAPE beyond 65535 heads.  The tensor-core (tcgen05) kernels cover bf16 with d_k = d_v = 64; narrower bf16
 *     rows are zero-padded to 64 entries in the workspace and run on the same kernels (the result is the same
 *     function: dot products and norms do not change) unless feature_groups > 1 or a state is handed over, whose
 *     layouts depend on the true width; everything else runs on the fp32 SIMT kernels.
 *   - Return value: KATA_OK (0) or a negative kata_status.  Errors detectable on the host
 *     launch nothing.  No exceptions, no abort, no device trap.  A bounded device-side wait
 *     that expires writes KATA_ERR_DEVICE_TIMEOUT to *opts->device_status (if non-null),
 *     visible after the caller synchronises the stream; the kernel still terminates.  How long a launch
 *     that has stalled takes to end: the waits of its warps run out side by side and a warp enters no further
 *     wait once one has failed, so it is one limit, not their sum -- 0.1 s on the streaming, quadratic, backward
 *     and first-order kernels (a limit on time), and on the feature-split chunked kernel 4 M polls of at most 1 us
 *     each (between 0.1 s and 4 s) plus at most 2 s for a CTA that waits for the other CTAs of its head.
 */
#ifndef KATA_H_
#define KATA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KATA_VERSION 100

typedef enum kata_status {
  KATA_OK = 0,
  KATA_ERR_INVALID_ARG = -1,        /* null pointer, non-positive size, bad enum, bad struct_size */
  KATA_ERR_UNSUPPORTED_SHAPE = -2,  /* d_k/d_v/C outside the supported set                        */
  KATA_ERR_ALIGNMENT = -3,          /* a tensor or workspace pointer is not 16-byte aligned        */
  KATA_ERR_WORKSPACE_TOO_SMALL = -4,
  KATA_ERR_ARCH = -5,               /* current device is not compute capability 10.x              */
  KATA_ERR_CUDA = -6,               /* a CUDA runtime call or a launch failed                      */
  KATA_ERR_DEVICE_TIMEOUT = -7      /* only ever written to *device_status                         */
} kata_status;

enum { KATA_F32 = 0, KATA_BF16 = 1 };                 /* kata_opts.dtype          */
enum { KATA_LAYOUT_DIRECT = 0, KATA_LAYOUT_PACKED = 1 }; /* kata_opts.state_layout */
enum { KATA_SEQUENTIAL = 0, KATA_SCAN = 1, KATA_INTER_AUTO = 2 };   /* kata_opts.inter_chunk */
enum { KATA_IMPL_AUTO = 0, KATA_IMPL_SIMT = 1, KATA_IMPL_TENSOR = 2 }; /* kata_opts.impl */
enum { KATA_FN_QUADRATIC = 0, KATA_FN_CHUNKED = 1, KATA_FN_CHUNK_STATE_SCAN = 2, KATA_FN_DECODE_STEP = 3,
       KATA_FN_BWD_QUADRATIC = 4, KATA_FN_BWD_CHUNKED = 5 };

/*
 * Options (plain data; zero-initialise, then set struct_size = sizeof(kata_opts)).
 *
 *  dtype          element type of q,k,v,out.
 *  feature_order  2: rank-one PSD lift of the normalised rows (default when 0 is passed).
 *                 1: rows of q,k are already-mapped features used as they are (no
 *                    normalisation, no lift; state d_k x d_v) -- the setting analysed in the appendix
 *                    "Associative-scan kernel", where the feature map has been applied beforehand.
 *  feature_groups 0 or 1: the full rank-one lift.  g = 2 or 4 (feature_order 2 only): the blockwise PSD map
 *                 psi_Mg(u) = (u_1 u_1^T, ..., u_g u_g^T) of the normalised row cut into g blocks of d_k/g
 *                 entries ("KATA-Mg"), with <psi(q),psi(k)> = sum_a (q_a . k_a)^2.  The state layouts then hold
 *                 the g blocks one after the other: DIRECT n_psi = g (d_k/g)^2, PACKED n_psi = g m(m+1)/2 with
 *                 m = d_k/g.
 *  state_layout   layout of the exported prefix states for feature_order 2:
 *                 DIRECT  n_psi = d_k^2, row a*d_k+b holds the (a,b) entry of sum k_hat k_hat^T (x) v;
 *                 PACKED  n_psi = d_k(d_k+1)/2, upper triangle a<=b in row-major order, diagonal
 *                         entries as they are and off-diagonal entries times sqrt(2) (the isometric
 *                         packing, so packed features keep the inner product (q_hat.k_hat)^2).
 *                 Ignored for feature_order 1 (n_psi = d_k).
 *  inter_chunk    kata_fwd_chunked only: SEQUENTIAL walks the chunks of a head in order
 *                 (Algorithm 1); SCAN splits the chunk axis into groups, reduces each group,
 *                 runs a log-depth exclusive scan over the group states and finishes every
 *                 group in parallel (section "Tree-scan inter-chunk reduction").  INTER_AUTO lets the
 *                 library choose: SCAN where the heads alone leave most of the GPU idle and the
 *                 sequence is long enough for the scan form's extra pass to pay (a model of the
 *                 tensor-core kernel's time in whole waves of CTAs decides); SEQUENTIAL otherwise,
 *                 on the fp32 kernels, for feature_order 1 (whose tensor-core path makes this choice
 *                 by itself) and whenever a state is handed in or out.  Both forms give the same
 *                 result up to the rounding order of the state sums.
 *  impl           AUTO picks the tensor-core kernels where they exist; SIMT / TENSOR force one
 *                 (TENSOR returns KATA_ERR_UNSUPPORTED_SHAPE where it does not exist).
 *  scan_group     chunks per scan group; 0 = library's choice (kata_chunk_state_scan: 1, i.e.
 *                 the paper's per-chunk pipeline, whenever s_pre/z_pre are requested).  The first-order
 *                 tensor-core path works in tiles of 128 tokens: it rounds the group up to whole tiles, and its
 *                 own choice may be a single group (one pass per head) when the heads alone fill the GPU;
 *                 kata_scan_plan reports what will run.  With more than one group it runs as ONE launch: the
 *                 CTAs take groups in order, build the state of a group alone, publish it, add up the groups
 *                 before it (a chained scan over the group states with an anchor every eighth group, summed in
 *                 a fixed order: bit-reproducible) and walk the group again for the outputs; the scan_rounds
 *                 that kata_scan_plan reports for this path are the anchor hops, not doubling rounds.  Its
 *                 waits on other CTAs are bounded (2 s); a CTA that gives up marks its group so that the
 *                 CTAs behind it give up at once.
 *  workspace      device scratch of at least kata_workspace_bytes(...) bytes, 256-byte aligned;
 *                 may be null when that size is 0.
 *  s_pre, z_pre   optional device outputs (fp32), both null or both non-null.
 *                 kata_chunk_state_scan: s_pre [B,H,N_C,n_psi,d_v], z_pre [B,H,N_C,n_psi], N_C = ceil(T/C),
 *                 the exclusive prefix chunk states, entry 0 along N_C being zero.
 *                 kata_fwd_chunked with inter_chunk = SEQUENTIAL (feature_order 2): s_pre [B,H,n_psi,d_v],
 *                 z_pre [B,H,n_psi], the state after the last token -- the state kata_decode_step
 *                 continues from (prefill -> decode).  Any other entry point: KATA_ERR_INVALID_ARG.
 *  device_status  optional device int, written only on a device-side timeout.
 *  stream         cudaStream_t as void* (null = the legacy default stream).
 *  s_init, z_init optional device inputs (fp32), both null or both non-null; kata_fwd_chunked with inter_chunk =
 *                 SEQUENTIAL and feature_order 2 only (anything else: KATA_ERR_INVALID_ARG).  The state before the
 *                 first token, s_init [B,H,n_psi,d_v], z_init [B,H,n_psi] in state_layout: the call continues a
 *                 sequence whose earlier tokens are summarised by that state (the recurrence "S_t = S_{t-1} +
 *                 psi(k_t) v_t^T" started from S_0 = s_init instead of 0), so feeding a long sequence in pieces,
 *                 each call's s_pre/z_pre being the next call's s_init/z_init, gives the outputs of the one long
 *                 call.  s_init may equal s_pre (and z_init z_pre): the state is then advanced in place.  Read
 *                 before anything is written.
 */
typedef struct kata_opts {
  uint32_t struct_size;
  int32_t dtype;
  int32_t feature_order;
  int32_t state_layout;
  int32_t inter_chunk;
  int32_t impl;
  int32_t scan_group;
  int32_t feature_groups;
  void* workspace;
  size_t workspace_bytes;
  float* s_pre;
  float* z_pre;
  int* device_status;
  void* stream;
  const float* s_init;
  const float* z_init;
} kata_opts;

/*
 * Quadratic ("flash-style") forward: the definition evaluated tile by tile, never forming
 * the d_k^2-wide state (section "Why the PSD feature keeps to O(T) or O(T^2)"; weights from
 * the rank-one lift identity <uu^T,vv^T>_F = (u^T v)^2).  O(T^2) work.  C is ignored.
 * Workspace: kata_workspace_bytes(KATA_FN_QUADRATIC, ...) -- the tensor-core path keeps the key scales
 * 1/||k||^2 there (one bf16 per key and head); the fp32 path needs none.
 */
int kata_fwd_quadratic(const void* q, const void* k, const void* v, void* out,
                       int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * Chunked-state forward: Algorithm 1 with the chunk equations
 *   S_[c+1] = S_[c] + Psi(K_[c])^T V_[c],  Z_[c+1] = Z_[c] + Psi(K_[c])^T 1,
 *   P = (Psi(Q_[c]) Psi(K_[c])^T) o M,  N = Psi(Q_[c]) S_[c] + P V_[c],
 *   D = Psi(Q_[c]) Z_[c] + P 1,  O_[c] = diag(D)^-1 N
 * (section "Chunkwise forward").  O(T) work, fp32 state.  opts->inter_chunk selects how
 * the inter-chunk recurrence is traversed; both give the same result up to fp32
 * re-association.  Workspace: kata_workspace_bytes(KATA_FN_CHUNKED, ...); the sequential walk on the tensor-core
 * path (bf16, d_k = d_v = 64, feature_order 2, no state pointers) splits the state of a head over
 * nine CTAs (five, six or ten with feature_groups 2 or 4) and needs about 0.15 KB per token, head and CTA there (scaled values, key scales, the CTAs' shares of the
 * output and a counter per tile); the environment variable KATA_CHUNKED_KERNEL=stream selects the one-CTA-per-value-
 * slice streaming kernel instead (no workspace; for comparisons).
 */
int kata_fwd_chunked(const void* q, const void* k, const void* v, void* out,
                     int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * Three-stage pipeline of the appendix "Associative-scan kernel": (i) chunk-local states
 * S_loc = Psi(K_[c])^T V_[c], Z_loc = 1^T Psi(K_[c]) for all (b,h,c) in parallel; (ii) exclusive
 * prefix along the chunk axis in ceil(log2 N) rounds; (iii) chunk output from the prefix and
 * the local C x C causal term.  Writes out; if opts->s_pre/z_pre are set it also writes the
 * exclusive-prefix chunk states there (which forces scan_group = 1).  With scan_group > 1 (or the library's choice)
 * the stages work on groups of chunks, which the paper's associativity argument allows: the same result up to the
 * rounding order of the state sums.  The first-order tensor-core path runs the three stages in one launch and its
 * stage (ii) as a chained scan over the group states (see opts->scan_group).
 * Workspace: kata_workspace_bytes(KATA_FN_CHUNK_STATE_SCAN, ...).
 */
int kata_chunk_state_scan(const void* q, const void* k, const void* v, void* out,
                          int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * One token of the recurrent form (section "Linear attention as a recurrence": S_t = S_{t-1} + psi(k_t) v_t^T,
 * Z_t = Z_{t-1} + psi(k_t), readout psi(q_t)^T S_t / psi(q_t)^T Z_t), for every (b,h): the constant-time decode
 * step that follows a prefill.
 *   q, k [B,H,d_k]; v, out [B,H,d_v] (element type opts->dtype, device pointers, 16-byte aligned);
 *   S [B,H,n_psi,d_v], Z [B,H,n_psi]: fp32 device state, updated IN PLACE (read and written once per call),
 *   in the layout of the exported prefix states (opts->state_layout / feature_order, see kata_opts): the
 *   s_pre/z_pre slice of a chunk written by kata_chunk_state_scan is a valid state to resume from, and an
 *   all-zero state starts a sequence.  out = 0 where the denominator is 0.
 * The state of a head is reduced in a fixed order: results are bit-reproducible.  opts->inter_chunk, impl,
 * scan_group are ignored; opts->s_pre/z_pre must be null.
 * Workspace: kata_workspace_bytes(KATA_FN_DECODE_STEP, B, H, 1, d_k, d_v, 0, opts).
 */
int kata_decode_step(const void* q, const void* k, const void* v, void* out, float* S, float* Z,
                     int B, int H, int d_k, int d_v, const kata_opts* opts);

/*
 * Backward of the forward pass: given dout = dL/dout [B,H,T,d_v], writes dq, dk [B,H,T,d_k] and dv [B,H,T,d_v]
 * (element type opts->dtype, device pointers, 16-byte aligned, fully overwritten), the gradients of
 * L = sum(dout * out) through out_t = sum_{i<=t} w_ti v_i / sum_{i<=t} w_ti, the weights w_ti and the l2
 * normalisation of the rows (chain rule through the definition; the forms of the forward are one function, so
 * this is the backward of all of them).  Evaluated tile by tile like kata_fwd_quadratic: the forward is
 * recomputed (no saved activations are needed), O(T^2) work, fp32 arithmetic, every sum in a fixed order
 * (bit-reproducible).  Rows whose normaliser is 0 (out = 0) and zero rows of q or k get zero gradients.
 * feature_order, feature_groups as in the forward; inter_chunk, scan_group, state_layout are ignored;
 * s_pre/z_pre/s_init/z_init must be null.  Tensor-core kernels for bf16 and feature_order 2: feature_groups 1 with
 * d_k = d_v = 64 or narrower rows zero-padded in the workspace, feature_groups 2 or 4 with d_k = d_v = 64 (the
 * weights P and E pass through bf16 there, as P does in the forward); fp32 kernels for everything else.
 * Workspace: kata_workspace_bytes(KATA_FN_BWD_QUADRATIC, B, H, T, d_k, d_v, 0, opts).
 */
int kata_bwd_quadratic(const void* q, const void* k, const void* v, const void* dout, void* dq, void* dk, void* dv,
                       int B, int H, int T, int d_k, int d_v, const kata_opts* opts);

/*
 * The same gradients as kata_bwd_quadratic in O(T) work: the two-pass linear-state backward of the table
 * "Training-step latency versus sequence length".  A forward sweep over the chunks carries the state of the forward
 * pass (S = sum psi(k_hat) v^T, Z = sum psi(k_hat)), recomputes out_t and its normaliser and produces dq; a reverse
 * sweep carries the state sum psi(q_hat_t) [dout_t / D_t, (dout_t . out_t) / D_t] of the tokens behind and produces dk
 * and dv; the terms inside a chunk come from its C x C causal scores.  Arguments, layouts and error values as for
 * kata_bwd_quadratic; C must be 64.  fp32 arithmetic on plain FMAs for both element types (bf16 tensors are widened on
 * load and rounded once on store), every sum in a fixed order (bit-reproducible).  Supported: feature_order 2,
 * feature_groups 1, d_k in {16, 32, 64}, d_v a multiple of 8 up to 64 (KATA_ERR_UNSUPPORTED_SHAPE otherwise,
 * also for opts->impl = KATA_IMPL_TENSOR); inter_chunk, scan_group, state_layout are ignored; s_pre/z_pre/s_init/
 * z_init must be null.  Rows whose normaliser is 0 and zero rows of q or k get zero gradients.
 * Workspace: kata_workspace_bytes(KATA_FN_BWD_CHUNKED, B, H, T, d_k, d_v, 64, opts) bytes, about
 * 4 (2 d_k + d_v + (d_v / 8)(d_k + 1) + 2) bytes per token and head (2.9 KB at d_k = d_v = 64).
 */
int kata_bwd_chunked(const void* q, const void* k, const void* v, const void* dout, void* dq, void* dk, void* dv,
                     int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * Same computation as entry point `fn` (a KATA_FN_* value) but q,k,v,out are HOST pointers
 * (pinned memory recommended).  The inputs are copied to a staging area inside the workspace,
 * the kernels run, and out is copied back, all enqueued on opts->stream; the caller synchronises
 * the stream before reading out.  Workspace: kata_workspace_bytes(fn | KATA_FN_HOST_IO, ...).
 * Long sequences (kata_fwd_chunked, inter_chunk = SEQUENTIAL, bf16, d_k = d_v = 64, feature_order 2, T >= 32768,
 * no state pointers in opts) are processed in up to sixteen pieces of the token axis: the copy in of the next piece
 * and the copy back of the previous one run on two streams owned by the library while the current piece is
 * computed, each piece starting from the state the previous one left ("Linear attention as a recurrence").  The
 * caller's stream waits for all of it -- also when a piece fails: the error is returned only after the caller's
 * stream has been made to wait for every copy already queued on the library's streams -- so the contract above is
 * unchanged.  The result is the same function as the one-pass call; the pieces run on the streaming kernel, which
 * rounds at other places than the feature-split kernel of the one-pass call (both inside the bf16 tolerance).
 * This route creates two streams and seven events per device on first use and keeps them; calls that take it are
 * serialised inside the library by a process-wide mutex; host memory that is not pinned makes the copies synchronous.
 * The paper has no counterpart; this is the end-to-end path measured by the benchmark.
 */
#define KATA_FN_HOST_IO 0x100
int kata_fwd_host(int fn, const void* q_host, const void* k_host, const void* v_host, void* out_host,
                  int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * kata_chunk_state_scan for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this entry point exists for integration reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework whose allocator
 * owns all device memory and hands out no scratch, in a plugin called under a "no allocation after
 * initialisation" rule, or on a serving path that must not touch the allocator because an
 * allocation may synchronise the device.  Such callers still pass q, k, v and out; only the scan
 * scratch (group states and the ping-pong buffer of the log-depth scan) is supplied by the library,
 * from a fixed device array of KATA_STATIC_SCRATCH_BYTES bytes that is part of the library image.
 * Every GPU context that loads the library holds that array until it exits.
 *
 *  - Same arguments, layouts, results and status codes as kata_chunk_state_scan, except:
 *    opts->workspace / workspace_bytes are ignored; opts->s_pre / z_pre must be null
 *    (KATA_ERR_INVALID_ARG otherwise); if opts->scan_group is 0 the library picks the smallest
 *    power-of-two group size whose scratch fits the array.
 *  - If the scratch needed exceeds KATA_STATIC_SCRATCH_BYTES (large B*H with a small scan_group, or
 *    simply too many heads), nothing is launched and KATA_ERR_WORKSPACE_TOO_SMALL is returned.  bf16 rows narrower
 *    than 64 entries take the zero-padded route of the tensor-core kernels, whose padded copies of q, k, v and out
 *    (4 * B*H*T * 128 bytes) must fit the array as well: about 65 thousand tokens over all heads.
 *  - The call allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *  - The first call on each device looks up the device address of the array (one
 *    cudaGetSymbolAddress, with that device current).  Make that first call outside any stream
 *    capture; later calls on the same device do no set-up.
 *  - All calls on a device share the one array, and it keeps whatever the last call left in it.
 *    Nothing in it has to start at zero: every word a call reads, the same call has written first.
 *    Two calls that overlap on the GPU (different streams, or different host threads without
 *    ordering between their streams) race on the array and give wrong results; serialise them.
 */
#define KATA_STATIC_SCRATCH_BYTES (32u << 20)
int kata_chunk_state_scan_static(const void* q, const void* k, const void* v, void* out,
                                 int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * Bytes of device workspace entry point `fn` needs for these sizes and options (0 if none);
 * returns 0 also for invalid arguments (the entry point itself reports the error).
 */
size_t kata_workspace_bytes(int fn, int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts);

/*
 * Pieces of the token axis kata_fwd_host(fn, ...) would work in for these sizes and options, given a workspace of
 * kata_workspace_bytes(fn | KATA_FN_HOST_IO, ...) bytes: 1 = copy in, run, copy back; more = the overlapped
 * piecewise route described at kata_fwd_host; *piece_tokens (may be null) receives the length of a piece.
 * Returns a KATA_ERR_* value for invalid arguments.  For reporting and tests.
 */
int kata_host_plan(int fn, int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts, int* pieces,
                   int* piece_tokens);

/* Number of scan groups, chunks per group and rounds of the scan over the group states (doubling rounds; anchor hops on
 * the first-order tensor-core path) the library would use; beyond 65535 heads, those of a full slab of heads.  For
 * reporting and tests. */
int kata_scan_plan(int fn, int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts,
                   int* n_groups, int* chunks_per_group, int* scan_rounds);

/* Number of kernels the last successful call on this host thread enqueued. */
int kata_last_launch_count(void);

/* Which kernels the last successful call on this host thread used: KATA_IMPL_SIMT or KATA_IMPL_TENSOR. */
int kata_last_impl(void);

const char* kata_status_string(int status);
int kata_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KATA_H_ */
