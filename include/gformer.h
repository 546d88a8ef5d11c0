/*
 * libgformer -- hybrid attention forward pass (GFormer) for NVIDIA B200 (sm_100a).
 *
 * The layer splits the H heads of Q, K, V into two groups (Sec. III-A): heads
 * [0, h_sparse) run causal windowed softmax attention, heads [h_sparse, H) run
 * causal linear attention; each head writes its own slot of the output.
 *
 * Conventions common to every entry point
 *   - q, k, v, o and every state buffer are DEVICE pointers owned by the caller.  The
 *     library never allocates, frees or keeps them.  Pointers must be 16-byte aligned.
 *   - Logical tensor shape is [B, H, N, d]; `layout` says how it is stored:
 *     GF_BHND = contiguous [B, H, N, d]; GF_BNHD = contiguous [B, N, H, d] (the order
 *     the paper writes, Sec. III-A).  d is 64 or 128.
 *   - dtype is the storage type of q, k, v, o and of the KV ring (GF_F32 or GF_BF16);
 *     all accumulation is fp32; the linear state S, z is always fp32.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t cast to void*, NULL = the
 *     legacy default stream) and return without synchronising.
 *   - The return value is a gf_status.  Argument errors are found on the host before
 *     anything is launched and leave every buffer untouched.  Nothing throws or aborts.
 *   - `ws` is caller-provided device scratch of at least gformer_workspace_bytes(...)
 *     bytes, 256-byte aligned; the tensor-core (bf16) kernels keep a device status word
 *     there, and the linear-attention kernel the per-segment states and flags through
 *     which the CTAs that share one (batch, head) chain hand the running state on.  The
 *     library clears what it needs inside the call, so ws may hold anything on entry, but
 *     two calls that run concurrently must not share one ws.
 *   - o must not alias an input.
 *   - Precondition of every call that runs causal linear attention on the tensor-core path
 *     (gformer_causal_linear_attn*, gformer_hybrid_attn*): when the plan cuts a chain into
 *     segments (gformer_linear_plan reports more than one), the kernel's CTAs -- at most one per
 *     SM, never more than the device has SMs -- wait for one another's states, so all of them
 *     must get an SM while the kernel runs.  On a device that is otherwise idle, or shared with
 *     kernels that end by themselves, they do.  Two such kernels side by side could each hold a
 *     part of the SMs and wait for the rest, so the library orders them per device: such a kernel
 *     starts only when the previous one -- from whatever stream or host thread -- has finished
 *     (an event wait in front of the launch).  Inside a stream capture that wait is not possible:
 *     graphs that contain such a call must not be replayed side by side on one device.  What must
 *     not run beside such a call is work that holds SMs until the call has finished (a persistent
 *     kernel that itself waits for this call's results): the waits are bounded, so the outcome is
 *     GF_ERR_TIMEOUT from
 *     gformer_last_device_status and undefined outputs, not a hang.  Whole chains (one segment),
 *     the windowed heads and the bidirectional layer have no such precondition: their CTAs
 *     never wait for other CTAs.
 */
#ifndef GFORMER_H_
#define GFORMER_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GF_OK = 0,
  GF_ERR_INVALID_ARG = 1, /* null/misaligned pointer, size out of range, aliasing */
  GF_ERR_UNSUPPORTED = 2, /* valid request the library has no kernel for (e.g. d = 96) */
  GF_ERR_WORKSPACE = 3,   /* ws missing or smaller than gformer_workspace_bytes */
  GF_ERR_CUDA = 4,        /* a CUDA call or launch failed */
  GF_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (see last_device_status) */
} gf_status;

typedef enum { GF_F32 = 0, GF_BF16 = 1 } gf_dtype;
typedef enum { GF_BHND = 0, GF_BNHD = 1 } gf_layout;
/* Feature map of the linear heads.
 * GF_PHI_ELU1: phi(x) = elu(x) + 1, element by element (Sec. II-B).
 * GF_PHI_FAVOR_POS: the positive random features Sec. III-A and III-C name ("positive orthogonal
 *   random features"; the paper prints no formula, this is the cited Performer paper's):
 *       phi_W(x)[a] = exp(<w_a, x> - |x|^2 / 2) / sqrt(d),   a = 0 .. d-1,
 *   with d features because the state of Algorithm 1 is d x d.  The projection vectors w_a are the
 *   caller's (argument W of the ..._w entry points): one d x d matrix per linear head, row a = w_a,
 *   in the storage dtype of q.  x is taken as passed (no extra scale, no stabiliser): the state S, z is
 *   the definition's.  The kernels use the fact that a factor common to all features of one query
 *   cancels in the output (they take the query features relative to the row's largest projection), so
 *   only the key features must be representable: |k|^2 / 2 - <w_a, k> up to about 85 (fp32) is fine. */
typedef enum { GF_PHI_ELU1 = 0, GF_PHI_FAVOR_POS = 1 } gf_phi;

/* Process-wide knobs for tests and benchmarks (gformer_set_tuning). */
typedef enum {
  GF_TUNE_FORCE_SIMT = 0, /* 1: never take the tensor-core kernels (default 0)              */
  GF_TUNE_LINEAR_SPLIT = 1, /* 128-row chunks per sequence segment of a linear chain: 0 = auto,
                               -1 = never cut a chain (the one-pass form of the kernel)          */
  GF_TUNE_LINEAR_CTAS = 2,  /* gformer_hybrid_attn: CTAs of the persistent linear-attention kernel
                               when it shares the GPU with the windowed heads; 0 = auto, else an
                               upper bound in [1, 65535] (the SM count bounds it too)              */
  GF_TUNE_WAIT_KCYCLES = 3, /* how long a device-side wait may last before the kernel gives up, in
                               units of 1024 SM cycles; 0 = the default (about two seconds)       */
  GF_TUNE_TEST_DROP_FLAG = 4 /* failure injection for tests: n > 0 makes the cut-chain form of the
                               linear kernel never raise the hand-over flag of its n-th segment, so
                               that the next segment's wait runs out; 0 = off                      */
} gf_tuning_key;

/* Decode-time state of one batch (see gformer_decode_step).  The struct lives in host
 * memory; the four pointers are device pointers owned by the caller. */
typedef struct {
  void* k_cache;   /* [B, h_sparse, w, d] dtype; ring: token j is in slot j mod w */
  void* v_cache;   /* [B, h_sparse, w, d] dtype                                   */
  float* S;        /* [B, H - h_sparse, d, d] fp32, S[a][c] = sum_j phi(k_j)[a] v_j[c] */
  float* z;        /* [B, H - h_sparse, d]    fp32, z[a]    = sum_j phi(k_j)[a]        */
  long long t;     /* tokens absorbed so far (whole batch in lock step)           */
  int B, H, d, w, h_sparse;
  int dtype;       /* gf_dtype of the ring                                         */
} gf_decode_state;

const char* gformer_status_string(int status);
int gformer_version(void);

/* Number of windowed heads used when a caller passes h_sparse < 0:
 * max(1, round(3 H / 16)) -- 3 of 16 heads is the causal optimum reported in Sec. IV-D. */
int gformer_default_h_sparse(int H);

/* Sets a gf_tuning_key; returns GF_OK or GF_ERR_INVALID_ARG.  Every entry point reads each knob
 * once when it is called; a knob changed while a call is being set up applies from the next call.
 * gformer_workspace_bytes depends on GF_TUNE_FORCE_SIMT and GF_TUNE_LINEAR_SPLIT: query it again
 * after changing one of them (a workspace that has become too small is refused with
 * GF_ERR_WORKSPACE, never overrun). */
int gformer_set_tuning(int key, int value);

/* How the tensor-core linear-attention kernel would cut `chains` (batch, head) sequences of N
 * tokens (bf16, d in {64, 128}) when it runs on `ctas` CTAs (0: one per SM of a B200): the
 * number of sequence segments per chain and the chunks (of 128 tokens) of the longest one.  One
 * segment with GF_TUNE_LINEAR_SPLIT on auto means the one-pass form of the kernel; more mean the
 * two-pass form with a state hand-over between segments (the chunked regrouping of Algorithm 1
 * is exact either way).  Host arithmetic only; honours GF_TUNE_LINEAR_SPLIT.  Returns GF_OK, or
 * GF_ERR_INVALID_ARG / GF_ERR_UNSUPPORTED without touching the outputs. */
int gformer_linear_plan(int chains, int N, int d, int ctas, int* segments, int* chunks_per_segment);

/* The same plan with its parts named.  With somewhat more chains than CTAs the kernel is launched
 * twice: the first *whole_chains chains (full rounds of one chain per CTA) in the one-pass form, the
 * leftover chains behind them in the two-pass form, cut into *segments segments of at most
 * *chunks_per_segment chunks -- the figures gformer_linear_plan reports.  *whole_chains is 0 when
 * every chain is cut and `chains` (with one segment) when none is.  Same arguments, status codes
 * and behaviour on error as gformer_linear_plan; whole_chains must not be null. */
int gformer_linear_plan_parts(int chains, int N, int d, int ctas, int* whole_chains, int* segments,
                              int* chunks_per_segment);

/* Algorithm 2 (Sec. III-D): the share p' in (0, 1) of a problem given to engine 0 at which the two
 * latency estimates  p size flops_per0 / perf0  and  (1 - p) size flops_per1 / perf1  are equal
 * (size cancels).  flops_per_i: work per unit of the part engine i runs; perf_i: that engine's
 * measured rate in the same work unit per second -- measured seconds per head and a rate of 1 do
 * as well.  Host arithmetic in fp64, no device work.  p_out: host pointer.  Returns GF_OK, or
 * GF_ERR_INVALID_ARG (null pointer, a non-positive or non-finite input) without touching *p_out. */
int gformer_partition_balance(double flops_per0, double flops_per1, double perf0, double perf1, double* p_out);

/* The FLOP model of Sec. III-D for H heads of width E over B sequences of N tokens with window W:
 * h_sparse windowed heads cost 5 B h_sparse N W / perf_sparse seconds and the H - h_sparse linear
 * heads 8 B N ((H - h_sparse) E)^2 / perf_linear (both formulas as the section prints them;
 * perf_* in FLOP/s).  *h_sparse_out receives the whole number of windowed heads in [0, H] for which
 * the two estimates are closest (the smaller count on a tie); the optional latency outputs (host
 * pointers, may be null) receive the two estimates at that count.  Host arithmetic in fp64.
 * Returns GF_OK, or GF_ERR_INVALID_ARG (null h_sparse_out, a size below 1, a non-positive or
 * non-finite rate) without touching the outputs. */
int gformer_partition_heads(int B, int H, int N, int E, int W, double perf_sparse, double perf_linear,
                            int* h_sparse_out, double* latency_sparse_out, double* latency_linear_out);

/* Algorithm 2 fed with measured times (Sec. III-D; the section feeds it micro-benchmarked rates): from the
 * seconds one windowed head and one linear head cost at this problem size, the balanced share
 * *p_out of windowed heads (gformer_partition_balance with the seconds as work and rates of 1), that
 * share as a whole number of the H heads (*h_sparse_out, nearest, in [0, H]), and the two rates in
 * the units of the section's FLOP model that the measurements imply: one windowed head is
 * 5 B N W flops, H linear heads together 8 B N (H E)^2.  All outputs are host pointers and must not be
 * null.  Host arithmetic in fp64.  Returns GF_OK, or GF_ERR_INVALID_ARG (null pointer, size below 1,
 * a non-positive or non-finite time) without touching the outputs. */
int gformer_partition_from_times(int B, int H, int N, int E, int W, double seconds_per_sparse_head,
                                 double seconds_per_linear_head, double* p_out, int* h_sparse_out,
                                 double* perf_sparse_out, double* perf_linear_out);

/* Number of kernels the library has launched in this process so far (all entry points,
 * all streams).  For accounting in benchmarks. */
unsigned long long gformer_launch_count(void);

/* Scratch bytes the attention entry points need for this problem (never 0). */
size_t gformer_workspace_bytes(int B, int H, int N, int d, int w, int h_sparse, int dtype);
/* The same for a given feature map of the linear heads: with GF_PHI_FAVOR_POS on the tensor-core path
 * the features of Q and K are written to the workspace first (two bf16 tensors of the linear heads'
 * size), so more is needed; with GF_PHI_ELU1 this is gformer_workspace_bytes. */
size_t gformer_workspace_bytes_phi(int B, int H, int N, int d, int w, int h_sparse, int dtype, int phi);

/* Synchronises `cuda_stream`, reads the device status word kept in ws and returns
 * GF_OK, GF_ERR_TIMEOUT (a bounded wait inside a tensor-core kernel gave up; outputs of
 * that call are undefined) or GF_ERR_CUDA.  ws must have been used by a previous call. */
int gformer_last_device_status(void* ws, void* cuda_stream);

/*
 * Causal windowed softmax attention on all H heads (Eq. 1 restricted by the causal
 * mask of Sec. II-A and the fixed left window of Sec. III-B):
 *   o_i = sum_j p_ij v_j,  p_ij = softmax_j(scale * <q_i, k_j>),  j in [max(0, i-w+1), i].
 * Token i attends to w keys, itself included; rows near the start see fewer.  w >= N is
 * full causal attention.  scale <= 0 selects 1/sqrt(d).  1 <= w; N >= 1.
 */
int gformer_window_attn(const void* q, const void* k, const void* v, void* o,
                        int B, int H, int N, int d, int w, float scale,
                        int dtype, int layout, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The windowed heads of the bidirectional ("self") layer (Sec. II-A: tokens attend to the
 * left and to the right, as in ViT): Eq. 1 without the causal mask over a two-sided window,
 *   j in [max(0, i-w+1), min(N-1, i+w-1)]   (the causal window mirrored: |i - j| < w;
 * the paper prints no two-sided rule, this is the reading taken).  Same arguments, layouts
 * and errors as gformer_window_attn.
 */
int gformer_window_attn_self(const void* q, const void* k, const void* v, void* o,
                        int B, int H, int N, int d, int w, float scale,
                        int dtype, int layout, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Causal linear attention on all H heads (Algorithm 1, readout after the updates of
 * step i; phi applied to raw q and k, no logit scale):
 *   S_i = S_{i-1} + phi(k_i) v_i^T,  z_i = z_{i-1} + phi(k_i),
 *   o_i = phi(q_i)^T S_i / <phi(q_i), z_i>.
 * The phi(K)^T V outer products are accumulated by prefix sum, `chunk` rows at a time on
 * the tensor-core path (0 = library default; otherwise 128).
 * S_io [B,H,d,d] / z_io [B,H,d] (fp32, both or neither): when given they hold the state
 * before token 0 on entry (zero them for a fresh sequence) and the state after token
 * N-1 on return.
 */
int gformer_causal_linear_attn(const void* q, const void* k, const void* v, void* o,
                               int B, int H, int N, int d, int phi, int chunk,
                               float* S_io, float* z_io,
                               int dtype, int layout, void* ws, size_t ws_bytes, void* cuda_stream);

/* gformer_causal_linear_attn with the feature map's parameter: W is null for GF_PHI_ELU1 and, for
 * GF_PHI_FAVOR_POS (Sec. III-A / III-C), a device pointer to the projections [H, d, d] in the storage
 * dtype of q (16-byte aligned; row a of head h's matrix is w_a).  Workspace: gformer_workspace_bytes_phi.
 * GF_ERR_INVALID_ARG when W and phi do not go together. */
int gformer_causal_linear_attn_w(const void* q, const void* k, const void* v, void* o,
                                 int B, int H, int N, int d, int phi, const void* W, int chunk,
                                 float* S_io, float* z_io,
                                 int dtype, int layout, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * gformer_causal_linear_attn for callers that cannot allocate device memory (no counterpart
 * in the paper; it exists for the deployment, not for the method).
 *
 * Who needs it: code that receives tensors and a stream but does not own an allocator --
 * a plug-in inside a framework whose memory pool holds the whole device, a capture-time or
 * real-time path in which cudaMalloc and the synchronisation it implies are off limits.  Such
 * a caller has nowhere to get the `ws` scratch the linear-attention kernel uses for the
 * states its thread blocks pass from one sequence segment to the next.
 *
 * This entry point takes that scratch from a fixed array of gformer_noalloc_scratch_bytes()
 * = 8 MiB that is part of the library image (each GPU that loads the library keeps it until
 * the process exits).  It allocates and frees nothing, in CUDA or on the host side of any
 * framework.  Arguments, results and status codes are those of gformer_causal_linear_attn;
 * in addition GF_ERR_WORKSPACE is returned, before anything is launched or written, when
 * gformer_workspace_bytes(B, H, N, d, 1, 0, dtype) exceeds the array (for d = 128 that is
 * about 120 sequence segments of 1024 tokens in total, e.g. B*H = 4 chains of 8192 tokens).
 *
 * The first call on a device looks up the array's device address; make that call once
 * outside any stream capture.  All calls share the one array: it still holds the previous
 * call's contents on entry (the kernel clears the words it relies on), and two calls whose
 * kernels overlap on the GPU -- different streams, or different host threads -- race on it.
 */
size_t gformer_noalloc_scratch_bytes(void);
int gformer_causal_linear_attn_noalloc(const void* q, const void* k, const void* v, void* o,
                                       int B, int H, int N, int d, int phi, int chunk,
                                       float* S_io, float* z_io, int dtype, int layout,
                                       void* cuda_stream);
/* The device status word of the fixed array on the current device, as gformer_last_device_status
 * reads it for a caller-owned workspace (which this entry point hides): synchronises `cuda_stream`
 * and returns GF_OK, GF_ERR_TIMEOUT (a bounded wait of the last call gave up -- what two calls that
 * overlapped on the GPU can cause; that call's outputs are undefined) or GF_ERR_CUDA.  No counterpart
 * in the paper.  Allocates nothing. */
int gformer_noalloc_last_device_status(void* cuda_stream);

/*
 * The hybrid layer (Sec. III-A): heads [0, h_sparse) as gformer_window_attn, heads
 * [h_sparse, H) as gformer_causal_linear_attn with a zero initial state; h_sparse < 0
 * selects gformer_default_h_sparse(H).  The two groups run side by side on the device (on two
 * streams of the library's own, forked from and joined back into `cuda_stream`, so the caller
 * sees a single-stream call that may also be captured into a CUDA graph).  Host threads may call
 * concurrently, each with its own workspace and stream; on one device their fork .. join sections
 * are enqueued one after the other.
 * state_out (may be NULL): if given, its B, H, d, w, h_sparse, dtype must match the call
 * and its buffers receive the decode state after the N tokens: the last min(N, w) keys
 * and values of the windowed heads in ring slots j mod w, the final S and z of the linear
 * heads, and t = N.
 */
int gformer_hybrid_attn(const void* q, const void* k, const void* v, void* o,
                        int B, int H, int N, int d, int w, int h_sparse, float scale,
                        int phi, int chunk, int dtype, int layout,
                        gf_decode_state* state_out,
                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The bidirectional ("self") layer (Sec. II-A / III-A: the same head split, no causal mask):
 * heads [0, h_sparse) as gformer_window_attn_self, heads [h_sparse, H) global linear attention,
 *   S = sum_j phi(k_j) v_j^T,  z = sum_j phi(k_j)  over all j,   o_i = phi(q_i)^T S / (phi(q_i) . z)
 * (Sec. II-B, rows normalised as in Algorithm 1).  bf16 storage takes the tensor-core kernels,
 * fp32 storage (or GF_TUNE_FORCE_SIMT) CUDA-core kernels in fp32 arithmetic, as in the causal
 * layer.  Streams, graph capture and host threads as for gformer_hybrid_attn.  Workspace:
 * gformer_workspace_bytes.
 */
int gformer_hybrid_attn_self(const void* q, const void* k, const void* v, void* o,
                             int B, int H, int N, int d, int w, int h_sparse, float scale,
                             int phi, int dtype, int layout,
                             void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * One autoregressive step for token index st->t: q, k, v, o are [B, H, d].  Windowed
 * heads store k, v in ring slot t mod w and take the softmax over the min(t+1, w) cached
 * keys (the window rule of Sec. III-B); linear heads run one iteration of Algorithm 1 on
 * (S, z).  Updates the state buffers in place and increments st->t on success.  The
 * result for token t equals row t of the full-sequence layer.
 */
int gformer_decode_step(const void* q, const void* k, const void* v, void* o,
                        gf_decode_state* st, float scale, int phi, void* cuda_stream);

/*
 * The same step for a batch whose sequences are at different positions (continuous batching):
 * t_seq is a device array of B token counts, 8-byte aligned, owned by the caller.  Sequence b is
 * processed as token index t_seq[b] exactly as gformer_decode_step would process it at st->t =
 * t_seq[b] (ring slot t_seq[b] mod w, softmax over min(t_seq[b] + 1, w) cached keys); a negative
 * entry marks an idle slot: its state is left untouched and its output rows are zero.  The step
 * itself increments the non-negative entries on the device (so a captured CUDA graph of steps
 * advances by itself); while a step is running, bits 48..62 of an entry count the heads that
 * have read it, so positions must stay below 2^48 and H at most 4096 (GF_ERR_UNSUPPORTED), and
 * the array must not be read or written while a step is in flight.  st->t is neither read nor
 * changed.  The paper decodes whole batches in
 * lock step (Sec. III-A); this entry point only lets the rows of one batch be at different t.
 */
int gformer_decode_step_ragged(const void* q, const void* k, const void* v, void* o,
                               gf_decode_state* st, long long* t_seq, float scale, int phi,
                               void* cuda_stream);

/* The three layer-level entry points with the feature map's parameter (see gformer_causal_linear_attn_w):
 * W [H - h_sparse, d, d] holds the projections of the linear heads only, in head order; null for
 * GF_PHI_ELU1.  Everything else as in gformer_hybrid_attn, gformer_hybrid_attn_self and
 * gformer_decode_step (a decode state filled by gformer_hybrid_attn_w must be advanced with the same phi
 * and W).  Workspace of the first two: gformer_workspace_bytes_phi. */
int gformer_hybrid_attn_w(const void* q, const void* k, const void* v, void* o,
                          int B, int H, int N, int d, int w, int h_sparse, float scale,
                          int phi, const void* W, int chunk, int dtype, int layout, gf_decode_state* state_out,
                          void* ws, size_t ws_bytes, void* cuda_stream);
int gformer_hybrid_attn_self_w(const void* q, const void* k, const void* v, void* o,
                               int B, int H, int N, int d, int w, int h_sparse, float scale,
                               int phi, const void* W, int dtype, int layout,
                               void* ws, size_t ws_bytes, void* cuda_stream);
int gformer_decode_step_w(const void* q, const void* k, const void* v, void* o,
                          gf_decode_state* st, float scale, int phi, const void* W, void* cuda_stream);
/* gformer_decode_step_ragged with the feature map's parameter (W as above). */
int gformer_decode_step_ragged_w(const void* q, const void* k, const void* v, void* o,
                                 gf_decode_state* st, long long* t_seq, float scale, int phi, const void* W,
                                 void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* GFORMER_H_ */
