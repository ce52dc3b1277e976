/*
 * mamba_spec -- multi-step Mamba verification step for speculative decoding,
 * hand-written for NVIDIA B200 (sm_100a).  C ABI; no C++ or framework types.
 *
 * What one call computes (paper: Sec. 4.2 "MultiStep" and Algorithm 2 "Verify";
 * Sec. 4.3 for the fusion of replay, multi-step decoding and caching in one
 * kernel and, in its footnote, the rolling window of the causal convolution;
 * Eq. 1 and Sec. 2.2 for the recurrence and its on-the-fly discretisation):
 *
 *   For sequence b the cache holds the SSM state h_i and the last W-1 conv
 *   inputs, both as of the last token folded into the cache.  The caller hands
 *   over T_b = j_b + k token rows: first the j_b = n_prev_accepted[b] tokens
 *   accepted last round (not yet folded in), then k = k_draft new draft tokens.
 *   For t = 0 .. T_b-1, head h, channel p, state column n:
 *
 *     xc_t[p]  = act( conv_b[c] + sum_{w<W-1} conv_w[c][w] * xin_{t-(W-1)+w}[p] + conv_w[c][W-1] * x_t[p] )
 *                (c = h*P + p; xin of negative index comes from conv_state; act = SiLU or identity)
 *     h_t[p,n] = exp(dt_t * A_h) * h_{t-1}[p,n] + dt_t * xc_t[p] * B_t[n]
 *     y_t[p]   = sum_n C_t[n] * h_t[p,n] + D_h * xc_t[p]          ( * SiLU(z_t[p]) when gated )
 *
 *   All T_b rows of y are returned (the caller's FirstConflict needs the k
 *   draft rows; the j_b replayed rows feed the next layer's replay).  Only the
 *   state and conv window AFTER token j_b-1 are written back, in place; when
 *   j_b = 0 the cache is left untouched.  No per-token state is materialised.
 *   With MAMBA_SPEC_FLAG_STATE_K the state and conv window after ALL T_b
 *   tokens (Algorithm 2's second cached state, h_k) go to a second pair of
 *   buffers as well; which of the two becomes the cache after a fully accepted
 *   round is the caller's choice.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the comment says HOST.  The
 *     caller owns all tensors and the stream; the library owns only the
 *     context (a few KB of device memory: pending n_prev, a status word).
 *   - Tensors are dense, row-major, last index fastest, 16-byte aligned.
 *     "act dtype" is float32 or bfloat16 as chosen at init; state, A, D,
 *     conv_w, conv_b are always float32.
 *   - Token rows are left-aligned in a [batch][t_max] slab; rows t >= T_b are
 *     never used (x, z, dt, B, C; the streaming kernel may fetch them) and never written (y).
 *   - Head h uses B group h / (n_heads / n_groups_b) and C group
 *     h / (n_heads / n_groups_c).
 *   - Calls are asynchronous on io->stream and ordered by it; nothing
 *     synchronises except mamba_spec_status, mamba_spec_get_n_prev and
 *     mamba_spec_destroy.  One context must not be used from two streams at
 *     the same time.
 *   - Every function returns MAMBA_SPEC_OK (0) or a negative MAMBA_SPEC_ERR_*;
 *     the message is available from mamba_spec_last_error.  Nothing throws,
 *     aborts or traps.  There is no CPU fallback: without a CUDA device init
 *     fails with MAMBA_SPEC_ERR_CUDA.
 */
#ifndef MAMBA_SPEC_H
#define MAMBA_SPEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MAMBA_SPEC_OK 0
#define MAMBA_SPEC_ERR_INVALID_ARG (-1) /* null pointer, negative size, value out of range      */
#define MAMBA_SPEC_ERR_BAD_SHAPE (-2)   /* shape inconsistent with the context's configuration  */
#define MAMBA_SPEC_ERR_MISALIGNED (-3)  /* a tensor pointer is not 16-byte aligned              */
#define MAMBA_SPEC_ERR_UNSUPPORTED (-4) /* shape outside what any kernel here handles           */
#define MAMBA_SPEC_ERR_CUDA (-5)        /* a CUDA runtime call failed (message has the detail)  */
#define MAMBA_SPEC_ERR_NOT_INIT (-6)    /* context is null or destroyed                         */

#define MAMBA_SPEC_DTYPE_F32 0
#define MAMBA_SPEC_DTYPE_BF16 1

#define MAMBA_SPEC_FLAG_GATE 1      /* y <- y * SiLU(z); io->z must then be non-null */
#define MAMBA_SPEC_FLAG_CONV_SILU 2 /* SiLU after the conv (else identity)           */
#define MAMBA_SPEC_FLAG_Y_F32 4     /* y is float32 whatever the act dtype is        */
#define MAMBA_SPEC_FLAG_STATE_K 8   /* second snapshot: the cache after ALL T_b tokens, to io->state_k /
                                       io->conv_state_k (Algorithm 2 caches h_j and h_k; Fig. 2)  */
#define MAMBA_SPEC_FLAG_MAMBA1 16   /* Mamba-1 parameterisation (Algorithm 1, Sec. 2.2: the form of the paper's pure-Mamba
                                       verifiers): the interval is per channel and A per channel and state column,
                                         h_t[p,n] = exp(dt_t[c] * A[c][n]) * h_{t-1}[p,n] + dt_t[c] * xc_t[p] * B_t[n],
                                         y_t[p]   = sum_n C_t[n] * h_t[p,n] + D[c] * xc_t[p],        c = h*P + p
                                       with dt [batch][t_max][H*P], A [H*P][N], D [H*P].  Runs in the generic kernel. */
#define MAMBA_SPEC_FLAG_DT_SOFTPLUS 32 /* dt arrives raw: the kernel uses softplus(dt + io->dt_bias) (Sec. 2.2: the
                                       intervals come out of a network)                                            */
#define MAMBA_SPEC_FLAG_COMMIT_SELECTS 64 /* needs FLAG_STATE_K.  Algorithm 2 keeps h_k when every draft was accepted and
                                       h_j otherwise: (state, conv_state) and (io->state_k, io->conv_state_k) become two
                                       equal buffers per sequence, one of which holds the sequence's cache.  A verify
                                       call reads the cache where it is, puts the state at the verified position back
                                       there and the state after all T_b tokens into the other buffer;
                                       mamba_spec_commit then makes the other buffer the cache of every sequence with
                                       accept_len == k_draft (nothing is pending for it any more) and records accept_len
                                       as pending for the rest.  mamba_spec_get_selection tells where each cache is.   */
#define MAMBA_SPEC_FLAG_GATED_RMSNORM 128 /* the normalisation that closes a Mamba-2 block (the hybrid Mamba2 models of
                                       Sec. 5): every output row is scaled to unit mean square over its H*P channels and
                                       multiplied by a per-channel weight, after the gate,
                                         y_t[c] <- io->norm_weight[c] * g_t[c] / sqrt(mean_c(g_t[c]^2) + io->norm_eps),
                                       g the (gated) output.  The verification kernel writes g in float32 to scratch owned
                                       by the context (allocated on first use) and a second kernel forms y from it, so the
                                       output is rounded to the activation dtype once.  Not available without a context
                                       (mamba_spec_verify_host_static).                                                 */
#define MAMBA_SPEC_FLAG_CONV_BC 256 /* the conv of a Mamba-2 block runs over x, B and C together: the B and C rows pass through
                                       a depthwise causal conv of their own (channels: the G_B*N columns of B, then the
                                       G_C*N columns of C; taps io->conv_w_bc, bias io->conv_b_bc, rolling window
                                       io->conv_state_bc, cached at the verified position like conv_state) and the same
                                       activation as x before they enter the recurrence.  Generic kernel only (the
                                       streaming kernel refuses the flag); not with FLAG_STATE_K.  The conv's float32
                                       outputs live in scratch owned by the context.                                   */

/* bits of the device status word reported by mamba_spec_status */
#define MAMBA_SPEC_STATUS_NPREV_CLAMPED 1  /* some n_prev_accepted[b] was outside [0, min(k_max, t_max-k)] */
#define MAMBA_SPEC_STATUS_ACCEPT_CLAMPED 2 /* some accept_len[b] was outside [0, k_draft]                  */
#define MAMBA_SPEC_STATUS_COPY_TIMEOUT 4   /* a kernel gave up waiting for one of its own async copies     */

/* kernel_select */
#define MAMBA_SPEC_KERNEL_AUTO 0     /* streaming kernel when the shape allows, else the generic one */
#define MAMBA_SPEC_KERNEL_GENERIC 1  /* plain sequential-recurrence kernel, any supported shape      */
#define MAMBA_SPEC_KERNEL_STREAM 2   /* streaming kernel; fail with UNSUPPORTED rather than fall back */

typedef struct mamba_spec_ctx mamba_spec_ctx; /* opaque; created by init, freed by destroy */

typedef struct {
    int32_t batch_max;     /* largest batch any call will use, >= 1                               */
    int32_t n_layers;      /* number of Mamba layers sharing this context (bookkeeping only)      */
    int32_t n_heads;       /* H                                                                   */
    int32_t head_dim;      /* P, channels per head                                                */
    int32_t d_state;       /* N, state columns per channel; 1..256                                */
    int32_t n_groups_b;    /* G_B, divides H                                                      */
    int32_t n_groups_c;    /* G_C, divides H                                                      */
    int32_t conv_width;    /* W, 1..8                                                             */
    int32_t k_max;         /* largest k_draft (hence largest n_prev_accepted) of any call, 0..32  */
    int32_t act_dtype;     /* MAMBA_SPEC_DTYPE_*                                                  */
    int32_t flags;         /* MAMBA_SPEC_FLAG_*                                                   */
    int32_t device;        /* CUDA device ordinal                                                 */
    int32_t kernel_select; /* MAMBA_SPEC_KERNEL_*                                                 */
} mamba_spec_config;

typedef struct {
    const float *conv_w; /* [H*P][W]   depthwise taps, tap W-1 multiplies the current token        */
    const float *conv_b; /* [H*P]                                                                  */
    const void *z;       /* [batch][t_max][H][P] act dtype; gate input, may be null if not gated   */
    void *y;             /* [batch][t_max][H][P] act dtype (float32 with FLAG_Y_F32); output       */
    int32_t batch;       /* 1..batch_max                                                           */
    int32_t layer;       /* 0..n_layers-1                                                          */
    int32_t t_max;       /* row count of the token slabs; >= k_draft                               */
    void *stream;        /* cudaStream_t (null = default stream)                                   */
    void *state_k;       /* DEVICE [batch][H][P][N] float32, output, FLAG_STATE_K only: the state after all
                            T_b = j_b + k tokens of every sequence (a copy of the input where T_b = 0);
                            must not overlap state                                                  */
    void *conv_state_k;  /* DEVICE [batch][W-1][H*P] act dtype, output, FLAG_STATE_K only: the conv window
                            after all T_b tokens; must not overlap conv_state                       */
    const float *dt_bias; /* DEVICE [H] float32 ([H*P] with FLAG_MAMBA1), FLAG_DT_SOFTPLUS only; null = no bias */
    const float *norm_weight; /* DEVICE [H*P] float32, FLAG_GATED_RMSNORM only                                */
    float norm_eps;       /* FLAG_GATED_RMSNORM only: added to the mean square (>= 0)                                */
    void *conv_state_bc;  /* DEVICE [batch][W-1][(G_B+G_C)*N] act dtype, in/out, FLAG_CONV_BC only: the last W-1 B and C
                             rows at the cached position, oldest first                                            */
    const float *conv_w_bc; /* DEVICE [(G_B+G_C)*N][W] float32, FLAG_CONV_BC only; tap W-1 multiplies the current token    */
    const float *conv_b_bc; /* DEVICE [(G_B+G_C)*N] float32, FLAG_CONV_BC only                                            */
} mamba_spec_io;

/* HOST cfg, HOST out.  Validates the configuration, selects the device and
 * allocates the context.  Does not touch any caller tensor. */
int mamba_spec_init(const mamba_spec_config *cfg, mamba_spec_ctx **out);

/* The verification call described at the top of this file.  One kernel launch -- except that the streaming
 * kernel takes at most 16 token rows of a sequence, of which at most 8 pending, per launch: a longer block
 * (j_b + k_draft up to t_max) runs as several launches that carry the state from one to the next (Sec. 4.2: the
 * same recurrence, applied piecewise; scratch for the carried state is allocated on the first such call; not
 * combined with FLAG_COMMIT_SELECTS or FLAG_MAMBA1, which run such blocks in the generic kernel).
 *   state           [batch][H][P][N] float32, in/out: h_i -> h_{i+j_b}
 *   conv_state      [batch][W-1][H*P] act dtype, in/out, oldest row first
 *   x               [batch][t_max][H][P] act dtype, pre-conv inputs
 *   dt              [batch][t_max][H]    act dtype, already positive (post-softplus) unless FLAG_DT_SOFTPLUS;
 *                   [batch][t_max][H*P] with FLAG_MAMBA1
 *   B               [batch][t_max][G_B][N] act dtype
 *   C               [batch][t_max][G_C][N] act dtype
 *   A               [H] float32, negative reals          D  [H] float32
 *                   ([H*P][N] and [H*P] with FLAG_MAMBA1)
 *   n_prev_accepted [batch] int32, or null to use what the last mamba_spec_commit recorded
 *                   (zeros before any commit).  Values outside [0, min(k_max, t_max-k_draft)]
 *                   are clamped on the device and flagged in the status word.
 *   k_draft         0..k_max; 0 is a pure advance (flush) over the pending accepted tokens
 *   io              HOST struct, read during the call only
 * x/z/dt/B/C/y must not alias state or conv_state. */
int mamba_spec_verify(mamba_spec_ctx *ctx, void *state, void *conv_state, const void *x, const void *dt,
                      const void *B, const void *C, const float *A, const float *D,
                      const int32_t *n_prev_accepted, int32_t k_draft, const mamba_spec_io *io);

/* Algorithm 2's "j <- k'": records accept_len[b] (device, [batch], each in
 * [0, k_draft of the last verify]) as the next call's n_prev_accepted.  Moves no
 * state: the cache advances lazily, as the replay prefix of the next verify.
 * With FLAG_COMMIT_SELECTS a fully accepted sequence switches to the buffer that
 * holds h_k instead and has nothing pending (see the flag). */
int mamba_spec_commit(mamba_spec_ctx *ctx, const int32_t *accept_len, int32_t batch, void *stream);

/* The verification call for a caller that hands over only the k_draft NEW rows of every sequence (Sec. 4.2:
 * "caching older entries"; Sec. 4.3, footnote: a circular buffer keeps old entries available for
 * recomputation).  The context keeps, per layer, the rows of the last call: the tokens accepted since -- the
 * first n_prev_accepted[b] of them, as recorded by mamba_spec_commit -- are replayed from there, so
 *   x_new, io->z   [batch][k_draft][H][P]      dt_new  [batch][k_draft][H]  ([..][H*P] with FLAG_MAMBA1)
 *   B_new          [batch][k_draft][G_B][N]    C_new   [batch][k_draft][G_C][N]
 *   io->y          [batch][k_draft][H][P], output: the rows of the new tokens only (the replayed rows'
 *                  outputs went out in the last call); io->t_max is ignored
 * state, conv_state, A, D, io->conv_w/conv_b/state_k/conv_state_k/dt_bias as in mamba_spec_verify.
 * One extra kernel lays the replayed and the new rows out for the verification kernel and keeps the new rows
 * for the next call; the row store (n_layers x batch_max x k_max rows per tensor) is allocated on the first
 * call.  The pending lengths are the context's (mamba_spec_commit); k_draft = 0 flushes them. */
int mamba_spec_verify_new(mamba_spec_ctx *ctx, void *state, void *conv_state, const void *x_new, const void *dt_new,
                          const void *B_new, const void *C_new, const float *A, const float *D, int32_t k_draft,
                          const mamba_spec_io *io);

/* Same computation with the per-step tensors in HOST memory (pinned memory
 * makes the copies asynchronous): x, dt, B, C, n_prev_accepted (nullable), io->z
 * are copied to context-owned device staging on io->stream, the kernel runs,
 * and y is copied back to io->y (HOST).  state, conv_state, A, D, io->conv_w,
 * io->conv_b stay DEVICE pointers.  The call returns after enqueueing; read y
 * after synchronising the stream.  The whole [batch][t_max] slab of y is copied
 * back, so rows t >= T_b of the host y hold unspecified values afterwards.
 * Staging is sized for batch_max x max(1, 2*k_max) rows: io->t_max must not exceed that. */
int mamba_spec_verify_host(mamba_spec_ctx *ctx, void *state, void *conv_state, const void *x_host,
                           const void *dt_host, const void *B_host, const void *C_host, const float *A,
                           const float *D, const int32_t *n_prev_accepted_host, int32_t k_draft,
                           const mamba_spec_io *io);

/* The same computation as mamba_spec_verify_host for callers that must not allocate device memory:
 * code running where cudaMalloc is off limits (inside a host callback or a latency-critical serving
 * loop, in a process whose memory is fully pre-reserved by another allocator, or after the device has
 * been handed over with no free memory left).  The paper has no counterpart; this is a convenience of
 * this library.  It needs no context: the device staging that mamba_spec_verify_host allocates lives
 * here in an 8 MiB array built into the library (every GPU that loads the library holds it until the
 * process exits), and the call itself makes no cudaMalloc/cudaFree or other allocating call.
 *   cfg        HOST, same meaning and rules as for mamba_spec_init (n_layers/batch_max only bound io)
 *   state, conv_state, A, D, io->conv_w, io->conv_b   DEVICE, as in mamba_spec_verify
 *   x_host, dt_host, B_host, C_host, io->z, io->y     HOST ([batch][t_max] slabs; pinned memory keeps
 *              the copies asynchronous); the whole y slab is copied back
 *   n_prev_accepted_host   HOST [batch], required (there is no context to remember a commit)
 *   device_flags_host      HOST, nullable: receives the MAMBA_SPEC_STATUS_* word of this call
 * Everything is enqueued on io->stream; read y and the flags after synchronising it.
 * Limits and caveats: a call whose slabs (x, z, dt, B, C, y and batch int32) exceed 8 MiB of staging is
 * refused with MAMBA_SPEC_ERR_UNSUPPORTED.  All calls on a device share the one array, which keeps the
 * previous call's contents (the status word is cleared by every call): two calls that overlap on the
 * GPU -- different streams, or a second call enqueued before the first has finished on another stream --
 * race on it.  The first call on each device looks up the array's device address; make that first
 * call before any stream capture.  Not safe to call from several host threads for the first time at once.
 * On failure the message is available from mamba_spec_last_error(NULL). */
int mamba_spec_verify_host_static(const mamba_spec_config *cfg, void *state, void *conv_state, const void *x_host,
                                  const void *dt_host, const void *B_host, const void *C_host, const float *A,
                                  const float *D, const int32_t *n_prev_accepted_host, int32_t k_draft,
                                  const mamba_spec_io *io, int32_t *device_flags_host);

/* Synchronises the context's last stream, returns the device status word in
 * *device_flags_out (HOST) and clears it. */
int mamba_spec_status(mamba_spec_ctx *ctx, int32_t *device_flags_out);

/* Copies the pending n_prev (what the next verify with a null n_prev_accepted
 * would use) to HOST memory; with state and conv_state this is a complete
 * checkpoint of a layer stack.  Synchronises. */
int mamba_spec_get_n_prev(mamba_spec_ctx *ctx, int32_t *n_prev_host, int32_t batch);

/* FLAG_COMMIT_SELECTS: copies to HOST memory, for each of the first `batch` sequences, 0 if its cache is in
 * (state, conv_state) and 1 if it is in (io->state_k, io->conv_state_k).  The same for every layer that
 * shares the context, since all layers see the same commits.  Synchronises. */
int mamba_spec_get_selection(mamba_spec_ctx *ctx, int32_t *sel_host, int32_t batch);

/* Which kernel a verify call of this shape would run, and with which launch plan, as text in buf (HOST,
 * buf_len bytes): "stream<...>" with the streaming kernel's ring depths, groups and grid, or "generic (reason)".
 * Host logic only: no tensor is touched and no kernel launched.  sm_count / smem_per_block describe the GPU
 * (multiprocessors, opt-in shared memory per block in bytes); pass 0 for both to ask the CUDA device cfg names. */
int mamba_spec_describe_plan(const mamba_spec_config *cfg, int32_t batch, int32_t t_max, int32_t k_draft,
                             int32_t sm_count, int64_t smem_per_block, char *buf, int32_t buf_len);

/* Number of kernels this context has launched so far (HOST counter). */
int64_t mamba_spec_launch_count(const mamba_spec_ctx *ctx);

/* Name of the kernel the last verify launched ("generic", "stream<...>"), HOST string owned by ctx. */
const char *mamba_spec_last_kernel(const mamba_spec_ctx *ctx);

/* Message of the last error on this context (or of the last failed init when ctx is null). */
const char *mamba_spec_last_error(const mamba_spec_ctx *ctx);

void mamba_spec_destroy(mamba_spec_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MAMBA_SPEC_H */
