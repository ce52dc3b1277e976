// Host side of the mamba_spec C ABI: argument validation, kernel selection and
// launch.  Every step of the verification call runs in the kernels; this file
// only checks, plans and enqueues.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/mamba_spec.h"
#include "common.cuh"

using namespace mspec;

// Encoded tensor maps of the streaming kernel, kept per context: a decode loop calls with the same
// buffers round after round, and encoding eight maps costs more host time than the launch itself.
// A map depends only on addresses and shapes, so an entry stays valid for as long as its key matches.
struct MapKey {
    const void *state, *conv_state, *x, *dt, *B, *C, *z, *state_k, *conv_state_k;
    int32_t batch, t_max, tcap, variant;
    bool operator==(const MapKey &o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapEntry {
    bool used = false;
    MapKey key;
    InputMaps maps;
};
constexpr size_t kMapCacheEntries = 512;   // direct-mapped

struct mamba_spec_ctx {
    mamba_spec_config cfg;
    int sm_count = 0;
    size_t smem_per_sm = 0, smem_optin = 0;
    int32_t *d_n_prev = nullptr;  // [batch_max] pending n_prev recorded by commit
    int32_t *d_status = nullptr;  // one word
    int32_t *d_sel = nullptr;     // [batch_max] which buffer holds each sequence's cache (FLAG_COMMIT_SELECTS)
    // device staging for mamba_spec_verify_host, allocated on its first use
    void *st_x = nullptr, *st_dt = nullptr, *st_B = nullptr, *st_C = nullptr, *st_z = nullptr, *st_y = nullptr;
    int32_t *st_n_prev = nullptr;
    bool staging_ready = false;
    // row store of mamba_spec_verify_new: per tensor (x, z, dt, B, C) the last call's new rows of every layer
    // [n_layers][batch_max][k_max][row], and one set of slabs [batch_max][2 k_max][row] that the kernels read
    void *ring[5] = {nullptr, nullptr, nullptr, nullptr, nullptr}, *slab[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    bool ring_ready = false;
    // token blocks of more than 16 rows go through the streaming kernel in segments: the state between two
    // segments lives here (two of each, used in turn), plus a vector of zeros (nothing pending after the first)
    float *split_state[2] = {nullptr, nullptr};
    void *split_conv[2] = {nullptr, nullptr};
    int32_t *d_zero = nullptr;
    // FLAG_GATED_RMSNORM: the verification kernel's float32 output rows, read by the normalising kernel; the weight
    // and eps of the call in progress
    float *norm_scratch = nullptr;
    size_t norm_scratch_bytes = 0;
    const float *norm_w = nullptr;
    float norm_eps = 0.f;
    // FLAG_CONV_BC: the float32 outputs of the conv over the B and C rows, and the call's window, taps and bias
    float *bc_scratch = nullptr;
    size_t bc_scratch_bytes = 0;
    ConvBC bc = {nullptr, nullptr, nullptr, nullptr};
    cudaStream_t last_stream = nullptr;
    int32_t last_k = -1;
    int64_t launches = 0;
    std::vector<MapEntry> map_cache;   // empty for contexts that must not allocate
    std::string err;
    char last_kernel[112] = "none";
};

constexpr int kAllFlags = MAMBA_SPEC_FLAG_GATE | MAMBA_SPEC_FLAG_CONV_SILU | MAMBA_SPEC_FLAG_Y_F32 | MAMBA_SPEC_FLAG_STATE_K |
                          MAMBA_SPEC_FLAG_MAMBA1 | MAMBA_SPEC_FLAG_DT_SOFTPLUS | MAMBA_SPEC_FLAG_COMMIT_SELECTS |
                          MAMBA_SPEC_FLAG_GATED_RMSNORM | MAMBA_SPEC_FLAG_CONV_BC;

static thread_local std::string g_init_error;

static int fail(mamba_spec_ctx *ctx, int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (ctx) ctx->err = buf; else g_init_error = buf;
    return code;
}

#define CUDA_TRY(ctx, call)                                                                          \
    do {                                                                                             \
        cudaError_t e_ = (call);                                                                     \
        if (e_ != cudaSuccess)                                                                       \
            return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));  \
    } while (0)

// ---- staging for mamba_spec_verify_host_static: device memory that exists without any allocation call.
// Every GPU that loads this library carries the array until the process exits.
constexpr size_t kStaticStagingBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_staging[kStaticStagingBytes];

struct StaticDevice {   // per device, filled on the first call there
    bool ready = false;
    unsigned char *base = nullptr;   // device address of g_static_staging on that device
    int sm_count = 0;
    size_t smem_per_sm = 0, smem_optin = 0;
};
static StaticDevice g_static_dev[64];

static size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }


namespace {

// Makes ctx's device current for the duration of a call and restores the caller's.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t act_bytes(const mamba_spec_config &c) { return c.act_dtype == MAMBA_SPEC_DTYPE_BF16 ? 2 : 4; }

// Lays out the token rows of one verify_new call for one tensor: slab[b][t] = the row kept from the last
// call for t < j_b (a token accepted since), then the k new rows; the new rows are kept for the next call.
// One thread per (sequence, piece of a row); U is the widest unit that divides a row.
template <typename U>
__global__ void assemble_rows_kernel(U *slab, U *ring, const U *fresh, const int32_t *n_prev, int batch, int k, int k_max,
                                     int slab_rows, int units, int j_cap) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)batch * units) return;
    const int b = (int)(i / units), u = (int)(i % units);
    int j = n_prev[b];
    j = j < 0 ? 0 : (j > j_cap ? j_cap : j);   // (the verification kernel clamps the same way and flags it)
    U *srow = slab + (size_t)b * slab_rows * units + u, *rrow = ring + (size_t)b * k_max * units + u;
    for (int t = 0; t < j; ++t) srow[(size_t)t * units] = rrow[(size_t)t * units];
    for (int t = 0; t < k; ++t) {
        const U v = fresh[((size_t)b * k + t) * units + u];
        srow[(size_t)(j + t) * units] = v;
        rrow[(size_t)t * units] = v;
    }
}

// Algorithm 2's choice of the state to keep: with `sel` a fully accepted sequence takes the buffer that holds
// the state after all tokens (h_k) and has nothing pending; every other sequence keeps h_j and replays.
__global__ void commit_kernel(int32_t *n_prev, const int32_t *accept_len, int batch, int k, int32_t *status, int32_t *sel) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    int a = accept_len[b];
    if (a < 0 || a > k) {
        atomicOr(status, kStatusAcceptClamped);
        a = a < 0 ? 0 : k;
    }
    if (sel != nullptr && a == k) {
        sel[b] ^= 1;
        a = 0;
    }
    n_prev[b] = a;
}

// The normalisation that closes a Mamba-2 block, on the float32 rows g the verification kernel left in scratch:
// y[c] = w[c] g[c] / sqrt(mean_c g[c]^2 + eps) over the C = H*P channels of a token.  One block per token row; rows
// beyond a sequence's T_b tokens are left alone.
template <typename out_t>
__global__ void __launch_bounds__(256) gated_rmsnorm_kernel(out_t *y, const float *g, const float *w, float eps, const int32_t *n_prev,
                                                            int j_cap, int k, int rows_per_seq, int C, int new_only) {
    const int row = blockIdx.x, b = row / rows_per_seq, t = row % rows_per_seq;
    int T = k;
    if (!new_only) {
        const int j = n_prev[b];
        T += j < 0 ? 0 : (j > j_cap ? j_cap : j);
    }
    if (t >= T) return;
    const float *gr = g + (size_t)row * C;
    float ss = 0.f;
    for (int c = threadIdx.x; c < C; c += blockDim.x) ss = fmaf(gr[c], gr[c], ss);
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
    __shared__ float part[8];
    __shared__ float scale;
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += part[i];
        scale = 1.0f / sqrtf(tot / (float)C + eps);
    }
    __syncthreads();
    const float r = scale;
    out_t *yr = y + (size_t)row * C;
    for (int c = threadIdx.x; c < C; c += blockDim.x) st_act(yr, c, w[c] * gr[c] * r);
}

}  // namespace

// the library is built with hidden visibility; only the C ABI below is exported
#pragma GCC visibility push(default)
extern "C" {

int mamba_spec_init(const mamba_spec_config *cfg, mamba_spec_ctx **out) {
    if (!cfg || !out) return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: null cfg or out");
    *out = nullptr;
    const mamba_spec_config &c = *cfg;
    if (c.batch_max < 1 || c.n_layers < 1 || c.n_heads < 1 || c.head_dim < 1 || c.d_state < 1)
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: batch_max, n_layers, n_heads, head_dim, d_state must be >= 1");
    if (c.d_state > kMaxStateDim)
        return fail(nullptr, MAMBA_SPEC_ERR_UNSUPPORTED, "init: d_state %d > %d", c.d_state, kMaxStateDim);
    if (c.conv_width < 1 || c.conv_width > kMaxConvWidth)
        return fail(nullptr, MAMBA_SPEC_ERR_UNSUPPORTED, "init: conv_width %d outside 1..%d", c.conv_width, kMaxConvWidth);
    if (c.n_groups_b < 1 || c.n_groups_c < 1 || c.n_heads % c.n_groups_b || c.n_heads % c.n_groups_c)
        return fail(nullptr, MAMBA_SPEC_ERR_BAD_SHAPE, "init: group counts (%d, %d) must divide n_heads %d",
                    c.n_groups_b, c.n_groups_c, c.n_heads);
    if (c.k_max < 0 || c.k_max > 32) return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: k_max %d outside 0..32", c.k_max);
    if (c.act_dtype != MAMBA_SPEC_DTYPE_F32 && c.act_dtype != MAMBA_SPEC_DTYPE_BF16)
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: unknown act_dtype %d", c.act_dtype);
    if (c.flags & ~(kAllFlags))
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: unknown flag bits 0x%x", c.flags);
    if (c.kernel_select < 0 || c.kernel_select > MAMBA_SPEC_KERNEL_STREAM)
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: unknown kernel_select %d", c.kernel_select);
    if ((c.flags & MAMBA_SPEC_FLAG_COMMIT_SELECTS) && !(c.flags & MAMBA_SPEC_FLAG_STATE_K))
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: FLAG_COMMIT_SELECTS needs FLAG_STATE_K");
    if ((c.flags & MAMBA_SPEC_FLAG_CONV_BC) && (c.flags & MAMBA_SPEC_FLAG_STATE_K))
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: FLAG_CONV_BC keeps one window of B and C rows: not with FLAG_STATE_K");
    if ((c.flags & MAMBA_SPEC_FLAG_CONV_BC) && c.kernel_select == MAMBA_SPEC_KERNEL_STREAM)
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: FLAG_CONV_BC runs in the generic kernel");
    // conv_state rows and token rows must keep 16-byte alignment per (sequence, row)
    if ((size_t)c.n_heads * c.head_dim * act_bytes(c) % 16)
        return fail(nullptr, MAMBA_SPEC_ERR_BAD_SHAPE, "init: H*P*sizeof(act) must be a multiple of 16 bytes");

    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess || ndev < 1)
        return fail(nullptr, MAMBA_SPEC_ERR_CUDA, "init: no CUDA device (%s); this library has no CPU path",
                    e == cudaSuccess ? "device count 0" : cudaGetErrorString(e));
    if (c.device < 0 || c.device >= ndev)
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: device %d outside 0..%d", c.device, ndev - 1);

    DeviceGuard guard(c.device);
    if (!guard.ok) return fail(nullptr, MAMBA_SPEC_ERR_CUDA, "init: cannot select device %d", c.device);
    mamba_spec_ctx *ctx = new (std::nothrow) mamba_spec_ctx();
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "init: out of host memory");
    ctx->cfg = c;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, c.device);
    if (e == cudaSuccess) {
        ctx->sm_count = prop.multiProcessorCount;
        ctx->smem_per_sm = prop.sharedMemPerMultiprocessor;
        ctx->smem_optin = prop.sharedMemPerBlockOptin;
        e = cudaMalloc(&ctx->d_n_prev, sizeof(int32_t) * (size_t)c.batch_max);
    }
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_sel, sizeof(int32_t) * (size_t)c.batch_max);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_sel, 0, sizeof(int32_t) * (size_t)c.batch_max);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_n_prev, 0, sizeof(int32_t) * (size_t)c.batch_max);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(int32_t));
    if (e != cudaSuccess) {
        cudaFree(ctx->d_n_prev);
        cudaFree(ctx->d_status);
        cudaFree(ctx->d_sel);
        delete ctx;
        return fail(nullptr, MAMBA_SPEC_ERR_CUDA, "init: %s", cudaGetErrorString(e));
    }
    ctx->map_cache.resize(kMapCacheEntries);
    *out = ctx;
    return MAMBA_SPEC_OK;
}

static int check_and_fill(mamba_spec_ctx *ctx, VerifyParams &p, void *state, void *conv_state, const void *x,
                          const void *dt, const void *B, const void *C, const float *A, const float *D,
                          const int32_t *n_prev, int32_t k_draft, const mamba_spec_io *io, const char *who) {
    const mamba_spec_config &c = ctx->cfg;
    if (!io) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: io is null", who);
    if (!state || !x || !dt || !B || !C || !A || !D || !io->conv_w || !io->conv_b || !io->y)
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: a required tensor pointer is null", who);
    if (c.conv_width > 1 && !conv_state) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: conv_state is null", who);
    if ((c.flags & MAMBA_SPEC_FLAG_GATE) && !io->z)
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: gating is on but io->z is null", who);
    if (io->batch < 1 || io->batch > c.batch_max)
        return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "%s: batch %d outside 1..%d", who, io->batch, c.batch_max);
    if (io->layer < 0 || io->layer >= c.n_layers)
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: layer %d outside 0..%d", who, io->layer, c.n_layers - 1);
    if (k_draft < 0 || k_draft > c.k_max)
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: k_draft %d outside 0..%d", who, k_draft, c.k_max);
    if (io->t_max < 1 || io->t_max < k_draft)
        return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "%s: t_max %d < max(1, k_draft %d)", who, io->t_max, k_draft);
    if ((c.flags & MAMBA_SPEC_FLAG_STATE_K) && (!io->state_k || !io->conv_state_k))
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: FLAG_STATE_K needs io->state_k and io->conv_state_k", who);
    if ((c.flags & MAMBA_SPEC_FLAG_STATE_K) && (io->state_k == state || io->conv_state_k == conv_state))
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: the second snapshot must not alias the cache", who);
    if (c.flags & MAMBA_SPEC_FLAG_GATED_RMSNORM) {
        if (!io->norm_weight || !aligned16(io->norm_weight))
            return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: FLAG_GATED_RMSNORM needs io->norm_weight (16-byte aligned)", who);
        if (!(io->norm_eps >= 0.f) || io->norm_eps > 3.0e38f)
            return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: io->norm_eps must be a finite number >= 0", who);
        ctx->norm_w = io->norm_weight;
        ctx->norm_eps = io->norm_eps;
    }
    if (c.flags & MAMBA_SPEC_FLAG_CONV_BC) {
        if (!io->conv_w_bc || !io->conv_b_bc || (c.conv_width > 1 && !io->conv_state_bc))
            return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "%s: FLAG_CONV_BC needs io->conv_state_bc, io->conv_w_bc and io->conv_b_bc", who);
        if (!aligned16(io->conv_w_bc) || !aligned16(io->conv_b_bc) || !aligned16(io->conv_state_bc))
            return fail(ctx, MAMBA_SPEC_ERR_MISALIGNED, "%s: a tensor of the conv over B and C is not 16-byte aligned", who);
        ctx->bc.window = io->conv_state_bc;
        ctx->bc.taps = io->conv_w_bc;
        ctx->bc.bias = io->conv_b_bc;
    }
    const void *ptrs[] = {state, conv_state, x, dt, B, C, A, D, io->conv_w, io->conv_b, io->z, io->y,
                          (c.flags & MAMBA_SPEC_FLAG_DT_SOFTPLUS) ? (const void *)io->dt_bias : nullptr,
                          (c.flags & MAMBA_SPEC_FLAG_STATE_K) ? io->state_k : nullptr,
                          (c.flags & MAMBA_SPEC_FLAG_STATE_K) ? io->conv_state_k : nullptr};
    for (const void *q : ptrs)
        if (q && !aligned16(q)) return fail(ctx, MAMBA_SPEC_ERR_MISALIGNED, "%s: tensor pointer %p is not 16-byte aligned", who, q);
    p.state = (float *)state;
    p.conv_state = conv_state;
    p.x = x; p.dt = dt; p.B = B; p.C = C; p.z = (c.flags & MAMBA_SPEC_FLAG_GATE) ? io->z : nullptr; p.y = io->y;
    p.A = A; p.D = D; p.conv_w = io->conv_w; p.conv_b = io->conv_b;
    p.row_off = nullptr; p.row_off_const = 0; p.row_off_cap = 0; p.n_prev_done = 0; p.n_prev_full = 0;
    p.dt_bias = (c.flags & MAMBA_SPEC_FLAG_DT_SOFTPLUS) ? io->dt_bias : nullptr;
    p.sel = (c.flags & MAMBA_SPEC_FLAG_COMMIT_SELECTS) ? ctx->d_sel : nullptr;
    p.state_k = (c.flags & MAMBA_SPEC_FLAG_STATE_K) ? (float *)io->state_k : nullptr;
    p.conv_state_k = (c.flags & MAMBA_SPEC_FLAG_STATE_K) ? io->conv_state_k : nullptr;
    p.n_prev = n_prev ? n_prev : ctx->d_n_prev;
    p.status = ctx->d_status;
    p.batch = io->batch; p.t_max = io->t_max; p.H = c.n_heads; p.P = c.head_dim; p.N = c.d_state;
    p.GB = c.n_groups_b; p.GC = c.n_groups_c; p.W = c.conv_width; p.k = k_draft;
    p.j_cap = c.k_max < io->t_max - k_draft ? c.k_max : io->t_max - k_draft;
    p.flags = c.flags;
    return MAMBA_SPEC_OK;
}

static int launch_one(mamba_spec_ctx *ctx, const VerifyParams &p, cudaStream_t stream, const char *who);

// A token block of more than 16 rows, for the streaming kernel: segments of at most 16 rows, one launch each.
// The first takes the pending tokens and as many drafts as fit, puts the state at the verified position back
// into the cache (Sec. 4.3 iii) and leaves the state after its last token in a scratch buffer, from which the
// next segment goes on with nothing pending, and so on; only the last writes a second snapshot if the caller
// wants one.  (The same unrolled form, applied segment by segment; the per-token states still never exist.)
static int launch_split(mamba_spec_ctx *ctx, const VerifyParams &p, cudaStream_t stream, const char *who) {
    const mamba_spec_config &c = ctx->cfg;
    const size_t n_state = (size_t)c.batch_max * c.n_heads * c.head_dim * c.d_state * sizeof(float);
    const size_t n_conv = (size_t)c.batch_max * (c.conv_width - 1) * c.n_heads * c.head_dim * act_bytes(c);
    if (!ctx->d_zero) {   // all or nothing
        cudaError_t e = cudaSuccess;
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaMalloc(&ctx->split_state[i], n_state);
            if (e == cudaSuccess) e = cudaMalloc(&ctx->split_conv[i], n_conv + 16);
        }
        int32_t *zero = nullptr;
        if (e == cudaSuccess) e = cudaMalloc(&zero, sizeof(int32_t) * (size_t)c.batch_max);
        if (e == cudaSuccess) e = cudaMemset(zero, 0, sizeof(int32_t) * (size_t)c.batch_max);
        if (e != cudaSuccess) {
            for (int i = 0; i < 2; ++i) {
                if (ctx->split_state[i]) cudaFree(ctx->split_state[i]);
                if (ctx->split_conv[i]) cudaFree(ctx->split_conv[i]);
                ctx->split_state[i] = nullptr;
                ctx->split_conv[i] = nullptr;
            }
            if (zero) cudaFree(zero);
            return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: scratch for a split token block: %s", who, cudaGetErrorString(e));
        }
        ctx->d_zero = zero;
    }
    const int kSeg = 16;
    int done = 0, seg = 0;
    const int k_first = kSeg - p.j_cap < p.k ? kSeg - p.j_cap : p.k;
    while (done < p.k || seg == 0) {
        const int k_i = seg == 0 ? k_first : (p.k - done < kSeg ? p.k - done : kSeg);
        const bool last = done + k_i >= p.k;
        VerifyParams q = p;
        q.k = k_i;
        if (seg > 0) {
            q.state = ctx->split_state[(seg - 1) & 1];
            q.conv_state = ctx->split_conv[(seg - 1) & 1];
            q.n_prev = ctx->d_zero;
            q.j_cap = 0;
            q.n_prev_done = 0;
            q.n_prev_full = 0;
            q.row_off = p.n_prev;
            q.row_off_cap = p.row_off_cap + p.j_cap;   // all of this sequence's pending rows come first
            q.row_off_const = done;
        }
        if (!last) {
            q.state_k = ctx->split_state[seg & 1];
            q.conv_state_k = ctx->split_conv[seg & 1];
        }
        const int rc = launch_one(ctx, q, stream, who);
        if (rc) return rc;
        done += k_i;
        ++seg;
    }
    return MAMBA_SPEC_OK;
}

// How a call is launched: as one kernel, or -- a token block of more than 16 rows, where the streaming kernel would
// take its pieces -- as `pending_only` launches that replay 8 pending rows each and then the rest in pieces of at
// most 16 rows (launch_split).
struct SplitPlan {
    bool split;
    int pending_only;     // launches without drafts that advance the cache over 8 pending rows each
    int launches;         // all launches of the call
    VerifyParams rest;    // the call that is left after them
    StreamPlan first;     // plan of the first launch that takes drafts
};
static const int kSegRows = 16, kSegPending = 8;   // rows and pending rows that one launch of the streaming kernel takes

static SplitPlan plan_split(const VerifyParams &p, const mamba_spec_config &c, int sm_count, size_t smem_optin) {
    SplitPlan sp;
    sp.split = false; sp.pending_only = 0; sp.launches = 1; sp.rest = p;
    if (p.j_cap + p.k <= kSegRows || c.kernel_select == MAMBA_SPEC_KERNEL_GENERIC || p.sel != nullptr ||
        (p.flags & (kFlagYNewOnly | kFlagMamba1)))
        return sp;
    const bool bf16 = c.act_dtype == MAMBA_SPEC_DTYPE_BF16;
    const int n_flush = p.j_cap > kSegPending ? (p.j_cap - 1) / kSegPending : 0;
    VerifyParams rest = p;
    if (n_flush > 0) {
        rest.n_prev_full = p.j_cap;
        rest.n_prev_done = kSegPending * n_flush;
        rest.j_cap = p.j_cap - kSegPending * n_flush;
        rest.row_off = p.n_prev;
        rest.row_off_cap = kSegPending * n_flush;
    }
    VerifyParams probe = rest;
    probe.k = rest.j_cap + p.k > kSegRows ? kSegRows - rest.j_cap : p.k;
    VerifyParams probe_flush = p;
    probe_flush.j_cap = kSegPending; probe_flush.k = 0; probe_flush.state_k = nullptr; probe_flush.conv_state_k = nullptr;
    sp.first = plan_verify_stream(probe, bf16, sm_count, smem_optin);
    if (!sp.first.ok || (n_flush > 0 && !plan_verify_stream(probe_flush, bf16, sm_count, smem_optin).ok)) return sp;
    sp.split = true;
    sp.pending_only = n_flush;
    sp.rest = rest;
    const int k_first = kSegRows - rest.j_cap < rest.k ? kSegRows - rest.j_cap : rest.k;
    sp.launches = n_flush + 1 + (rest.k - k_first + kSegRows - 1) / kSegRows;
    return sp;
}

static int launch_blocks(mamba_spec_ctx *ctx, const VerifyParams &p, cudaStream_t stream, const char *who) {
    if (ctx->map_cache.size() > 0) {   // (a context that may allocate: the carried state needs scratch)
        const SplitPlan sp = plan_split(p, ctx->cfg, ctx->sm_count, ctx->smem_optin);
        if (sp.split) {
            // more than 8 pending rows: the first ones are replayed 8 at a time, each launch advancing the cache
            // in place (a call with no drafts), until at most 8 are left for the launch that takes the drafts
            for (int i = 0; i < sp.pending_only; ++i) {
                VerifyParams q = p;
                q.j_cap = kSegPending; q.k = 0; q.state_k = nullptr; q.conv_state_k = nullptr;
                q.n_prev_full = p.j_cap;
                q.n_prev_done = kSegPending * i;
                q.row_off = p.n_prev;
                q.row_off_cap = kSegPending * i;
                const int rc = launch_one(ctx, q, stream, who);
                if (rc) return rc;
            }
            return sp.rest.j_cap + sp.rest.k > kSegRows ? launch_split(ctx, sp.rest, stream, who) : launch_one(ctx, sp.rest, stream, who);
        }
    }
    return launch_one(ctx, p, stream, who);
}

// The whole call: the verification launches and, with FLAG_GATED_RMSNORM, the normalising kernel after them (the
// verification kernel then writes its output rows in float32 to the context's scratch).
static int launch(mamba_spec_ctx *ctx, const VerifyParams &p, cudaStream_t stream, const char *who) {
    if (!(p.flags & kFlagGatedRmsnorm)) return launch_blocks(ctx, p, stream, who);
    const bool new_only = (p.flags & kFlagYNewOnly) != 0;
    const int rows_per_seq = new_only ? p.k : p.t_max, C = p.H * p.P;
    if (rows_per_seq < 1) return launch_blocks(ctx, p, stream, who);   // no output rows at all
    const size_t need = (size_t)p.batch * rows_per_seq * C * sizeof(float);
    if (ctx->norm_scratch_bytes < need) {
        if (ctx->norm_scratch) cudaFree(ctx->norm_scratch);   // (synchronises: no launch still uses it)
        ctx->norm_scratch = nullptr;
        ctx->norm_scratch_bytes = 0;
        const cudaError_t e = cudaMalloc(&ctx->norm_scratch, need);
        if (e != cudaSuccess) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: scratch for the normalised output: %s", who, cudaGetErrorString(e));
        ctx->norm_scratch_bytes = need;
    }
    VerifyParams q = p;
    q.y = ctx->norm_scratch;
    q.flags |= kFlagYF32;
    const int rc = launch_blocks(ctx, q, stream, who);
    if (rc) return rc;
    const long long blocks = (long long)p.batch * rows_per_seq;
    if (blocks > 0x7fffffffLL) return fail(ctx, MAMBA_SPEC_ERR_UNSUPPORTED, "%s: too many output rows for the normalising kernel", who);
    const bool out_f32 = (p.flags & kFlagYF32) != 0 || ctx->cfg.act_dtype != MAMBA_SPEC_DTYPE_BF16;
    if (out_f32)
        gated_rmsnorm_kernel<float><<<(unsigned)blocks, 256, 0, stream>>>((float *)p.y, ctx->norm_scratch, ctx->norm_w, ctx->norm_eps, p.n_prev,
                                                                           p.j_cap, p.k, rows_per_seq, C, new_only ? 1 : 0);
    else
        gated_rmsnorm_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, stream>>>((__nv_bfloat16 *)p.y, ctx->norm_scratch, ctx->norm_w, ctx->norm_eps,
                                                                                   p.n_prev, p.j_cap, p.k, rows_per_seq, C, new_only ? 1 : 0);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: normalising kernel: %s", who, cudaGetErrorString(e));
    ctx->launches++;
    return MAMBA_SPEC_OK;
}

static int launch_one(mamba_spec_ctx *ctx, const VerifyParams &p, cudaStream_t stream, const char *who) {
    const mamba_spec_config &c = ctx->cfg;
    const bool bf16 = c.act_dtype == MAMBA_SPEC_DTYPE_BF16;
    cudaError_t e;
    if (c.kernel_select == MAMBA_SPEC_KERNEL_AUTO || c.kernel_select == MAMBA_SPEC_KERNEL_STREAM) {
        StreamPlan plan = plan_verify_stream(p, bf16, ctx->sm_count, ctx->smem_optin);
        if (plan.ok) {
            InputMaps fresh;
            const InputMaps *maps = &fresh;
            MapKey key;
            memset(&key, 0, sizeof key);
            key.state = p.state; key.conv_state = p.conv_state; key.x = p.x; key.dt = p.dt; key.B = p.B; key.C = p.C;
            key.z = p.z; key.state_k = p.state_k; key.conv_state_k = p.conv_state_k; key.batch = p.batch; key.t_max = p.t_max; key.tcap = plan.layout.TCAP;
            key.variant = plan.variant;
            MapEntry *slot = nullptr;
            if (!ctx->map_cache.empty()) {
                const uintptr_t hsh = (reinterpret_cast<uintptr_t>(p.x) >> 8) * 0x9E3779B97F4A7C15ull ^
                                      (reinterpret_cast<uintptr_t>(p.state) >> 8) * 0xC2B2AE3D27D4EB4Full;
                slot = &ctx->map_cache[(hsh >> 20) % ctx->map_cache.size()];
            }
            if (slot && slot->used && slot->key == key) {
                maps = &slot->maps;
            } else {
                InputMaps *dst = slot ? &slot->maps : &fresh;
                if (slot) slot->used = false;
                if (!encode_stream_maps(p, plan, dst))
                    return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: the driver refused a tensor map for this shape", who);
                if (slot) { slot->key = key; slot->used = true; }
                maps = dst;
            }
            e = launch_verify_stream(p, plan, *maps, stream);
            if (e != cudaSuccess) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: stream launch: %s", who, cudaGetErrorString(e));
            memcpy(ctx->last_kernel, plan.name, sizeof ctx->last_kernel);
            ctx->launches++;
            return MAMBA_SPEC_OK;
        }
        if (c.kernel_select == MAMBA_SPEC_KERNEL_STREAM)
            return fail(ctx, MAMBA_SPEC_ERR_UNSUPPORTED, "%s: streaming kernel does not take this shape (%s)", who, plan.name);
    }
    const ConvBC *bcp = nullptr;
    if (p.flags & kFlagConvBC) {   // the conv over the B and C rows runs first, into scratch
        const size_t need = (size_t)p.batch * p.t_max * (p.GB + p.GC) * p.N * sizeof(float);
        if (ctx->bc_scratch_bytes < need) {
            if (ctx->map_cache.empty())
                return fail(ctx, MAMBA_SPEC_ERR_UNSUPPORTED, "%s: FLAG_CONV_BC needs a context (scratch for the conv's outputs)", who);
            if (ctx->bc_scratch) cudaFree(ctx->bc_scratch);   // (synchronises: no launch still uses it)
            ctx->bc_scratch = nullptr;
            ctx->bc_scratch_bytes = 0;
            e = cudaMalloc(&ctx->bc_scratch, need);
            if (e != cudaSuccess) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: scratch for the conv over B and C: %s", who, cudaGetErrorString(e));
            ctx->bc_scratch_bytes = need;
        }
        ctx->bc.out = ctx->bc_scratch;
        bcp = &ctx->bc;
        ctx->launches++;
    }
    e = launch_verify_generic(p, bf16, stream, bcp);
    if (e != cudaSuccess) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "%s: generic launch: %s", who, cudaGetErrorString(e));
    snprintf(ctx->last_kernel, sizeof ctx->last_kernel, "generic");
    ctx->launches++;
    return MAMBA_SPEC_OK;
}

int mamba_spec_verify(mamba_spec_ctx *ctx, void *state, void *conv_state, const void *x, const void *dt,
                      const void *B, const void *C, const float *A, const float *D,
                      const int32_t *n_prev_accepted, int32_t k_draft, const mamba_spec_io *io) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "verify: ctx is null");
    VerifyParams p;
    int rc = check_and_fill(ctx, p, state, conv_state, x, dt, B, C, A, D, n_prev_accepted, k_draft, io, "verify");
    if (rc) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "verify: cannot select device %d", ctx->cfg.device);
    cudaStream_t stream = (cudaStream_t)io->stream;
    rc = launch(ctx, p, stream, "verify");
    if (rc) return rc;
    ctx->last_stream = stream;
    ctx->last_k = k_draft;
    return MAMBA_SPEC_OK;
}

int mamba_spec_commit(mamba_spec_ctx *ctx, const int32_t *accept_len, int32_t batch, void *stream) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "commit: ctx is null");
    if (!accept_len) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "commit: accept_len is null");
    if (batch < 1 || batch > ctx->cfg.batch_max)
        return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "commit: batch %d outside 1..%d", batch, ctx->cfg.batch_max);
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "commit: cannot select device %d", ctx->cfg.device);
    const int k = ctx->last_k >= 0 ? ctx->last_k : ctx->cfg.k_max;
    cudaStream_t s = (cudaStream_t)stream;
    commit_kernel<<<(batch + 127) / 128, 128, 0, s>>>(ctx->d_n_prev, accept_len, batch, k, ctx->d_status,
                                                      (ctx->cfg.flags & MAMBA_SPEC_FLAG_COMMIT_SELECTS) ? ctx->d_sel : nullptr);
    CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    ctx->last_stream = s;
    return MAMBA_SPEC_OK;
}

static cudaError_t assemble_rows(void *slab, void *ring, const void *fresh, const int32_t *n_prev, int batch, int k, int k_max,
                                 int slab_rows, size_t row_bytes, int j_cap, cudaStream_t s) {
    const int unit = row_bytes % 16 == 0 ? 16 : row_bytes % 4 == 0 ? 4 : 2;
    const int units = (int)(row_bytes / unit);
    const long long n = (long long)batch * units;
    const unsigned blocks = (unsigned)((n + 255) / 256);
    if (unit == 16)
        assemble_rows_kernel<uint4><<<blocks, 256, 0, s>>>((uint4 *)slab, (uint4 *)ring, (const uint4 *)fresh, n_prev, batch, k, k_max, slab_rows, units, j_cap);
    else if (unit == 4)
        assemble_rows_kernel<uint32_t><<<blocks, 256, 0, s>>>((uint32_t *)slab, (uint32_t *)ring, (const uint32_t *)fresh, n_prev, batch, k, k_max, slab_rows, units, j_cap);
    else
        assemble_rows_kernel<uint16_t><<<blocks, 256, 0, s>>>((uint16_t *)slab, (uint16_t *)ring, (const uint16_t *)fresh, n_prev, batch, k, k_max, slab_rows, units, j_cap);
    return cudaGetLastError();
}

int mamba_spec_verify_new(mamba_spec_ctx *ctx, void *state, void *conv_state, const void *x_new, const void *dt_new,
                          const void *B_new, const void *C_new, const float *A, const float *D, int32_t k_draft,
                          const mamba_spec_io *io) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "verify_new: ctx is null");
    if (!io) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_new: io is null");
    const mamba_spec_config &c = ctx->cfg;
    if (k_draft < 0 || k_draft > c.k_max) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_new: k_draft %d outside 0..%d", k_draft, c.k_max);
    if (io->batch < 1 || io->batch > c.batch_max) return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "verify_new: batch %d outside 1..%d", io->batch, c.batch_max);
    if (io->layer < 0 || io->layer >= c.n_layers) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_new: layer %d outside 0..%d", io->layer, c.n_layers - 1);
    const bool gate = (c.flags & MAMBA_SPEC_FLAG_GATE) != 0;
    if (k_draft > 0 && (!x_new || !dt_new || !B_new || !C_new || (gate && !io->z)))
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_new: a required tensor pointer is null");
    if (c.k_max < 1) return fail(ctx, MAMBA_SPEC_ERR_UNSUPPORTED, "verify_new: the context was made with k_max = 0");
    DeviceGuard guard(c.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "verify_new: cannot select device %d", c.device);
    const size_t ab = act_bytes(c), hp = (size_t)c.n_heads * c.head_dim;
    const size_t row_bytes[5] = {hp * ab, hp * ab, ((c.flags & MAMBA_SPEC_FLAG_MAMBA1) ? hp : (size_t)c.n_heads) * ab,
                                 (size_t)c.n_groups_b * c.d_state * ab, (size_t)c.n_groups_c * c.d_state * ab};
    const int slab_rows = 2 * c.k_max;
    if (!ctx->ring_ready) {   // all or nothing
        cudaError_t e = cudaSuccess;
        for (int i = 0; i < 5 && e == cudaSuccess; ++i) {
            // (16 spare bytes: the streaming kernel's boxes may read a little past the last row of dt)
            e = cudaMalloc(&ctx->ring[i], (size_t)c.n_layers * c.batch_max * c.k_max * row_bytes[i] + 16);
            if (e == cudaSuccess) e = cudaMalloc(&ctx->slab[i], (size_t)c.batch_max * slab_rows * row_bytes[i] + 16);
            if (e == cudaSuccess) e = cudaMemset(ctx->slab[i], 0, (size_t)c.batch_max * slab_rows * row_bytes[i] + 16);
            if (e == cudaSuccess) e = cudaMemset(ctx->ring[i], 0, (size_t)c.n_layers * c.batch_max * c.k_max * row_bytes[i] + 16);
        }
        if (e != cudaSuccess) {
            for (int i = 0; i < 5; ++i) {
                if (ctx->ring[i]) cudaFree(ctx->ring[i]);
                if (ctx->slab[i]) cudaFree(ctx->slab[i]);
                ctx->ring[i] = ctx->slab[i] = nullptr;
            }
            return fail(ctx, MAMBA_SPEC_ERR_CUDA, "verify_new: row store allocation failed: %s", cudaGetErrorString(e));
        }
        ctx->ring_ready = true;
    }
    cudaStream_t s = (cudaStream_t)io->stream;
    const void *fresh[5] = {x_new, io->z, dt_new, B_new, C_new};
    for (int i = 0; i < 5; ++i) {
        if (i == 1 && !gate) continue;
        char *ring = (char *)ctx->ring[i] + (size_t)io->layer * c.batch_max * c.k_max * row_bytes[i];
        CUDA_TRY(ctx, assemble_rows(ctx->slab[i], ring, fresh[i], ctx->d_n_prev, io->batch, k_draft, c.k_max, slab_rows, row_bytes[i],
                                    c.k_max, s));
        ctx->launches++;
    }
    mamba_spec_io dio = *io;
    dio.z = gate ? ctx->slab[1] : nullptr;
    dio.t_max = slab_rows;
    VerifyParams p;
    int rc = check_and_fill(ctx, p, state, conv_state, ctx->slab[0], ctx->slab[2], ctx->slab[3], ctx->slab[4], A, D, nullptr, k_draft, &dio,
                            "verify_new");
    if (rc) return rc;
    p.flags |= kFlagYNewOnly;
    rc = launch(ctx, p, s, "verify_new");
    if (rc) return rc;
    ctx->last_stream = s;
    ctx->last_k = k_draft;
    return MAMBA_SPEC_OK;
}

int mamba_spec_verify_host(mamba_spec_ctx *ctx, void *state, void *conv_state, const void *x_host,
                           const void *dt_host, const void *B_host, const void *C_host, const float *A,
                           const float *D, const int32_t *n_prev_accepted_host, int32_t k_draft,
                           const mamba_spec_io *io) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "verify_host: ctx is null");
    if (!io) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host: io is null");
    const mamba_spec_config &c = ctx->cfg;
    const int t_cap = 2 * c.k_max > 1 ? 2 * c.k_max : 1;
    if (io->t_max > t_cap)
        return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "verify_host: t_max %d exceeds the staging rows %d", io->t_max, t_cap);
    if (!x_host || !dt_host || !B_host || !C_host || !io->y)
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host: a required host pointer is null");
    DeviceGuard guard(c.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "verify_host: cannot select device %d", c.device);
    const size_t ab = act_bytes(c), rows = (size_t)c.batch_max * t_cap;
    const size_t n_x = rows * c.n_heads * c.head_dim * ab, n_dt = (c.flags & MAMBA_SPEC_FLAG_MAMBA1) ? n_x : rows * c.n_heads * ab;
    const size_t n_B = rows * c.n_groups_b * c.d_state * ab, n_C = rows * c.n_groups_c * c.d_state * ab;
    if (!ctx->staging_ready) {   // all or nothing: a failed allocation leaves no half-built staging behind
        void **slots[] = {&ctx->st_x, &ctx->st_z, &ctx->st_y, &ctx->st_dt, &ctx->st_B, &ctx->st_C, (void **)&ctx->st_n_prev};
        const size_t sizes[] = {n_x, n_x, (c.flags & MAMBA_SPEC_FLAG_Y_F32) ? n_x / ab * 4 : n_x, n_dt + 16, n_B, n_C,
                                sizeof(int32_t) * (size_t)c.batch_max};
        cudaError_t e = cudaSuccess;
        for (int i = 0; i < 7 && e == cudaSuccess; ++i) e = cudaMalloc(slots[i], sizes[i]);
        if (e != cudaSuccess) {
            for (void **q : slots) { if (*q) cudaFree(*q); *q = nullptr; }
            return fail(ctx, MAMBA_SPEC_ERR_CUDA, "verify_host: staging allocation failed: %s", cudaGetErrorString(e));
        }
        ctx->staging_ready = true;
    }
    mamba_spec_io dio = *io;
    dio.z = (c.flags & MAMBA_SPEC_FLAG_GATE) ? ctx->st_z : nullptr;
    dio.y = ctx->st_y;
    VerifyParams p;
    int rc = check_and_fill(ctx, p, state, conv_state, ctx->st_x, ctx->st_dt, ctx->st_B, ctx->st_C, A, D,
                            n_prev_accepted_host ? ctx->st_n_prev : nullptr, k_draft, &dio, "verify_host");
    if (rc) return rc;
    if ((c.flags & MAMBA_SPEC_FLAG_GATE) && !io->z)
        return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host: gating is on but io->z is null");
    cudaStream_t s = (cudaStream_t)io->stream;
    const size_t used = (size_t)io->batch * io->t_max;
    const size_t b_x = used * c.n_heads * c.head_dim * ab;
    CUDA_TRY(ctx, cudaMemcpyAsync(ctx->st_x, x_host, b_x, cudaMemcpyHostToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(ctx->st_dt, dt_host, (c.flags & MAMBA_SPEC_FLAG_MAMBA1) ? b_x : used * c.n_heads * ab, cudaMemcpyHostToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(ctx->st_B, B_host, used * c.n_groups_b * c.d_state * ab, cudaMemcpyHostToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(ctx->st_C, C_host, used * c.n_groups_c * c.d_state * ab, cudaMemcpyHostToDevice, s));
    if (c.flags & MAMBA_SPEC_FLAG_GATE) CUDA_TRY(ctx, cudaMemcpyAsync(ctx->st_z, io->z, b_x, cudaMemcpyHostToDevice, s));
    if (n_prev_accepted_host)
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->st_n_prev, n_prev_accepted_host, sizeof(int32_t) * (size_t)io->batch,
                                      cudaMemcpyHostToDevice, s));
    rc = launch(ctx, p, s, "verify_host");
    if (rc) return rc;
    CUDA_TRY(ctx, cudaMemcpyAsync(io->y, ctx->st_y, (c.flags & MAMBA_SPEC_FLAG_Y_F32) ? b_x / ab * 4 : b_x,
                                  cudaMemcpyDeviceToHost, s));
    ctx->last_stream = s;
    ctx->last_k = k_draft;
    return MAMBA_SPEC_OK;
}

static int verify_host_static_impl(mamba_spec_ctx *tmp, void *state, void *conv_state, const void *x_host,
                                   const void *dt_host, const void *B_host, const void *C_host, const float *A,
                                   const float *D, const int32_t *n_prev_host, int32_t k_draft, const mamba_spec_io *io,
                                   int32_t *flags_host) {
    const mamba_spec_config &c = tmp->cfg;
    if (c.batch_max < 1 || c.n_layers < 1 || c.n_heads < 1 || c.head_dim < 1 || c.d_state < 1 || c.d_state > kMaxStateDim ||
        c.conv_width < 1 || c.conv_width > kMaxConvWidth || c.n_groups_b < 1 || c.n_groups_c < 1 ||
        c.n_heads % c.n_groups_b || c.n_heads % c.n_groups_c || c.k_max < 0 || c.k_max > 32 ||
        (c.act_dtype != MAMBA_SPEC_DTYPE_F32 && c.act_dtype != MAMBA_SPEC_DTYPE_BF16) ||
        (c.flags & ~(kAllFlags)) || c.kernel_select < 0 ||
        c.kernel_select > MAMBA_SPEC_KERNEL_STREAM || ((size_t)c.n_heads * c.head_dim * act_bytes(c)) % 16)
        return fail(tmp, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host_static: configuration rejected (same rules as mamba_spec_init)");
    if (c.flags & MAMBA_SPEC_FLAG_COMMIT_SELECTS)
        return fail(tmp, MAMBA_SPEC_ERR_UNSUPPORTED, "verify_host_static: FLAG_COMMIT_SELECTS needs a context");
    if (c.flags & MAMBA_SPEC_FLAG_GATED_RMSNORM)
        return fail(tmp, MAMBA_SPEC_ERR_UNSUPPORTED, "verify_host_static: FLAG_GATED_RMSNORM needs a context (scratch for the float32 rows)");
    if (c.flags & MAMBA_SPEC_FLAG_CONV_BC)
        return fail(tmp, MAMBA_SPEC_ERR_UNSUPPORTED, "verify_host_static: FLAG_CONV_BC needs a context (scratch for the conv's outputs)");
    if (!io) return fail(tmp, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host_static: io is null");
    if (!x_host || !dt_host || !B_host || !C_host || !n_prev_host || !io->y)
        return fail(tmp, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host_static: a required host pointer is null");
    if ((c.flags & MAMBA_SPEC_FLAG_GATE) && !io->z)
        return fail(tmp, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host_static: gating is on but io->z is null");
    if (io->batch < 1 || io->batch > c.batch_max || io->t_max < 1)
        return fail(tmp, MAMBA_SPEC_ERR_BAD_SHAPE, "verify_host_static: batch %d or t_max %d out of range", io->batch, io->t_max);
    if (c.device < 0 || c.device >= 64) return fail(tmp, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host_static: device %d outside 0..63", c.device);
    DeviceGuard guard(c.device);
    if (!guard.ok) return fail(tmp, MAMBA_SPEC_ERR_CUDA, "verify_host_static: cannot select device %d", c.device);
    StaticDevice &sd = g_static_dev[c.device];
    if (!sd.ready) {   // first call on this device: the array's name is only a host-side handle, ask for its device address
        void *ptr = nullptr;
        CUDA_TRY(tmp, cudaGetSymbolAddress(&ptr, g_static_staging));
        cudaDeviceProp prop;
        CUDA_TRY(tmp, cudaGetDeviceProperties(&prop, c.device));
        sd.base = static_cast<unsigned char *>(ptr);
        sd.sm_count = prop.multiProcessorCount;
        sd.smem_per_sm = prop.sharedMemPerMultiprocessor;
        sd.smem_optin = prop.sharedMemPerBlockOptin;
        sd.ready = true;
    }
    // carve the staging array: pending lengths, status word, then the token slabs
    const size_t ab = act_bytes(c), used = (size_t)io->batch * io->t_max;
    const size_t b_x = used * c.n_heads * c.head_dim * ab, b_dt = (c.flags & MAMBA_SPEC_FLAG_MAMBA1) ? b_x : used * c.n_heads * ab;
    const size_t b_B = used * c.n_groups_b * c.d_state * ab, b_C = used * c.n_groups_c * c.d_state * ab;
    const size_t b_y = (c.flags & MAMBA_SPEC_FLAG_Y_F32) ? b_x / ab * 4 : b_x;
    // every factor is a positive int32, so no single product above can wrap a 64-bit size_t unless it is far
    // beyond the array anyway; refuse those before summing
    const double approx = (double)used * c.n_heads * c.head_dim * 4.0 + (double)used * (c.n_groups_b + c.n_groups_c) * c.d_state * 4.0;
    if (approx > (double)kStaticStagingBytes * 4.0 || b_x > kStaticStagingBytes || b_y > kStaticStagingBytes ||
        b_B > kStaticStagingBytes || b_C > kStaticStagingBytes || b_dt > kStaticStagingBytes)
        return fail(tmp, MAMBA_SPEC_ERR_UNSUPPORTED, "verify_host_static: this call's slabs exceed the built-in %zu-byte staging array",
                    kStaticStagingBytes);
    size_t o = 0;
    const size_t o_np = o; o += up256(sizeof(int32_t) * (size_t)io->batch);
    const size_t o_st = o; o += 256;
    const size_t o_x = o;  o += up256(b_x);
    const size_t o_z = o;  o += (c.flags & MAMBA_SPEC_FLAG_GATE) ? up256(b_x) : 0;
    const size_t o_dt = o; o += up256(b_dt + 16);
    const size_t o_B = o;  o += up256(b_B);
    const size_t o_C = o;  o += up256(b_C);
    const size_t o_y = o;  o += up256(b_y);
    if (o > kStaticStagingBytes)
        return fail(tmp, MAMBA_SPEC_ERR_UNSUPPORTED, "verify_host_static: this call needs %zu bytes of staging, the built-in array holds %zu",
                    o, kStaticStagingBytes);
    unsigned char *base = sd.base;
    tmp->sm_count = sd.sm_count; tmp->smem_per_sm = sd.smem_per_sm; tmp->smem_optin = sd.smem_optin;
    tmp->d_n_prev = reinterpret_cast<int32_t *>(base + o_np);
    tmp->d_status = reinterpret_cast<int32_t *>(base + o_st);
    mamba_spec_io dio = *io;
    dio.z = (c.flags & MAMBA_SPEC_FLAG_GATE) ? base + o_z : nullptr;
    dio.y = base + o_y;
    VerifyParams p;
    int rc = check_and_fill(tmp, p, state, conv_state, base + o_x, base + o_dt, base + o_B, base + o_C, A, D,
                            tmp->d_n_prev, k_draft, &dio, "verify_host_static");
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)io->stream;
    CUDA_TRY(tmp, cudaMemsetAsync(base + o_st, 0, sizeof(int32_t), s));   // the array keeps the last call's contents
    CUDA_TRY(tmp, cudaMemcpyAsync(base + o_np, n_prev_host, sizeof(int32_t) * (size_t)io->batch, cudaMemcpyHostToDevice, s));
    CUDA_TRY(tmp, cudaMemcpyAsync(base + o_x, x_host, b_x, cudaMemcpyHostToDevice, s));
    CUDA_TRY(tmp, cudaMemcpyAsync(base + o_dt, dt_host, b_dt, cudaMemcpyHostToDevice, s));
    CUDA_TRY(tmp, cudaMemcpyAsync(base + o_B, B_host, b_B, cudaMemcpyHostToDevice, s));
    CUDA_TRY(tmp, cudaMemcpyAsync(base + o_C, C_host, b_C, cudaMemcpyHostToDevice, s));
    if (c.flags & MAMBA_SPEC_FLAG_GATE) CUDA_TRY(tmp, cudaMemcpyAsync(base + o_z, io->z, b_x, cudaMemcpyHostToDevice, s));
    rc = launch(tmp, p, s, "verify_host_static");
    if (rc) return rc;
    CUDA_TRY(tmp, cudaMemcpyAsync(io->y, base + o_y, b_y, cudaMemcpyDeviceToHost, s));
    if (flags_host) CUDA_TRY(tmp, cudaMemcpyAsync(flags_host, base + o_st, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    return MAMBA_SPEC_OK;
}

int mamba_spec_verify_host_static(const mamba_spec_config *cfg, void *state, void *conv_state, const void *x_host,
                                  const void *dt_host, const void *B_host, const void *C_host, const float *A,
                                  const float *D, const int32_t *n_prev_accepted_host, int32_t k_draft,
                                  const mamba_spec_io *io, int32_t *device_flags_host) {
    if (!cfg) return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "verify_host_static: cfg is null");
    mamba_spec_ctx tmp;   // lives for this call only; owns no device memory
    tmp.cfg = *cfg;
    const int rc = verify_host_static_impl(&tmp, state, conv_state, x_host, dt_host, B_host, C_host, A, D,
                                           n_prev_accepted_host, k_draft, io, device_flags_host);
    if (rc) g_init_error = tmp.err;   // reported by mamba_spec_last_error(NULL)
    return rc;
}

int mamba_spec_status(mamba_spec_ctx *ctx, int32_t *device_flags_out) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "status: ctx is null");
    if (!device_flags_out) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "status: output pointer is null");
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "status: cannot select device %d", ctx->cfg.device);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    CUDA_TRY(ctx, cudaMemcpy(device_flags_out, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    CUDA_TRY(ctx, cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    return MAMBA_SPEC_OK;
}

int mamba_spec_get_n_prev(mamba_spec_ctx *ctx, int32_t *n_prev_host, int32_t batch) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "get_n_prev: ctx is null");
    if (!n_prev_host) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "get_n_prev: output pointer is null");
    if (batch < 1 || batch > ctx->cfg.batch_max)
        return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "get_n_prev: batch %d outside 1..%d", batch, ctx->cfg.batch_max);
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "get_n_prev: cannot select device %d", ctx->cfg.device);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    CUDA_TRY(ctx, cudaMemcpy(n_prev_host, ctx->d_n_prev, sizeof(int32_t) * (size_t)batch, cudaMemcpyDeviceToHost));
    return MAMBA_SPEC_OK;
}

int mamba_spec_get_selection(mamba_spec_ctx *ctx, int32_t *sel_host, int32_t batch) {
    if (!ctx) return fail(nullptr, MAMBA_SPEC_ERR_NOT_INIT, "get_selection: ctx is null");
    if (!sel_host) return fail(ctx, MAMBA_SPEC_ERR_INVALID_ARG, "get_selection: output pointer is null");
    if (batch < 1 || batch > ctx->cfg.batch_max)
        return fail(ctx, MAMBA_SPEC_ERR_BAD_SHAPE, "get_selection: batch %d outside 1..%d", batch, ctx->cfg.batch_max);
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, MAMBA_SPEC_ERR_CUDA, "get_selection: cannot select device %d", ctx->cfg.device);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    CUDA_TRY(ctx, cudaMemcpy(sel_host, ctx->d_sel, sizeof(int32_t) * (size_t)batch, cudaMemcpyDeviceToHost));
    return MAMBA_SPEC_OK;
}

int mamba_spec_describe_plan(const mamba_spec_config *cfg, int32_t batch, int32_t t_max, int32_t k_draft,
                             int32_t sm_count, int64_t smem_per_block, char *buf, int32_t buf_len) {
    if (!cfg || !buf || buf_len < 1) return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "describe_plan: null cfg or buffer");
    const mamba_spec_config &c = *cfg;
    if (c.n_heads < 1 || c.head_dim < 1 || c.d_state < 1 || c.n_groups_b < 1 || c.n_groups_c < 1 || c.n_heads % c.n_groups_b ||
        c.n_heads % c.n_groups_c || batch < 1 || t_max < 1 || k_draft < 0 || k_draft > t_max || c.k_max < 0)
        return fail(nullptr, MAMBA_SPEC_ERR_INVALID_ARG, "describe_plan: shape out of range");
    if (sm_count <= 0 || smem_per_block <= 0) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, c.device) != cudaSuccess)
            return fail(nullptr, MAMBA_SPEC_ERR_CUDA, "describe_plan: no CUDA device %d to ask", c.device);
        sm_count = prop.multiProcessorCount;
        smem_per_block = (int64_t)prop.sharedMemPerBlockOptin;
    }
    VerifyParams p;
    memset(&p, 0, sizeof p);
    p.batch = batch; p.t_max = t_max; p.H = c.n_heads; p.P = c.head_dim; p.N = c.d_state;
    p.GB = c.n_groups_b; p.GC = c.n_groups_c; p.W = c.conv_width; p.k = k_draft;
    p.j_cap = c.k_max < t_max - k_draft ? c.k_max : t_max - k_draft;
    p.flags = c.flags;
    // the planner only looks at whether these are set
    p.z = (c.flags & MAMBA_SPEC_FLAG_GATE) ? (const void *)buf : nullptr;
    p.state_k = (c.flags & MAMBA_SPEC_FLAG_STATE_K) ? (float *)buf : nullptr;
    const bool bf16 = c.act_dtype == MAMBA_SPEC_DTYPE_BF16;
    if (c.kernel_select != MAMBA_SPEC_KERNEL_GENERIC) {
        if (c.flags & MAMBA_SPEC_FLAG_COMMIT_SELECTS) p.sel = reinterpret_cast<const int32_t *>(buf);
        const SplitPlan sp = plan_split(p, c, sm_count, (size_t)smem_per_block);
        const StreamPlan plan = sp.split ? sp.first : plan_verify_stream(p, bf16, sm_count, (size_t)smem_per_block);
        if (sp.split) snprintf(buf, (size_t)buf_len, "split(launches=%d,pending_only=%d) first %s", sp.launches, sp.pending_only, plan.name);
        else if (plan.ok) snprintf(buf, (size_t)buf_len, "%s", plan.name);
        else snprintf(buf, (size_t)buf_len, "generic (%s)", plan.name);
    } else {
        snprintf(buf, (size_t)buf_len, "generic (selected)");
    }
    return MAMBA_SPEC_OK;
}

int64_t mamba_spec_launch_count(const mamba_spec_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *mamba_spec_last_kernel(const mamba_spec_ctx *ctx) { return ctx ? ctx->last_kernel : "none"; }

const char *mamba_spec_last_error(const mamba_spec_ctx *ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

void mamba_spec_destroy(mamba_spec_ctx *ctx) {
    if (!ctx) return;
    {
        DeviceGuard guard(ctx->cfg.device);
        if (guard.ok) {
            cudaDeviceSynchronize();
            for (int i = 0; i < 5; ++i) {
                if (ctx->ring[i]) cudaFree(ctx->ring[i]);
                if (ctx->slab[i]) cudaFree(ctx->slab[i]);
            }
            for (int i = 0; i < 2; ++i) {
                if (ctx->split_state[i]) cudaFree(ctx->split_state[i]);
                if (ctx->split_conv[i]) cudaFree(ctx->split_conv[i]);
            }
            if (ctx->d_zero) cudaFree(ctx->d_zero);
            if (ctx->norm_scratch) cudaFree(ctx->norm_scratch);
            if (ctx->bc_scratch) cudaFree(ctx->bc_scratch);
            void *bufs[] = {ctx->d_n_prev, ctx->d_status, ctx->d_sel, ctx->st_x, ctx->st_dt, ctx->st_B, ctx->st_C,
                            ctx->st_z, ctx->st_y, ctx->st_n_prev};
            for (void *b : bufs)
                if (b) cudaFree(b);
        }
    }
    delete ctx;
}

}  // extern "C"
#pragma GCC visibility pop
