// Shared declarations of the CUDA side of mamba_spec (host API <-> kernels).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mspec {

constexpr int kMaxConvWidth = 8;
constexpr int kMaxStateDim = 256;

// Everything one verification launch needs.  All pointers are device pointers.
struct VerifyParams {
    float *state;            // [batch][H][P][N]
    void *conv_state;        // [batch][W-1][H*P] act dtype
    const void *x;           // [batch][t_max][H][P]
    const void *dt;          // [batch][t_max][H]; Mamba-1 form: [batch][t_max][H*P]
    const void *B;           // [batch][t_max][GB][N]
    const void *C;           // [batch][t_max][GC][N]
    const void *z;           // [batch][t_max][H][P] or null
    void *y;                 // [batch][t_max][H][P]
    float *state_k;          // [batch][H][P][N], second snapshot (after all tokens), or null
    void *conv_state_k;      // [batch][W-1][H*P] act dtype, second snapshot, or null
    const float *A;          // [H]; Mamba-1 form: [H*P][N]
    const float *D;          // [H]; Mamba-1 form: [H*P]
    const float *dt_bias;    // [H] ([H*P] in the Mamba-1 form) or null: added to the raw interval before its softplus
    const int32_t *sel;      // [batch] or null: which of (state, state_k) holds each sequence's cache (commit-selects mode)
    const int32_t *row_off;  // [batch] or null: token t of sequence b is row row_off[b] + row_off_const + t of its slab
    int32_t row_off_const;   //   (later segments of a token block that is split over several launches)
    int32_t row_off_cap;     //   largest legal row_off[b]
    int32_t n_prev_done;     // pending rows of each sequence that earlier launches of this call have replayed already
    int32_t n_prev_full;     //   and, when non-zero, the bound on n_prev[b] itself (j_cap bounds what is left of it)
    const float *conv_w;     // [H*P][W]
    const float *conv_b;     // [H*P]
    const int32_t *n_prev;   // [batch]
    int32_t *status;         // device status word (atomicOr)
    int32_t batch, t_max, H, P, N, GB, GC, W;
    int32_t k;               // draft tokens this call
    int32_t j_cap;           // largest legal n_prev: min(k_max, t_max - k)
    int32_t flags;           // MAMBA_SPEC_FLAG_*
};

constexpr int kFlagGate = 1;
constexpr int kFlagConvSilu = 2;
constexpr int kFlagYF32 = 4;
constexpr int kFlagStateK = 8;
constexpr int kFlagMamba1 = 16;        // interval per channel, A per (channel, state column), D per channel
constexpr int kFlagDtSoftplus = 32;    // dt arrives raw: softplus(dt + dt_bias) is taken in the kernel
constexpr int kFlagCommitSelects = 64; // the cache of sequence b is state or state_k as sel[b] says
constexpr int kFlagConvBC = 256;       // B and C pass through a depthwise conv of their own first (generic kernel only)
constexpr int kFlagGatedRmsnorm = 128; // host side: y goes through float32 scratch and a normalising epilogue kernel
constexpr int kFlagYNewOnly = 1 << 16; // internal: y holds only the k new rows of each sequence, [batch][k]
constexpr int kStatusNprevClamped = 1;
constexpr int kStatusAcceptClamped = 2;
constexpr int kStatusCopyTimeout = 4;

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }
// softplus, the identity where exp would overflow into it anyway
__device__ __forceinline__ float softplus_f(float v) { return v > 20.f ? v : log1pf(expf(v)); }

__device__ __forceinline__ float ld_act(const float *p, size_t i) { return p[i]; }
__device__ __forceinline__ float ld_act(const __nv_bfloat16 *p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st_act(float *p, size_t i, float v) { p[i] = v; }
__device__ __forceinline__ void st_act(__nv_bfloat16 *p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

// First slab row of sequence b's tokens in this launch (0 unless the block was split; the offsets are pending
// lengths, clamped like them).
__device__ __forceinline__ int first_row(const VerifyParams &p, int b) {
    int off = p.row_off_const;
    if (p.row_off != nullptr) {
        const int v = p.row_off[b];
        off += v < 0 ? 0 : (v > p.row_off_cap ? p.row_off_cap : v);
    }
    return off;
}

// Reads n_prev[b], clamps it into [0, j_cap] and flags the status word if it had to.
__device__ __forceinline__ int load_n_prev(const VerifyParams &p, int b) {
    int j = p.n_prev[b];
    const int full = p.n_prev_full ? p.n_prev_full : p.j_cap;
    if (j < 0 || j > full) {
        atomicOr(p.status, kStatusNprevClamped);
        j = j < 0 ? 0 : full;
    }
    j -= p.n_prev_done;
    return j < 0 ? 0 : (j > p.j_cap ? p.j_cap : j);
}
// The same value without the report (for a second kernel that reads the same entry).
__device__ __forceinline__ int peek_n_prev(const VerifyParams &p, int b) {
    int j = p.n_prev[b];
    const int full = p.n_prev_full ? p.n_prev_full : p.j_cap;
    j = j < 0 ? 0 : (j > full ? full : j);
    j -= p.n_prev_done;
    return j < 0 ? 0 : (j > p.j_cap ? p.j_cap : j);
}

// Launchers (defined in verify_generic.cu / verify_stream.cu).  Return cudaGetLastError().
// FLAG_CONV_BC: what the conv over the B and C channels needs beside VerifyParams.  Channel c of the
// (GB + GC) * N channels is column c of B for c < GB * N, else column c - GB * N of C.
struct ConvBC {
    void *window;        // [batch][W-1][(GB+GC)*N] act dtype, in/out: the last W-1 B and C rows at the cached position
    const float *taps;   // [(GB+GC)*N][W]
    const float *bias;   // [(GB+GC)*N]
    float *out;          // scratch, float32: the conv's outputs laid out like B, [batch][t_max][GB][N], then like C
};
cudaError_t launch_verify_generic(const VerifyParams &p, bool bf16, cudaStream_t stream, const ConvBC *bc = nullptr);

// Shared-memory plan of the streaming kernel: ring depths and byte offsets (all multiples of 16).
struct StreamLayout {
    int S, R;           // stages of the state ring and of the raw-input ring
    int ngroups;        // compute groups in use (each needs a buffer)
    int TCAP, JCAP;     // token rows / replayed tokens the buffers are sized for
    int lead;           // chunks by which the small-input copies run ahead of the state copies
    float inv_hpg_b, inv_hpg_c;   // 1 / (heads per B group), 1 / (heads per C group)
    int state_off, state_stride;
    int raw_off, raw_stride, raw_tx, r_x, r_z, r_B, r_C, r_dt, r_cst, r_cw, r_cb;   // raw_tx: bytes one fill brings in
    int grp_off, grp_stride, c_Cf, c_Bf, c_gz, c_xc, c_G, c_hc, c_part;   // per compute group
};
struct StreamPlan {
    bool ok;
    int grid, variant;
    size_t smem_bytes;
    StreamLayout layout;
    char name[112];
};
// Tensor maps of one launch (opaque 128-byte descriptors, the driver's CUtensorMap): one TMA request then
// fetches the rows of all tokens of a chunk (the rows of one token are H*P apart in memory).
struct alignas(64) TensorMapBytes {
    unsigned char opaque[128];
};
struct alignas(64) InputMaps {
    TensorMapBytes x, z, B, C, dt, cst;
    TensorMapBytes state;    // [32 columns][rows][N/32 quarters], 128-byte swizzle
    TensorMapBytes state_k;  // the same over the second snapshot's buffer (FLAG_STATE_K only)
    TensorMapBytes cst_k;    // the conv window of the second pair of buffers (commit-selects mode)
};
StreamPlan plan_verify_stream(const VerifyParams &p, bool bf16, int sm_count, size_t smem_per_block_optin);
// Encodes the tensor maps of a launch (host work: eight driver calls); false if the driver refuses.
bool encode_stream_maps(const VerifyParams &p, const StreamPlan &plan, InputMaps *tm);
cudaError_t launch_verify_stream(const VerifyParams &p, const StreamPlan &plan, const InputMaps &tm, cudaStream_t stream);

}  // namespace mspec
