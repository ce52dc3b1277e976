// Generic verification kernel: the plain sequential recurrence (Eq. 1 with the
// on-the-fly discretisation of Sec. 2.2), one warp per state row, for any
// supported shape and either activation dtype.  It is the path for shapes the
// streaming kernel does not take (tiny heads, fp32 activations, odd conv
// widths) and an in-library cross-check of the streaming kernel's algebra.
//
// A warp owns row (b, h, p): its N state values live in registers, lane l
// holding columns l, l+32, ...  Per token it evaluates the causal conv tap sum
// for its channel (every lane redundantly; the window is W-1 registers),
// decays and updates the row, reduces C.h by warp shuffles and lets lane 0
// store y.  After token j_b-1 the row and the conv window are written back;
// the k draft tokens that follow only ever touch registers (Sec. 4.2: the
// snapshot h_j is saved before the drafts are evaluated; Sec. 4.3 i)-iii)).
//
// The same kernel covers the variants of the parameterisation: the Mamba-1 form
// (Algorithm 1: interval per channel, A per channel and state column, where the
// decay is an exp per state element), the softplus of a raw interval taken in the
// kernel, the mode in which each sequence's cache is one of two buffers
// (Algorithm 2 keeps h_j or h_k), and outputs for the new rows only.
#include "common.cuh"

namespace mspec {

// FLAG_CONV_BC: the rolling depthwise causal conv (Sec. 4.3, footnote) over the B and C rows, one thread per
// (sequence, channel), ahead of the recurrence: outputs in float32 to scratch laid out like B and C
// ([batch][t_max][GB][N] followed by [batch][t_max][GC][N]), the window at the verified position written back.
template <typename act_t>
__global__ void __launch_bounds__(128) conv_bc_kernel(const VerifyParams p, const ConvBC bc) {
    const int chB = p.GB * p.N, chC = p.GC * p.N, ch = chB + chC;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)p.batch * ch) return;
    const int b = (int)(i / ch), c = (int)(i % ch);
    const int j = peek_n_prev(p, b), T = j + p.k, W = p.W;
    const bool isB = c < chB;
    const act_t *src = isB ? (const act_t *)p.B : (const act_t *)p.C;
    const int cc = isB ? c : c - chB, cw = isB ? chB : chC;
    float *dst = bc.out + (isB ? 0 : (size_t)p.batch * p.t_max * chB);
    act_t *window = (act_t *)bc.window;
    float win[kMaxConvWidth - 1], tap[kMaxConvWidth];
#pragma unroll
    for (int w = 0; w < kMaxConvWidth - 1; ++w) win[w] = (w < W - 1) ? ld_act(window, ((size_t)b * (W - 1) + w) * ch + c) : 0.f;
#pragma unroll
    for (int w = 0; w < kMaxConvWidth; ++w) tap[w] = (w < W) ? bc.taps[(size_t)c * W + w] : 0.f;
    const float bias = bc.bias[c];
    const int row_first = first_row(p, b);
    for (int t = 0; t < T; ++t) {
        const size_t bt = (size_t)b * p.t_max + row_first + t;
        const float in = ld_act(src, bt * cw + cc);
        float acc = bias;
#pragma unroll
        for (int w = 0; w < kMaxConvWidth - 1; ++w)
            if (w < W - 1) acc = fmaf(tap[w], win[w], acc);
#pragma unroll
        for (int w = 0; w < kMaxConvWidth; ++w)
            if (w == W - 1) acc = fmaf(tap[w], in, acc);
        dst[bt * cw + cc] = (p.flags & kFlagConvSilu) ? silu_f(acc) : acc;
#pragma unroll
        for (int w = 0; w < kMaxConvWidth - 2; ++w)
            if (w < W - 2) win[w] = win[w + 1];
#pragma unroll
        for (int w = 0; w < kMaxConvWidth - 1; ++w)
            if (w == W - 2) win[w] = in;
        if (t == j - 1) {
#pragma unroll
            for (int w = 0; w < kMaxConvWidth - 1; ++w)
                if (w < W - 1) st_act(window, ((size_t)b * (W - 1) + w) * ch + c, win[w]);
        }
    }
}

template <typename act_t, bool M1, typename bc_t>
__global__ void __launch_bounds__(128) verify_generic_kernel(const VerifyParams p) {
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long rows = (long long)p.batch * p.H * p.P;
    if (row >= rows) return;
    const int pr = (int)(row % p.P);
    const int h = (int)((row / p.P) % p.H);
    const int b = (int)(row / ((long long)p.P * p.H));
    const int j = load_n_prev(p, b);
    const int T = j + p.k;
    if (T == 0 && p.state_k == nullptr) return;

    const int N = p.N, W = p.W, H = p.H, P = p.P;
    const int Cch = H * P, c = h * P + pr;
    const act_t *x = (const act_t *)p.x, *dt = (const act_t *)p.dt, *z = (const act_t *)p.z;
    const bc_t *Bm = (const bc_t *)p.B, *Cm = (const bc_t *)p.C;   // (float32 after their own conv, FLAG_CONV_BC)
    act_t *y = (act_t *)p.y;
    // commit-selects mode: this sequence's cache is the second pair of buffers when sel says so; the state
    // at the verified position goes back to where the cache is, the state after all tokens to the other pair
    const bool swapped = p.sel != nullptr && p.sel[b] != 0;
    act_t *cst = (act_t *)(swapped ? p.conv_state_k : p.conv_state), *cst_other = (act_t *)(swapped ? p.conv_state : p.conv_state_k);
    float *st_cur = swapped ? p.state_k : p.state, *st_other = swapped ? p.state : p.state_k;
    const int gB = h / (H / p.GB), gC = h / (H / p.GC);
    const int row_first = first_row(p, b);

    float win[kMaxConvWidth - 1], tap[kMaxConvWidth];
#pragma unroll
    for (int w = 0; w < kMaxConvWidth - 1; ++w)
        win[w] = (w < W - 1) ? ld_act(cst, ((size_t)b * (W - 1) + w) * Cch + c) : 0.f;
#pragma unroll
    for (int w = 0; w < kMaxConvWidth; ++w) tap[w] = (w < W) ? p.conv_w[(size_t)c * W + w] : 0.f;
    const float bias = p.conv_b[c], A_h = M1 ? 0.f : p.A[h], D_h = p.D[M1 ? c : h];
    const bool sp = (p.flags & kFlagDtSoftplus) != 0, y_new = (p.flags & kFlagYNewOnly) != 0;
    const float dtb = (sp && p.dt_bias) ? p.dt_bias[M1 ? c : h] : 0.f;

    constexpr int kRegs = kMaxStateDim / 32;
    float hreg[kRegs];
    float *srow = st_cur + (size_t)row * N;
    float Areg[M1 ? kRegs : 1];   // Mamba-1 form: this channel's row of A
    if (M1) {
#pragma unroll
        for (int i = 0; i < kRegs; ++i) Areg[M1 ? i : 0] = (lane + 32 * i < N) ? p.A[(size_t)c * N + lane + 32 * i] : 0.f;
    }
#pragma unroll
    for (int i = 0; i < kRegs; ++i) hreg[i] = (lane + 32 * i < N) ? srow[lane + 32 * i] : 0.f;

    for (int t = 0; t < T; ++t) {
        const size_t bt = (size_t)b * p.t_max + row_first + t;
        const float xin = ld_act(x, (bt * H + h) * P + pr);
        float acc = bias;
#pragma unroll
        for (int w = 0; w < kMaxConvWidth - 1; ++w)
            if (w < W - 1) acc = fmaf(tap[w], win[w], acc);
#pragma unroll
        for (int w = 0; w < kMaxConvWidth; ++w)
            if (w == W - 1) acc = fmaf(tap[w], xin, acc);
        const float xc = (p.flags & kFlagConvSilu) ? silu_f(acc) : acc;
#pragma unroll
        for (int w = 0; w < kMaxConvWidth - 2; ++w)
            if (w < W - 2) win[w] = win[w + 1];
#pragma unroll
        for (int w = 0; w < kMaxConvWidth - 1; ++w)
            if (w == W - 2) win[w] = xin;

        float dtv = ld_act(dt, M1 ? bt * Cch + c : bt * H + h);
        if (sp) dtv = softplus_f(dtv + dtb);
        const float a = M1 ? 0.f : expf(dtv * A_h), u = dtv * xc;
        const bc_t *Bv = Bm + (bt * p.GB + gB) * N, *Cv = Cm + (bt * p.GC + gC) * N;
        float part = 0.f;
#pragma unroll
        for (int i = 0; i < kRegs; ++i) {
            const int n = lane + 32 * i;
            if (n < N) {
                hreg[i] = fmaf(M1 ? expf(dtv * Areg[M1 ? i : 0]) : a, hreg[i], u * ld_act(Bv, n));
                part = fmaf(ld_act(Cv, n), hreg[i], part);
            }
        }
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) part += __shfl_xor_sync(0xffffffffu, part, m);
        if (lane == 0) {
            float v = fmaf(D_h, xc, part);
            if ((p.flags & kFlagGate) && z) v *= silu_f(ld_act(z, (bt * H + h) * P + pr));
            // (with new rows only: y is [batch][k], the replayed rows' outputs are dropped)
            const size_t yi = y_new ? (((size_t)b * p.k + (t - j)) * H + h) * P + pr : (bt * H + h) * P + pr;
            if (!y_new || t >= j) {
                if (p.flags & kFlagYF32) reinterpret_cast<float *>(p.y)[yi] = v;
                else st_act(y, yi, v);
            }
        }
        if (t == j - 1) {  // the newly verified position: cache the state and the conv window here
#pragma unroll
            for (int i = 0; i < kRegs; ++i)
                if (lane + 32 * i < N) srow[lane + 32 * i] = hreg[i];
            if (lane == 0) {
#pragma unroll
                for (int w = 0; w < kMaxConvWidth - 1; ++w)
                    if (w < W - 1) st_act(cst, ((size_t)b * (W - 1) + w) * Cch + c, win[w]);
            }
        }
    }
    if (p.state_k) {  // second snapshot: the cache after all T tokens (Algorithm 2: h_k)
        float *krow = st_other + (size_t)row * N;
#pragma unroll
        for (int i = 0; i < kRegs; ++i)
            if (lane + 32 * i < N) krow[lane + 32 * i] = hreg[i];
        if (lane == 0) {
            act_t *cstk = cst_other;
#pragma unroll
            for (int w = 0; w < kMaxConvWidth - 1; ++w)
                if (w < W - 1) st_act(cstk, ((size_t)b * (W - 1) + w) * Cch + c, win[w]);
        }
    }
}

cudaError_t launch_verify_generic(const VerifyParams &p, bool bf16, cudaStream_t stream, const ConvBC *bc) {
    const long long rows = (long long)p.batch * p.H * p.P;
    const int warps_per_block = 4;
    const long long blocks = (rows + warps_per_block - 1) / warps_per_block;
    if (blocks <= 0 || blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const bool m1 = (p.flags & kFlagMamba1) != 0;
    const unsigned nb = (unsigned)blocks, nt = warps_per_block * 32;
    if (bc != nullptr) {
        // the conv over the B and C rows first; the recurrence then reads its float32 outputs in their place
        const long long items = (long long)p.batch * (p.GB + p.GC) * p.N, cblocks = (items + 127) / 128;
        if (cblocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
        if (bf16) conv_bc_kernel<__nv_bfloat16><<<(unsigned)cblocks, 128, 0, stream>>>(p, *bc);
        else conv_bc_kernel<float><<<(unsigned)cblocks, 128, 0, stream>>>(p, *bc);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        VerifyParams q = p;
        q.B = bc->out;
        q.C = bc->out + (size_t)p.batch * p.t_max * p.GB * p.N;
        if (bf16 && m1) verify_generic_kernel<__nv_bfloat16, true, float><<<nb, nt, 0, stream>>>(q);
        else if (bf16) verify_generic_kernel<__nv_bfloat16, false, float><<<nb, nt, 0, stream>>>(q);
        else if (m1) verify_generic_kernel<float, true, float><<<nb, nt, 0, stream>>>(q);
        else verify_generic_kernel<float, false, float><<<nb, nt, 0, stream>>>(q);
        return cudaGetLastError();
    }
    if (bf16 && m1) verify_generic_kernel<__nv_bfloat16, true, __nv_bfloat16><<<nb, nt, 0, stream>>>(p);
    else if (bf16) verify_generic_kernel<__nv_bfloat16, false, __nv_bfloat16><<<nb, nt, 0, stream>>>(p);
    else if (m1) verify_generic_kernel<float, true, float><<<nb, nt, 0, stream>>>(p);
    else verify_generic_kernel<float, false, float><<<nb, nt, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace mspec
