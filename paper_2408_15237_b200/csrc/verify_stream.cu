// Streaming verification kernel for sm_100a: bf16 activations, fp32 state, conv
// width 4, state dim 64 or 128, head dim a multiple of 32.
//
// The call has to read (and, where tokens were accepted, re-write) the fp32
// state once; everything else is small.  One persistent CTA per SM takes every
// gridDim.x-th chunk (a chunk = CR state rows of one (sequence, head)) and runs:
//
//   producer warp    per chunk one TMA request for the state rows (a 3-D tiled
//                    tensor map that lays the rows down as swizzled 32-column
//                    quarters) into a ring of state stages, and eight more for the
//                    small inputs (x, z, B, C, dt rows of all tokens through 2-D
//                    tensor maps, the conv window, taps and bias) into a ring of raw
//                    stages.  A request costs the TMA unit 60-80 cycles whatever its
//                    size, so there are few and large ones; per-thread cp.async or
//                    per-token bulk copies were several times slower.
//   compute groups   kGroups groups of four warps, all running the same code (small
//                    instruction footprint; three role-specific code paths thrashed
//                    the instruction cache).  Group g takes every ngroups-th chunk
//                    and does both of its phases:
//                    prologue: what depends on the inputs but not on the state --
//                      causal conv + SiLU with the rolling window (Sec. 4.3, footnote),
//                      the gate SiLU(z), the on-the-fly discretisation (Sec. 2.2), an
//                      fp32 copy of C, the small matrices of the unrolled recurrence,
//                      and the conv window at the verified position j (written back);
//                    stream: one thread per state row and 32-column quarter -- dot
//                      products with every C_t, the state at position j formed in
//                      registers, put back into the stage and stored by one TMA
//                      request (Sec. 4.3 iii), and y.
//                    While one group is in its prologue the others stream.
//
// Rings and groups are connected by full/empty mbarriers; the only other
// barriers are named barriers inside a group.  The kernel is launched with
// programmatic stream serialisation: its on-chip set-up overlaps the tail of the
// previous kernel.
//
// The recurrence (Eq. 1, discretised on the fly) is evaluated in its unrolled
// form, the same sum in another order.  With a_t = exp(dt_t A_h), the cached
// state h and xc the post-conv input:
//     y_t[p]   = alpha_t (C_t . h[p,:]) + w_t[p],
//     w_t[p]   = sum_{s<=t} G[t][s] xc_s[p] + D_h xc_t[p],
//     G[t][s]  = (C_t . B_s) dt_s prod_{s<r<=t} a_r,      alpha_t = prod_{r<=t} a_r,
//     h_j[p,:] = alpha_{j-1} h[p,:] + sum_{s<j} (dt_s prod_{s<r<j} a_r) xc_s[p] B_s.
// Each state element is touched by T multiply-adds for the outputs and j+1 for
// the new state; the per-token states never exist (Sec. 4.2) and the state at
// the verified position is formed and stored once.  Multiply-adds on the state
// are packed f32x2 operations, no tensor cores (fp32 state, exact products
// wanted); only the small T x T table of bf16 dot products C_t . B_s, exact in
// fp32, is formed with warp-level matrix instructions.  D_h rides on the
// diagonal of G.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace mspec {
namespace {

constexpr int kGroups = 3;
constexpr int kGroupWarps = 4, kGroupThreads = kGroupWarps * 32;
constexpr int kThreads = (kGroups * kGroupWarps + 1) * 32;
constexpr int kMaxS = 8, kMaxR = 12;
constexpr int kJTable = 1024;   // sequences whose pending length is kept in shared memory
constexpr int kW = 4;           // conv width handled here
constexpr int kMaxT = 16;       // token rows per sequence handled here
constexpr int kMaxJ = 8;
constexpr int kMaxHeads = 256;  // A and D of all heads are kept in shared memory
#ifndef MSPEC_WAIT_LIMIT_CYCLES
#define MSPEC_WAIT_LIMIT_CYCLES 4000000000ll   // a wait that lasts about 2 s is reported, not sat out
#endif
constexpr long long kWaitLimitCycles = MSPEC_WAIT_LIMIT_CYCLES;

struct Ctrl {
    unsigned long long state_full[kMaxS], state_empty[kMaxS];
    unsigned long long raw_full[kMaxR], raw_empty[kMaxR];
    int abort;
    int state_par[kMaxS];  // parity of the producer's last fill of each state stage, -1 before any
    int raw_par[kMaxR];    // the same for the raw stages
    int jarr[kJTable];
    float A[kMaxHeads], D[kMaxHeads];
    int walk[1 + 8 + 4 * kGroups];   // a WalkInfo, see below
};
constexpr int kCtrlBytes = (sizeof(Ctrl) + 127) / 128 * 128;

// Per-chunk scalars of one head, private to a compute group.
struct HeadConst {
    float alpha[kMaxT];  // prod_{r<=t} a_r
    float wsp[kMaxJ];    // dt_s prod_{s<r<j} a_r
    float alpha_j;       // prod_{r<j} a_r
    float D;
    float alpha_jT;      // prod_{j<=r<T} a_r             (second snapshot only)
    float pad[5];
    float wspT[kMaxT];   // dt_s prod_{s<r<T} a_r, s >= j  (second snapshot only)
};
static_assert(sizeof(HeadConst) % 16 == 0, "HeadConst must keep 16-byte alignment");
static_assert(sizeof(CUtensorMap) == sizeof(TensorMapBytes), "a tensor map is 128 bytes");

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Same, letting the hardware park the thread for up to `hint_ns` while the phase is incomplete.
__device__ __forceinline__ bool mbar_try_park(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Slow path of a wait, kept out of line so that the many wait sites stay small.  Waiting threads are
// parked by the hardware, not spun.  False if the phase did not complete within the cycle limit or
// another role gave up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const volatile int *abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_park(bar, parity, 20000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitLimitCycles) return false;
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int *abort_flag) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag);
}
// Global -> shared bulk copy through the TMA engine; src, dst and bytes are multiples of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// 2-D tiled TMA load (no multicast): box at element coordinates (x, y) of the tensor map -> shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
// 3-D tiled TMA load / store (no multicast) of the box at element coordinates (x, y, z).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int x, int y, int z, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
                 "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map), "r"(src),
                 "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until the executing thread's bulk stores have finished READING shared memory.
__device__ __forceinline__ void bulk_wait_group_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ float bf16_bits_to_f32(uint32_t lo16) { return __uint_as_float(lo16 << 16); }
// SiLU from the hardware exp2 and reciprocal approximations (relative error about 3e-7, far inside the
// fp32 tolerance of the outputs): a handful of instructions.
__device__ __forceinline__ float silu_fast(float v) { return __fdividef(v, 1.0f + __expf(-v)); }

// D += A B for a 16 x 16 (row-major) by 16 x 8 (column-major) pair of bf16 fragments, fp32 accumulators.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ const CUtensorMap *as_map(const TensorMapBytes *m) { return reinterpret_cast<const CUtensorMap *>(m); }
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 lo2(const float4 &v) { return make_float2(v.x, v.y); }
__device__ __forceinline__ float2 hi2(const float4 &v) { return make_float2(v.z, v.w); }

// ---------------------------------------------------------------- chunk enumeration
// CTA i owns chunks i, i + gridDim.x, ..., which mixes sequences (and so chunks with and without a
// state write) evenly over the CTAs; its `it`-th chunk goes through stage it % S of the state ring and
// it % R of the raw ring and is computed by group it % ngroups.  Positions are advanced incrementally:
// the divisions that decompose a chunk index into (sequence, head, chunk-of-head) are done once per
// CTA by one thread and left in shared memory.
struct Pos {
    int q, b, h, rc;
};
struct Step {
    int dq, db, dh, drc;
};
struct WalkInfo {
    int nmine;               // chunks of this CTA
    Step one, grp;           // gridDim.x chunks; gridDim.x * ngroups chunks
    Pos start[kGroups];      // first chunk of every compute group (start[0] is the CTA's first chunk)
};
static_assert(sizeof(WalkInfo) <= sizeof(int) * (1 + 8 + 4 * kGroups), "Ctrl::walk too small");
__device__ __forceinline__ Pos decompose(int q, int H, int cph) {
    Pos x;
    x.q = q;
    x.rc = q % cph;
    x.h = (q / cph) % H;
    x.b = q / (cph * H);
    return x;
}
__device__ __forceinline__ void advance(Pos &x, const Step &d, int H, int cph) {
    x.q += d.dq;
    x.rc += d.drc;
    if (x.rc >= cph) { x.rc -= cph; ++x.h; }
    x.h += d.dh;
    if (x.h >= H) { x.h -= H; ++x.b; }
    x.b += d.db;
}
__device__ __forceinline__ void ring_advance(int &idx, int &par, int n, int size) {
    idx += n;
    while (idx >= size) { idx -= size; par ^= 1; }
}
__device__ __forceinline__ int pending_of(const VerifyParams &p, const Ctrl &ctl, int b) {
    return b < kJTable ? ctl.jarr[b] : load_n_prev(p, b);
}

// ---------------------------------------------------------------- producer
// Requests the small inputs of one chunk: nine TMA requests issued by nine lanes (x, z, B, C, dt and
// the conv window through tensor maps, each covering all TCAP token rows; taps and bias as plain bulk
// copies).  Rows beyond the sequence's T tokens are fetched but never used.
template <int N, int CR, bool EXT>
__device__ __forceinline__ bool issue_raw(const VerifyParams &p, const StreamLayout &L, const InputMaps &tm,
                                          uint32_t smem_base, Ctrl &ctl, int rs, int rp, int b, int h, int rc, int lane) {
    if (!mbar_wait(smem_u32(&ctl.raw_empty[rs]), (uint32_t)rp ^ 1u, &ctl.abort)) return false;
    const uint32_t raw = smem_base + L.raw_off + rs * L.raw_stride, bar = smem_u32(&ctl.raw_full[rs]);
    const int c0 = h * p.P + rc * CR, row0 = b * p.t_max + (EXT ? first_row(p, b) : 0);
#ifdef MSPEC_TEST_RAW_NEVER_FULL
    // Test build only: one transaction byte more is expected than is requested, so every copy lands and the
    // barrier still never completes -- the consumers' bounded wait runs out.
    if (lane == 0) { ctl.raw_par[rs] = rp; mbar_arrive_expect_tx(bar, (uint32_t)L.raw_tx + 16u); }
#else
    if (lane == 0) { ctl.raw_par[rs] = rp; mbar_arrive_expect_tx(bar, (uint32_t)L.raw_tx); }
#endif
    __syncwarp();
    // One tensor-load instruction for the six 2-D boxes (lane l takes map l of InputMaps: x, z, B, C, dt,
    // conv window) and one bulk-copy instruction for taps and bias: issued convergently, the requests queue
    // up in the TMA unit instead of costing the warp one issue round trip each.
    if (lane < 6) {
        const int cx = lane <= 1 ? c0 : lane == 2 ? (int)((h + 0.5f) * L.inv_hpg_b) * N
                                     : lane == 3 ? (int)((h + 0.5f) * L.inv_hpg_c) * N : lane == 4 ? (h & ~7) : c0;
        const int cy = lane == 5 ? b * (kW - 1) : row0;
        const uint32_t dst = raw + (lane == 0 ? L.r_x : lane == 1 ? L.r_z : lane == 2 ? L.r_B : lane == 3 ? L.r_C
                                                                   : lane == 4 ? L.r_dt : L.r_cst);
        // (commit-selects mode: the conv window comes from whichever buffer holds this sequence's cache)
        const TensorMapBytes *map = (EXT && lane == 5 && p.sel != nullptr && p.sel[b] != 0) ? &tm.cst_k : &tm.x + lane;
        if (lane != 1 || p.z != nullptr) tma_load_2d(dst, as_map(map), cx, cy, bar);
    } else if (lane < 8) {
        const bool taps = lane == 6;
        bulk_g2s(raw + (taps ? L.r_cw : L.r_cb), taps ? (const void *)(p.conv_w + (size_t)c0 * kW) : (const void *)(p.conv_b + c0),
                 taps ? CR * kW * 4 : CR * 4, bar);
    }
    return true;
}

// The small inputs of a chunk are requested `lead` chunks before its state rows: they feed the
// prologue, whose results are needed at the moment the state lands.
template <int N, int CR, bool EXT>
__device__ __forceinline__ void producer_role(const VerifyParams &p, const StreamLayout &L, unsigned char *smem,
                                              Ctrl &ctl, const InputMaps &tm, int lane) {
    constexpr uint32_t kStateBytes = CR * N * 4;
    const uint32_t smem_base = smem_u32(smem);
    const WalkInfo &wi = *reinterpret_cast<const WalkInfo *>(ctl.walk);
    const int H = p.H, cph = p.P / CR, nmine = wi.nmine;
    Pos ps = wi.start[0], pr = wi.start[0];   // state position and the raw position that runs ahead of it
    int ss = 0, sp = 0, rs = 0, rp = 0, itr = 0;
    for (int it = 0; it < nmine; ++it) {
        const int rlim = it + L.lead + 1 < nmine ? it + L.lead + 1 : nmine;
        for (; itr < rlim; ++itr) {
            if (!issue_raw<N, CR, EXT>(p, L, tm, smem_base, ctl, rs, rp, pr.b, pr.h, pr.rc, lane)) {
                atomicOr(p.status, kStatusCopyTimeout);
                ctl.abort = 1;
                return;
            }
            advance(pr, wi.one, H, cph);
            ring_advance(rs, rp, 1, L.R);
        }
        {
            if (!mbar_wait(smem_u32(&ctl.state_empty[ss]), (uint32_t)sp ^ 1u, &ctl.abort)) {
                atomicOr(p.status, kStatusCopyTimeout);
                ctl.abort = 1;
                return;
            }
            if (lane == 0) {
                const uint32_t sbar = smem_u32(&ctl.state_full[ss]);
                ctl.state_par[ss] = sp;
                mbar_arrive_expect_tx(sbar, kStateBytes);
                const bool swapped = EXT && p.sel != nullptr && p.sel[ps.b] != 0;   // commit-selects mode: where this sequence's cache is
                tma_load_3d(smem_base + L.state_off + ss * L.state_stride, as_map(swapped ? &tm.state_k : &tm.state), 0, ps.q * CR, 0, sbar);
            }
        }
        advance(ps, wi.one, H, cph);
        ring_advance(ss, sp, 1, L.S);
    }
}

// ---------------------------------------------------------------- prologue phase of a compute group
// Everything of one chunk that does not need the state, left in the group's buffer `gb`.  The jobs are
// independent of one another (each reads only the raw inputs), so there is no barrier inside: the
// caller's barrier before the stream phase orders all of it.  The jobs are dealt to the four warps so that
// they finish together, and written for short dependent chains: the kernel is bound by latency, not by
// arithmetic.
//   pairs   G[t][s] = (C_t . B_s) dt_s prod_{s<r<=t} a_r for s <= t (+ D_h on the diagonal), by the last
//           warp with matrix instructions straight from the bf16 rows; the decay product is one exp of
//           A_h sum_{s<r<=t} dt_r (Sec. 2.2: a_r = exp(dt_r A_h))
//   conv    xc_t = SiLU(causal conv) of the rolling window, thread = (token class, row pair)
//   gate    SiLU(z_t), same mapping; conv window at position j -> global (Sec. 4.3 iii)
//   rows    fp32 copies of the C rows and of the B rows s < j, which the stream phase reads as broadcasts
//   decay   alpha_t, wsp_s, alpha_j by the lanes of the warp before the last
template <int N, int CR, bool SNAP, bool EXT>
__device__ __forceinline__ void prologue_phase(const VerifyParams &p, const StreamLayout &L, const unsigned char *raw,
                                               unsigned char *gb, int b, int h, int rc, int j, int T,
                                               float A_of_head, float D_of_head, int gtid, bool swapped) {
    constexpr int HR = CR / 2;      // row pairs
    constexpr int CPR = N / 8;      // 16-byte pieces (8 bf16) per B or C row
    const int H = p.H, P = p.P;
    const bool gate = p.z != nullptr, conv_silu = (p.flags & kFlagConvSilu) != 0;
    const int pw = gtid >> 5, lane = gtid & 31;
    HeadConst *hc = reinterpret_cast<HeadConst *>(gb + L.c_hc);
    float *Gm = reinterpret_cast<float *>(gb + L.c_G);    // [kMaxT][kMaxT], entries s <= t < T
    float *xcs = reinterpret_cast<float *>(gb + L.c_xc);  // [t][CR]
    const unsigned short *dtr = reinterpret_cast<const unsigned short *>(raw + L.r_dt) + (h & 7);   // dt_t at [t * 8]
    // the sampling interval of token r: as it arrives, or softplus(raw + bias) when it arrives raw (Sec. 2.2)
    const bool dt_raw = EXT && (p.flags & kFlagDtSoftplus) != 0;
    const float dt_b = (dt_raw && p.dt_bias != nullptr) ? p.dt_bias[h] : 0.f;
    auto dt_at = [&](int r) {
        const float v = bf16_bits_to_f32(dtr[r * 8]);
        return dt_raw ? softplus_f(v + dt_b) : v;
    };
    const uint32_t *cs32 = reinterpret_cast<const uint32_t *>(raw + L.r_cst), *xs32 = reinterpret_cast<const uint32_t *>(raw + L.r_x);

    // ---- pairs, by the last warp: the T x T products C_t . B_s are a small bf16 matrix product, exact in
    //      fp32, formed with warp-level matrix instructions (16 x 8 x 16 per instruction; thread (g, tq) =
    //      (lane / 4, lane % 4) supplies rows g and g + 8 of C, row g of a block of eight B rows, and of
    //      every 32 columns the eight columns 8 tq .. 8 tq + 7 -- the order in which the instruction walks the
    //      columns does not matter as long as both operands use the same one).  Each thread then scales
    //      its entries by dt_s prod_{s<r<=t} a_r, one exp of a difference of prefix sums of dt, and writes
    //      zeros above the diagonal and in the padding, which the output loop reads in float4 pieces.
    if (pw == kGroupWarps - 1) {
        const int g = lane >> 2, tq = lane & 3, rmax = L.TCAP - 1;
        const bool two = T > 8;
        const unsigned char *Cb = raw + L.r_C + tq * 16, *Bb = raw + L.r_B + tq * 16;
        const int r0 = g < rmax ? g : rmax, r1 = g + 8 < rmax ? g + 8 : rmax;   // rows past the buffers: never used
        float acc[2][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i >> 2][i & 3] = 0.f;
#pragma unroll
        for (int c32 = 0; c32 < N / 32; ++c32) {
            const uint4 a_lo = *reinterpret_cast<const uint4 *>(Cb + r0 * (N * 2) + c32 * 64);
            uint4 a_hi = make_uint4(0u, 0u, 0u, 0u);
            if (two) a_hi = *reinterpret_cast<const uint4 *>(Cb + r1 * (N * 2) + c32 * 64);
            const uint4 b_lo = *reinterpret_cast<const uint4 *>(Bb + r0 * (N * 2) + c32 * 64);
            mma_bf16_16816(acc[0], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b_lo.x, b_lo.y);
            mma_bf16_16816(acc[0], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b_lo.z, b_lo.w);
            if (two) {
                const uint4 b_hi = *reinterpret_cast<const uint4 *>(Bb + r1 * (N * 2) + c32 * 64);
                mma_bf16_16816(acc[1], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b_hi.x, b_hi.y);
                mma_bf16_16816(acc[1], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b_hi.z, b_hi.w);
            }
        }
        // lane r holds dt_r and E_r = sum_{r' <= r} dt_r'
        const float dtv = lane < T ? dt_at(lane) : 0.f;
        float E = dtv;
#pragma unroll
        for (int m = 1; m < kMaxT; m <<= 1) {
            const float up = __shfl_up_sync(0xffffffffu, E, m);
            if (lane >= m) E += up;
        }
        const float Et0 = __shfl_sync(0xffffffffu, E, g), Et1 = __shfl_sync(0xffffffffu, E, g + 8);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            if (nt == 1 && !two) break;
            float2 lo, hi;   // rows g and g + 8, columns s0, s0 + 1
            const int s0 = nt * 8 + 2 * tq;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int s2 = s0 + e;
                const float Es = __shfl_sync(0xffffffffu, E, s2), ds = __shfl_sync(0xffffffffu, dtv, s2);
                float v0 = (s2 <= g && g < T) ? acc[nt][e] * ds * expf(A_of_head * (Et0 - Es)) : 0.f;
                float v1 = (s2 <= g + 8 && g + 8 < T) ? acc[nt][2 + e] * ds * expf(A_of_head * (Et1 - Es)) : 0.f;
                if (s2 == g) v0 += D_of_head;   // the skip term D xc_t rides on the diagonal
                if (s2 == g + 8) v1 += D_of_head;
                if (e == 0) { lo.x = v0; hi.x = v1; } else { lo.y = v0; hi.y = v1; }
            }
            *reinterpret_cast<float2 *>(Gm + g * kMaxT + s0) = lo;
            if (two) *reinterpret_cast<float2 *>(Gm + (g + 8) * kMaxT + s0) = hi;
        }
    }

    // ---- conv and gate: warp w takes the tokens t = w (mod 4) -- the last warp, which has the pairs, the
    //      fewest -- and lane = row pair
    if (lane < HR) {
        const float4 wa = reinterpret_cast<const float4 *>(raw + L.r_cw)[2 * lane], wb = reinterpret_cast<const float4 *>(raw + L.r_cw)[2 * lane + 1];
        const float2 bias = reinterpret_cast<const float2 *>(raw + L.r_cb)[lane];
        const uint32_t *zs32 = reinterpret_cast<const uint32_t *>(raw + L.r_z);
        float2 *gz = reinterpret_cast<float2 *>(gb + L.c_gz);
#pragma unroll 2
        for (int t = pw; t < T; t += kGroupWarps) {
            // inputs t-3 .. t: the cached window covers the negative positions
            const uint32_t r0 = t >= 3 ? xs32[(t - 3) * HR + lane] : cs32[t * HR + lane];
            const uint32_t r1 = t >= 2 ? xs32[(t - 2) * HR + lane] : cs32[(t + 1) * HR + lane];
            const uint32_t r2 = t >= 1 ? xs32[(t - 1) * HR + lane] : cs32[(t + 2) * HR + lane];
            const uint32_t r3 = xs32[t * HR + lane];
            float va = fmaf(wa.w, __uint_as_float(r3 << 16), fmaf(wa.z, __uint_as_float(r2 << 16),
                       fmaf(wa.y, __uint_as_float(r1 << 16), fmaf(wa.x, __uint_as_float(r0 << 16), bias.x))));
            float vb = fmaf(wb.w, __uint_as_float(r3 & 0xffff0000u), fmaf(wb.z, __uint_as_float(r2 & 0xffff0000u),
                       fmaf(wb.y, __uint_as_float(r1 & 0xffff0000u), fmaf(wb.x, __uint_as_float(r0 & 0xffff0000u), bias.y))));
            if (conv_silu) { va = silu_fast(va); vb = silu_fast(vb); }
            reinterpret_cast<float2 *>(xcs)[t * HR + lane] = make_float2(va, vb);
            if (gate) {
                const uint32_t r = zs32[t * HR + lane];
                gz[t * HR + lane] = make_float2(silu_fast(__uint_as_float(r << 16)), silu_fast(__uint_as_float(r & 0xffff0000u)));
            }
        }
        if (pw == 0)   // zero rows up to the next multiple of four tokens (read, times zero, by the output loop)
            for (int t = T; t < ((T + 3) & ~3); ++t) reinterpret_cast<float2 *>(xcs)[t * HR + lane] = make_float2(0.f, 0.f);
        if (j > 0 && pw < kW - 1) {  // the last W-1 inputs up to token j-1 become the cached window: warp i writes slot i
            uint32_t *out = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned short *>(swapped ? p.conv_state_k : p.conv_state) +
                                                         (size_t)b * (kW - 1) * (H * P) + h * P + rc * CR) + lane;
            const int tau = j - (kW - 1) + pw;
            out[(size_t)pw * (H * P / 2)] = tau < 0 ? cs32[(kW - 1 + tau) * HR + lane] : xs32[tau * HR + lane];
        }
        if (SNAP && pw < kW - 1) {  // second snapshot: the window after all T tokens
            uint32_t *out = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned short *>(swapped ? p.conv_state : p.conv_state_k) +
                                                         (size_t)b * (kW - 1) * (H * P) + h * P + rc * CR) + lane;
            const int tau = T - (kW - 1) + pw;
            out[(size_t)pw * (H * P / 2)] = tau < 0 ? cs32[(kW - 1 + tau) * HR + lane] : xs32[tau * HR + lane];
        }
    }

    // ---- fp32 copies of the C rows (all tokens) and of the B rows s < j, eight columns per thread
    {
        const int row0 = gtid / CPR, c = gtid % CPR;
        float *Cf = reinterpret_cast<float *>(gb + L.c_Cf), *Bf = reinterpret_cast<float *>(gb + L.c_Bf);
#pragma unroll 2
        for (int t = row0; t < T; t += kGroupThreads / CPR) {
            const uint4 v = reinterpret_cast<const uint4 *>(raw + L.r_C + t * (N * 2))[c];
            float4 *dst = reinterpret_cast<float4 *>(Cf + t * N + c * 8);
            dst[0] = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
            dst[1] = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u), __uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
        }
        const int nB = SNAP ? T : j;   // the second snapshot replays all tokens
        for (int t = row0; t < nB; t += kGroupThreads / CPR) {
            const uint4 v = reinterpret_cast<const uint4 *>(raw + L.r_B + t * (N * 2))[c];
            float4 *dst = reinterpret_cast<float4 *>(Bf + t * N + c * 8);
            dst[0] = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
            dst[1] = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u), __uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
        }
    }

    // ---- decay products, by the warp before the last (the last has the pairs): lane t < T: alpha_t = exp(A_h sum_{r<=t} dt_r); lane 16+s, s < j:
    //      wsp_s = dt_s exp(A_h sum_{s<r<j} dt_r); lane 31: alpha_j = exp(A_h sum_{r<j} dt_r), and D
    if (pw == kGroupWarps - 2) {
        const bool is_wsp = lane >= 16 && lane - 16 < j && lane - 16 < kMaxJ;
        const int lo = is_wsp ? lane - 15 : 0;
        const int hi = lane < 16 ? (lane < T ? lane + 1 : 0) : ((is_wsp || lane == 31) ? j : 0);
        float sum = 0.f;   // every lane walks all T tokens (uniform broadcast loads, nothing to wait for in turn)
#pragma unroll 4
        for (int r = 0; r < T; ++r) {
            const float v = dt_at(r);
            sum += (r >= lo && r < hi) ? v : 0.f;
        }
        const float ex = expf(A_of_head * sum);
        if (lane < T && lane < 16) hc->alpha[lane] = ex;
        if (is_wsp) hc->wsp[lane - 16] = dt_at(lane - 16) * ex;
        if (lane == 31) {
            hc->alpha_j = ex;
            hc->D = D_of_head;
        }
        if (SNAP) {   // second snapshot: from position j on to the end of the block
            const int lo2 = lane < 16 ? lane + 1 : j, hi2 = (lane < 16 ? (lane >= j && lane < T) : lane == 31) ? T : 0;
            float sum2 = 0.f;
#pragma unroll 4
            for (int r = 0; r < T; ++r) {
                const float v = dt_at(r);
                sum2 += (r >= lo2 && r < hi2) ? v : 0.f;
            }
            const float ex2 = expf(A_of_head * sum2);
            if (lane < 16 && lane >= j && lane < T) hc->wspT[lane] = dt_at(lane) * ex2;
            if (lane == 31) hc->alpha_jT = ex2;
        }
    }
}

// ---------------------------------------------------------------- stream phase of a compute group
// The state chunk sits in shared memory as the TMA engine wrote it: 32-column quarters of the rows,
// quarter-major ([quarter][row][32 floats], 128 bytes per line) with the 128-byte swizzle, so that
// the threads of a warp -- one per row -- read 16-byte pieces of 32 different rows without bank
// conflicts.  Warp w of the group owns column quarter w % NQ; a thread owns RPT rows and holds its
// 32 columns of them in registers.  Per token the row's partial dot product with C_t (read as warp
// broadcasts) goes to shared memory; after a group barrier the quarters are summed and y is formed
// with fully coalesced stores.  Where tokens were accepted the state at position j is formed in the
// same registers, written back into the stage and stored to global memory by one TMA request.
template <int N, int CR, bool SNAP, bool EXT>
__device__ __forceinline__ bool stream_phase(const VerifyParams &p, const StreamLayout &L, const InputMaps &tm,
                                             unsigned char *st, unsigned char *gb, uint32_t empty_bar, int bar_id, int q,
                                             int b, int h, int rc, int j, int T, int gtid, bool swapped) {
    constexpr int NQ = N / 32;                                  // column quarters of a row
    constexpr int RBK = kGroupWarps / NQ;                       // row blocks (warps per quarter)
    constexpr int RPT = (CR / (32 * RBK)) > 0 ? CR / (32 * RBK) : 1;  // rows per thread
    constexpr int LGCR = (CR == 64) ? 6 : 5;
    const int warp = gtid >> 5, lane = gtid & 31, qq = warp % NQ, rblk = warp / NQ;
    const int rbase = rblk * 32 * RPT + lane;
    const bool active = rblk * 32 * RPT < CR;   // warp-uniform
    const bool gate = p.z != nullptr, y_f32 = (p.flags & kFlagYF32) != 0;
    const HeadConst *hc = reinterpret_cast<const HeadConst *>(gb + L.c_hc);
    float *part = reinterpret_cast<float *>(gb + L.c_part);   // [NQ][TCAP][CR]

    float4 hv[RPT][8];
    if (active) {
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const int row = rbase + 32 * i;
            const unsigned char *line = st + (size_t)(qq * CR + row) * 128;
#pragma unroll
            for (int k = 0; k < 8; ++k) hv[i][k] = *reinterpret_cast<const float4 *>(line + ((k ^ (row & 7)) << 4));
        }
    }
    constexpr bool snap2 = SNAP;   // second snapshot compiled in (a kernel variant of its own)
    if (j == 0 && !snap2) {   // nothing is written back: the stage is free as soon as the rows are in registers
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar);
    }
    if (active) {
#pragma unroll 2
        for (int t = 0; t < T; ++t) {
            const float4 *crow = reinterpret_cast<const float4 *>(gb + L.c_Cf + (size_t)t * (N * 4)) + qq * 8;
            float2 a0[RPT], a1[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) a0[i] = a1[i] = make_float2(0.f, 0.f);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float4 cv = crow[k];
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    a0[i] = ffma2(lo2(hv[i][k]), lo2(cv), a0[i]);
                    a1[i] = ffma2(hi2(hv[i][k]), hi2(cv), a1[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < RPT; ++i)
                part[((qq * L.TCAP + t) << LGCR) + rbase + 32 * i] = (a0[i].x + a0[i].y) + (a1[i].x + a1[i].y);
        }
        if (j > 0) {  // state at the verified position (Sec. 4.3 iii), formed in place
            const float *xcs = reinterpret_cast<const float *>(gb + L.c_xc);
            const float aj = hc->alpha_j;
            const float2 aj2 = make_float2(aj, aj);
#pragma unroll
            for (int i = 0; i < RPT; ++i)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float2 l = __fmul2_rn(lo2(hv[i][k]), aj2), h2 = __fmul2_rn(hi2(hv[i][k]), aj2);
                    hv[i][k] = make_float4(l.x, l.y, h2.x, h2.y);
                }
#pragma unroll 1
            for (int s = 0; s < j; ++s) {
                const float4 *brow = reinterpret_cast<const float4 *>(gb + L.c_Bf + (size_t)s * (N * 4)) + qq * 8;
                float2 cf[RPT];
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    const float c = hc->wsp[s] * xcs[(s << LGCR) + rbase + 32 * i];   // wsp_s xc_s[p]
                    cf[i] = make_float2(c, c);
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float4 bv = brow[k];
#pragma unroll
                    for (int i = 0; i < RPT; ++i) {
                        const float2 l = ffma2(cf[i], lo2(bv), lo2(hv[i][k])), h2 = ffma2(cf[i], hi2(bv), hi2(hv[i][k]));
                        hv[i][k] = make_float4(l.x, l.y, h2.x, h2.y);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int row = rbase + 32 * i;
                unsigned char *line = st + (size_t)(qq * CR + row) * 128;
#pragma unroll
                for (int k = 0; k < 8; ++k) *reinterpret_cast<float4 *>(line + ((k ^ (row & 7)) << 4)) = hv[i][k];
            }
            fence_proxy_async();   // the TMA store below reads what was just written
        }
    }
    named_bar_sync(bar_id, kGroupThreads);   // partial sums and (if any) the new state are in shared memory
    if (j > 0 && gtid == 0) {
        tma_store_3d(as_map(swapped ? &tm.state_k : &tm.state), smem_u32(st), 0, q * CR, 0);
        bulk_commit_group();
    }
    if (snap2) {
        // Second snapshot (Algorithm 2 caches h_j and h_k): carry the registers on from position j to the end
        // of the block, h_T = (prod_{j<=r<T} a_r) h_j + sum_{j<=s<T} (dt_s prod_{s<r<T} a_r) xc_s B_s, put the
        // result into the stage once the first store has read it, and store it to the second buffer.
        if (gtid == 0 && j > 0) bulk_wait_group_read0();
        if (active) {
            const float *xcs = reinterpret_cast<const float *>(gb + L.c_xc);
            const float aT = hc->alpha_jT;
            const float2 aT2 = make_float2(aT, aT);
#pragma unroll
            for (int i = 0; i < RPT; ++i)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float2 l = __fmul2_rn(lo2(hv[i][k]), aT2), h2 = __fmul2_rn(hi2(hv[i][k]), aT2);
                    hv[i][k] = make_float4(l.x, l.y, h2.x, h2.y);
                }
#pragma unroll 1
            for (int s = j; s < T; ++s) {
                const float4 *brow = reinterpret_cast<const float4 *>(gb + L.c_Bf + (size_t)s * (N * 4)) + qq * 8;
                float2 cf[RPT];
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    const float c = hc->wspT[s] * xcs[(s << LGCR) + rbase + 32 * i];
                    cf[i] = make_float2(c, c);
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float4 bv = brow[k];
#pragma unroll
                    for (int i = 0; i < RPT; ++i) {
                        const float2 l = ffma2(cf[i], lo2(bv), lo2(hv[i][k])), h2 = ffma2(cf[i], hi2(bv), hi2(hv[i][k]));
                        hv[i][k] = make_float4(l.x, l.y, h2.x, h2.y);
                    }
                }
            }
        }
        named_bar_sync(bar_id, kGroupThreads);   // the first store has read the stage (thread 0 waited above)
        if (active) {
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int row = rbase + 32 * i;
                unsigned char *line = st + (size_t)(qq * CR + row) * 128;
#pragma unroll
                for (int k = 0; k < 8; ++k) *reinterpret_cast<float4 *>(line + ((k ^ (row & 7)) << 4)) = hv[i][k];
            }
            fence_proxy_async();
        }
        named_bar_sync(bar_id, kGroupThreads);
        if (gtid == 0) {
            tma_store_3d(as_map(swapped ? &tm.state : &tm.state_k), smem_u32(st), 0, q * CR, 0);
            bulk_commit_group();
        }
    }
    // ---- outputs: y_t[p] = alpha_t (C_t . h[p,:]) + sum_{s<=t} G[t][s] xc_s[p] + D xc_t[p], gated;
    //      element (t, row) per thread, rows contiguous; the prologue has put D on the diagonal of G
    {
        const float *xcs = reinterpret_cast<const float *>(gb + L.c_xc), *gz = reinterpret_cast<const float *>(gb + L.c_gz);
        const float *Gm = reinterpret_cast<const float *>(gb + L.c_G);
        // (with new rows only, y is [batch][k]: token j is its row 0 and the replayed rows' outputs are dropped)
        const bool y_new = EXT && (p.flags & kFlagYNewOnly) != 0;
        const size_t y0 = (((size_t)b * (y_new ? p.k : p.t_max) - (y_new ? j : 0) + ((y_new || !EXT) ? 0 : first_row(p, b))) * p.H + h) * p.P + rc * CR;
        const size_t tstride = (size_t)p.H * p.P;
        // a thread's elements share their row (the group's thread count is a multiple of CR): its xc values
        // are read once; D sits on the diagonal of G
        static_assert(kGroupThreads % CR == 0, "elements of a thread share a row");
        const int row = gtid & (CR - 1), TR = (T + 3) & ~3;
        float xr[kMaxT];
#pragma unroll
        for (int s = 0; s < kMaxT; ++s) xr[s] = s < TR ? xcs[(s << LGCR) + row] : 0.f;
#pragma unroll 2
        for (int t = gtid >> LGCR; t < T; t += kGroupThreads / CR) {
            const int e = (t << LGCR) + row;
            float v = part[e];
#pragma unroll
            for (int c = 1; c < NQ; ++c) v += part[((c * L.TCAP) << LGCR) + e];
            float w = 0.f;
#pragma unroll
            for (int s4 = 0; s4 < kMaxT; s4 += 4) {   // G is zero above the diagonal; xc rows up to a multiple of four exist
                if (s4 <= t) {
                    const float4 g4 = *reinterpret_cast<const float4 *>(Gm + t * kMaxT + s4);
                    w = fmaf(g4.x, xr[s4], w);
                    w = fmaf(g4.y, xr[s4 + 1], w);
                    w = fmaf(g4.z, xr[s4 + 2], w);
                    w = fmaf(g4.w, xr[s4 + 3], w);
                }
            }
            float y = fmaf(hc->alpha[t], v, w);
            if (gate) y *= gz[e];
            const size_t yi = y0 + t * tstride + row;
            if (y_new && t < j) continue;
            if (y_f32) reinterpret_cast<float *>(p.y)[yi] = y;
            else reinterpret_cast<__nv_bfloat16 *>(p.y)[yi] = __float2bfloat16_rn(y);
        }
    }
    // the stage may be refilled once the store has read it: the caller waits for that later, off the
    // critical path (release_stage)
    return (j > 0 || snap2) && gtid == 0;
}
__device__ __forceinline__ void release_stage(uint32_t empty_bar) {
    bulk_wait_group_read0();
    mbar_arrive_n(empty_bar, kGroupWarps);
}

// Barrier over the `n` threads of a compute group that also ANDs a predicate, so that a wait that gave
// up is seen by the whole group and nobody is left behind at the next barrier.
__device__ __forceinline__ bool named_bar_and(int id, int n, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %3, 0;\n\t"
        "bar.red.and.pred p, %1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(n), "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}

template <int N, int CR, bool SNAP, bool EXT>
__device__ __forceinline__ void compute_role(const VerifyParams &p, const StreamLayout &L, unsigned char *smem, Ctrl &ctl,
                                             const InputMaps &tm, int group, int gtid) {
    const int lane = gtid & 31, bar_id = 1 + group;
    unsigned char *gb = smem + L.grp_off + (size_t)group * L.grp_stride;
    if (group >= L.ngroups) return;   // long token blocks leave room for fewer group buffers
    const WalkInfo &wi = *reinterpret_cast<const WalkInfo *>(ctl.walk);
    const int H = p.H, cph = p.P / CR, nmine = wi.nmine;
    Pos x = wi.start[group];
    int ss = 0, sp = 0, rs = 0, rp = 0, it = group;
    bool store_pending = false;   // this thread's TMA store of the previous chunk may still be reading its stage
    uint32_t pending_bar = 0;
    ring_advance(ss, sp, group, L.S);
    ring_advance(rs, rp, group, L.R);
    for (; it < nmine; it += L.ngroups) {
        const int j = pending_of(p, ctl, x.b), T = j + p.k;
        const bool swapped = EXT && SNAP && p.sel != nullptr && p.sel[x.b] != 0;   // commit-selects mode: the cache is in the second buffers
        // the group's buffer is free once every warp has left the previous chunk; the inputs must be in
        bool ok = mbar_wait(smem_u32(&ctl.raw_full[rs]), (uint32_t)rp, &ctl.abort);
        ok = named_bar_and(bar_id, kGroupThreads, ok);
        if (!ok) break;
        if (store_pending) { release_stage(pending_bar); store_pending = false; }
        const unsigned char *raw = smem + L.raw_off + (size_t)rs * L.raw_stride;
        prologue_phase<N, CR, SNAP, EXT>(p, L, raw, gb, x.b, x.h, x.rc, j, T, ctl.A[x.h], ctl.D[x.h], gtid, swapped);
        ok = mbar_wait(smem_u32(&ctl.state_full[ss]), (uint32_t)sp, &ctl.abort);
        ok = named_bar_and(bar_id, kGroupThreads, ok);   // also: the group's buffer is complete
        if (lane == 0) mbar_arrive(smem_u32(&ctl.raw_empty[rs]));
        if (!ok) break;
        unsigned char *st = smem + L.state_off + (size_t)ss * L.state_stride;
        pending_bar = smem_u32(&ctl.state_empty[ss]);
        store_pending = stream_phase<N, CR, SNAP, EXT>(p, L, tm, st, gb, pending_bar, bar_id, x.q, x.b, x.h, x.rc, j, T, gtid, swapped);
        advance(x, wi.grp, H, cph);
        ring_advance(ss, sp, L.ngroups, L.S);
        ring_advance(rs, rp, L.ngroups, L.R);
    }
    if (store_pending) release_stage(pending_bar);   // also keeps shared memory alive until the last store has read it
    if (ctl.abort == 0 && it < nmine) {   // left the loop because a wait gave up
        atomicOr(p.status, kStatusCopyTimeout);
        ctl.abort = 1;
    }
}

// ---------------------------------------------------------------- the kernel
template <int N, int CR, bool SNAP, bool EXT>
__global__ void __launch_bounds__(kThreads, 1)
verify_stream_kernel(const __grid_constant__ VerifyParams p, const __grid_constant__ StreamLayout L,
                     const __grid_constant__ InputMaps tm) {
    extern __shared__ __align__(1024) unsigned char smem[];
    Ctrl &ctl = *reinterpret_cast<Ctrl *>(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cph = p.P / CR;
    const int nchunks = p.batch * p.H * cph;   // the planner keeps this below 2^30
    if ((int)blockIdx.x >= nchunks) return;
    if (tid == 0) {
        for (int s = 0; s < L.S; ++s) {
            mbar_init(smem_u32(&ctl.state_full[s]), 1);
            mbar_init(smem_u32(&ctl.state_empty[s]), kGroupWarps);
        }
        for (int s = 0; s < L.R; ++s) {
            mbar_init(smem_u32(&ctl.raw_full[s]), 1);
            mbar_init(smem_u32(&ctl.raw_empty[s]), kGroupWarps);
        }
        for (int s = 0; s < kMaxS; ++s) ctl.state_par[s] = -1;
        for (int s = 0; s < kMaxR; ++s) ctl.raw_par[s] = -1;
        ctl.abort = 0;
        fence_mbar_init();
        WalkInfo &wi = *reinterpret_cast<WalkInfo *>(ctl.walk);
        const int G = (int)gridDim.x, H = p.H;
        wi.nmine = (nchunks - (int)blockIdx.x + G - 1) / G;
        const Pos one = decompose(G, H, cph), grp = decompose(G * L.ngroups, H, cph);
        wi.one = Step{one.q, one.b, one.h, one.rc};
        wi.grp = Step{grp.q, grp.b, grp.h, grp.rc};
        for (int g = 0; g < kGroups; ++g) wi.start[g] = decompose((int)blockIdx.x + g * G, H, cph);
    }
    __syncthreads();
    const bool is_producer = warp == kThreads / 32 - 1;
    // Nothing reads global memory before everything launched earlier in the stream has completed; only the
    // set-up above overlaps with the previous kernel's tail, and L2 prefetches of what the first chunk reads
    // first (no architectural effect: they take cold misses off the path).  First state requests ahead of the
    // wait, for callers that can promise an unrelated previous kernel, were measured and lost 5 %.
    if (is_producer) {
        // the nine tensor maps into the descriptor cache, so that the first requests do not wait for them
        if (lane < 9) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<const void *>(&tm.x + lane)) : "memory");
        const WalkInfo &wi = *reinterpret_cast<const WalkInfo *>(ctl.walk);
        const Pos x0 = wi.start[0];
        const size_t trow = ((size_t)x0.b * p.t_max + (lane < p.t_max ? lane : 0)) ;
        if (lane < L.TCAP && lane < p.t_max) {
            const char *xr = reinterpret_cast<const char *>(p.x) + ((trow * p.H + x0.h) * p.P + x0.rc * CR) * 2;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(xr));
            if (p.z) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.z) + (xr - reinterpret_cast<const char *>(p.x))));
            const char *br = reinterpret_cast<const char *>(p.B) + ((trow * p.GB + (int)((x0.h + 0.5f) * L.inv_hpg_b)) * N) * 2;
            const char *cr = reinterpret_cast<const char *>(p.C) + ((trow * p.GC + (int)((x0.h + 0.5f) * L.inv_hpg_c)) * N) * 2;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(br));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(cr));
            if (N == 128) {
                asm volatile("prefetch.global.L2 [%0];" ::"l"(br + 128));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(cr + 128));
            }
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.dt) + (trow * p.H + x0.h) * 2));
        } else if (lane >= 16 && lane < 16 + kW - 1) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.conv_state) + (((size_t)x0.b * (kW - 1) + (lane - 16)) * p.H * p.P + x0.h * p.P + x0.rc * CR) * 2));
        } else if (lane == 20) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.n_prev));
        } else if (lane == 21) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.A));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.D));
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The next kernel of the stream is let in only now, so that what it does ahead of its own wait can overlap
    // with this kernel but with nothing older.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (is_producer) {
        producer_role<N, CR, EXT>(p, L, smem, ctl, tm, lane);
    } else {
        constexpr int kComputeThreads = kGroups * kGroupThreads;
        const int ntab = p.batch < kJTable ? p.batch : kJTable;
#pragma unroll 1
        for (int i = tid; i < ntab; i += kComputeThreads) ctl.jarr[i] = load_n_prev(p, i);
#pragma unroll 1
        for (int i = tid; i < p.H; i += kComputeThreads) { ctl.A[i] = p.A[i]; ctl.D[i] = p.D[i]; }
        named_bar_sync(15, kComputeThreads);
        compute_role<N, CR, SNAP, EXT>(p, L, smem, ctl, tm, warp / kGroupWarps, tid % kGroupThreads);
    }

    __syncthreads();
    if (ctl.abort && tid == 0) {
        // Some wait gave up.  Give every bulk copy that was started a bounded chance to land before the
        // CTA's shared memory is released.
        for (int s = 0; s < L.S; ++s) {
            const long long t0 = clock64();
            if (ctl.state_par[s] >= 0)
                while (!mbar_try_park(smem_u32(&ctl.state_full[s]), (uint32_t)ctl.state_par[s], 20000u) &&
                       clock64() - t0 < kWaitLimitCycles) {}
        }
        for (int s = 0; s < L.R; ++s) {
            const long long t0 = clock64();
            if (ctl.raw_par[s] >= 0)
                while (!mbar_try_park(smem_u32(&ctl.raw_full[s]), (uint32_t)ctl.raw_par[s], 20000u) &&
                       clock64() - t0 < kWaitLimitCycles) {}
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link libcuda).
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// bf16 matrix [rows][cols] (row-major, dense) read in boxes of box_rows x box_cols; out-of-range rows read as zero.
bool encode_2d(EncodeTiledFn fn, TensorMapBytes *map, const void *base, size_t cols, size_t rows, int box_cols, int box_rows) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(reinterpret_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// fp32 state [rows][N] as [32 columns][rows][N/32 quarters], boxes of one chunk's rows, 128-byte swizzle
bool encode_state(EncodeTiledFn fn, TensorMapBytes *map, const void *base, size_t rows, int N, int CR) {
    const cuuint64_t dims[3] = {32, (cuuint64_t)rows, (cuuint64_t)(N / 32)};
    const cuuint64_t strides[2] = {(cuuint64_t)N * 4, 128};
    const cuuint32_t box[3] = {32, (cuuint32_t)CR, (cuuint32_t)(N / 32)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(reinterpret_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int N, int CR, bool SNAP, bool EXT>
cudaError_t launch_variant(const VerifyParams &p, const StreamPlan &plan, const InputMaps &tm, cudaStream_t stream) {
    auto kern = verify_stream_kernel<N, CR, SNAP, EXT>;
    static size_t configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (configured[dev] < plan.smem_bytes) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
        if (e != cudaSuccess) return e;
        configured[dev] = plan.smem_bytes;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel itself waits (griddepcontrol.wait)
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p, plan.layout, tm);
}

int align128(int v) { return (v + 127) & ~127; }

}  // namespace

StreamPlan plan_verify_stream(const VerifyParams &p, bool bf16, int sm_count, size_t smem_per_block_optin) {
    StreamPlan plan{};
    plan.ok = false;
    auto reject = [&](const char *why) {
        snprintf(plan.name, sizeof plan.name, "%s", why);
        return plan;
    };
    if (!bf16) return reject("activations are not bf16");
    if (p.flags & kFlagMamba1) return reject("the Mamba-1 parameterisation runs in the generic kernel");
    if (p.flags & kFlagConvBC) return reject("the conv over the B and C channels runs with the generic kernel");
    if (p.W != kW) return reject("conv width is not 4");
    if (p.N != 64 && p.N != 128) return reject("state dim is not 64 or 128");
    if (p.P % 32) return reject("head dim is not a multiple of 32");
    if (p.H % 8 || p.H > kMaxHeads) return reject("head count is not a multiple of 8 up to 256");
    const int t_cap = p.j_cap + p.k;
    if (t_cap > kMaxT || p.j_cap > kMaxJ) return reject("more than 16 token rows or more than 8 replayed tokens");
    // 64-row chunks, or 32-row ones where the head dim asks for it or 64-row chunks would leave SMs idle
    const bool few = (long long)p.batch * p.H * (p.P / 64) < sm_count;
    const int CR = (p.P % 64 == 0 && !few) ? 64 : 32, N = p.N;
    StreamLayout &L = plan.layout;
    L.TCAP = t_cap < 4 ? 4 : (t_cap + 3) & ~3;
    L.JCAP = p.j_cap < 1 ? 1 : p.j_cap;
    // raw stage: what the producer requests; every sub-buffer is a TMA destination (128-byte aligned)
    const bool gate = p.z != nullptr;
    int o = 0;
    L.r_x = o;   o = align128(o + L.TCAP * CR * 2);
    L.r_z = o;   o = align128(o + L.TCAP * CR * 2);
    L.r_B = o;   o = align128(o + L.TCAP * N * 2);
    L.r_C = o;   o = align128(o + L.TCAP * N * 2);
    L.r_dt = o;  o = align128(o + L.TCAP * 16);
    L.r_cst = o; o = align128(o + (kW - 1) * CR * 2);
    L.r_cw = o;  o = align128(o + CR * kW * 4);
    L.r_cb = o;  o = align128(o + CR * 4);
    L.raw_stride = o;
    L.raw_tx = L.TCAP * (CR * 2 * (gate ? 2 : 1) + 2 * N * 2 + 16) + (kW - 1) * CR * 2 + CR * kW * 4 + CR * 4;
    // per-group buffer: what the prologue phase leaves for the stream phase
    o = 0;
    L.c_Cf = o;  o += L.TCAP * N * 4;
    L.c_Bf = o;  o += (p.state_k != nullptr ? L.TCAP : L.JCAP) * N * 4;   // the second snapshot replays all tokens
    L.c_gz = o;  o += L.TCAP * CR * 4;
    L.c_xc = o;  o += L.TCAP * CR * 4;
    L.c_G = o;   o += kMaxT * kMaxT * 4;
    L.c_hc = o;  o += (int)sizeof(HeadConst);
    L.c_part = o; o += (N / 32) * L.TCAP * CR * 4;   // partial sums of the stream phase
    L.grp_stride = align128(o);
    L.state_stride = CR * N * 4;
    L.inv_hpg_b = 1.0f / (float)(p.H / p.GB);
    L.inv_hpg_c = 1.0f / (float)(p.H / p.GC);
    L.R = kGroups + 1;   // every group can hold a raw stage while the producer fills one ahead
    L.lead = 1;
    auto fixed_bytes = [&]() {
        return (size_t)((kCtrlBytes + 1023) & ~1023) + (size_t)L.R * L.raw_stride + (size_t)L.ngroups * L.grp_stride;
    };
    // Long token blocks make the buffers large.  Wanted, in this order: three state stages before two; as many
    // compute groups as possible; a raw ring as deep as asked for, but at least one stage more than groups.
    {
        const int want_R = L.R;
        bool found = false;
        for (int stages = 3; stages >= 2 && !found; --stages)
            for (int ng = kGroups; ng >= 1 && !found; --ng)
                for (int R = want_R; R >= ng + 1 && !found; --R) {
                    L.ngroups = ng;
                    L.R = R;
                    found = smem_per_block_optin >= fixed_bytes() + (size_t)stages * L.state_stride;
                }
        if (!found) return reject("not enough shared memory for two state stages");
    }
    const size_t fixed = fixed_bytes();
    if (smem_per_block_optin < fixed + 2 * (size_t)L.state_stride) return reject("not enough shared memory for two state stages");
    int S = (int)((smem_per_block_optin - fixed) / L.state_stride);
    if (S > kMaxS) S = kMaxS;
    if (S > 5) S = 5;   // more bytes in flight only lengthen every request's latency once HBM is saturated
    if (L.lead > L.R - 1) L.lead = L.R - 1;

    const long long cph = p.P / CR, nchunks = (long long)p.batch * p.H * cph;
    if (nchunks >= (1ll << 30)) return reject("more than 2^30 chunks");
    long long grid = sm_count;
    if (grid > nchunks) grid = nchunks;
    if (grid < 1) return reject("empty problem");
    const long long per_cta = (nchunks + grid - 1) / grid;
    if (S > per_cta) S = per_cta < 2 ? 2 : (int)per_cta;
    // with few chunks per CTA the state requests should not queue behind a second chunk's small inputs
    // (measured: batch 4 and 16 gain 2 % with lead 0, batch 64 loses 1 %)
    if (per_cta <= 16) L.lead = 0;
    // A group hands a stage with a pending store back only when it starts its next chunk, after that chunk's
    // small inputs are in; the producer requests those only once it has the stage (lead 0), or one chunk earlier
    // (lead 1).  So no more groups than stages + lead may hold stages, unless the CTA never reuses a stage.
    while (L.ngroups > 1 && L.ngroups > S + L.lead && per_cta > S) --L.ngroups;
    L.S = S;
    L.state_off = (kCtrlBytes + 1023) & ~1023;   // the swizzled state stages need 1024-byte alignment
    L.raw_off = L.state_off + S * L.state_stride;
    L.grp_off = L.raw_off + L.R * L.raw_stride;

    plan.ok = true;
    plan.grid = (int)grid;
    const bool ext = (p.flags & (kFlagDtSoftplus | kFlagYNewOnly)) != 0 || p.sel != nullptr || p.row_off != nullptr ||
                     p.row_off_const != 0;
    plan.variant = (N == 128 ? 0 : 2) + (CR == 64 ? 0 : 1) + (p.state_k != nullptr ? 4 : 0) + (ext ? 8 : 0);
    plan.smem_bytes = (size_t)L.grp_off + (size_t)L.ngroups * L.grp_stride;
    snprintf(plan.name, sizeof plan.name, "stream<N=%d,CR=%d,groups=%d,TCAP=%d,S=%d,R=%d,lead=%d,grid=%d%s>", N, CR, L.ngroups,
             L.TCAP, L.S, L.R, L.lead, (int)grid, ext ? ",ext" : "");
    return plan;
}

bool encode_stream_maps(const VerifyParams &p, const StreamPlan &plan, InputMaps *tm) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const StreamLayout &L = plan.layout;
    const int CR = (plan.variant & 1) ? 32 : 64;
    const size_t rows = (size_t)p.batch * p.t_max, hp = (size_t)p.H * p.P, srows = (size_t)p.batch * p.H * p.P;
    bool ok = encode_2d(fn, &tm->x, p.x, hp, rows, CR, L.TCAP) &&
              encode_2d(fn, &tm->z, p.z ? p.z : p.x, hp, rows, CR, L.TCAP) &&
              encode_2d(fn, &tm->B, p.B, (size_t)p.GB * p.N, rows, p.N, L.TCAP) &&
              encode_2d(fn, &tm->C, p.C, (size_t)p.GC * p.N, rows, p.N, L.TCAP) &&
              encode_2d(fn, &tm->dt, p.dt, (size_t)p.H, rows, 8, L.TCAP) &&
              encode_2d(fn, &tm->cst, p.conv_state, hp, (size_t)p.batch * (kW - 1), CR, kW - 1) &&
              encode_state(fn, &tm->state, p.state, srows, p.N, CR);
    if (p.state_k) ok = ok && encode_state(fn, &tm->state_k, p.state_k, srows, p.N, CR) &&
                        encode_2d(fn, &tm->cst_k, p.conv_state_k, hp, (size_t)p.batch * (kW - 1), CR, kW - 1);
    else {
        memcpy(&tm->state_k, &tm->state, sizeof(TensorMapBytes));
        memcpy(&tm->cst_k, &tm->cst, sizeof(TensorMapBytes));
    }
    return ok;
}

cudaError_t launch_verify_stream(const VerifyParams &p, const StreamPlan &plan, const InputMaps &tm, cudaStream_t stream) {
    // bit 0: 32-row chunks; bit 1: N = 64; bit 2: second snapshot; bit 3: the variants of the call (raw interval,
    // cache in either of two buffers, outputs for new rows only, rows at an offset) compiled in
    switch (plan.variant) {
#define MSPEC_CASE(v, n, cr, snap, ext) case v: return launch_variant<n, cr, snap, ext>(p, plan, tm, stream);
        MSPEC_CASE(0, 128, 64, false, false) MSPEC_CASE(1, 128, 32, false, false)
        MSPEC_CASE(2, 64, 64, false, false) MSPEC_CASE(3, 64, 32, false, false)
        MSPEC_CASE(4, 128, 64, true, false) MSPEC_CASE(5, 128, 32, true, false)
        MSPEC_CASE(6, 64, 64, true, false) MSPEC_CASE(7, 64, 32, true, false)
        MSPEC_CASE(8, 128, 64, false, true) MSPEC_CASE(9, 128, 32, false, true)
        MSPEC_CASE(10, 64, 64, false, true) MSPEC_CASE(11, 64, 32, false, true)
        MSPEC_CASE(12, 128, 64, true, true) MSPEC_CASE(13, 128, 32, true, true)
        MSPEC_CASE(14, 64, 64, true, true) MSPEC_CASE(15, 64, 32, true, true)
        default: return cudaErrorInvalidValue;
#undef MSPEC_CASE
    }
}

}  // namespace mspec
