// Streaming verification kernel for sm_100a: bf16 activations, fp32 state, conv
// width 4, state dim 64 or 128, head dim a multiple of 32, up to 16 token rows.
//
// The call has to read (and, where tokens were accepted, re-write) the fp32
// state once; everything else is small.  The state rows are independent
// recurrences, so the kernel is organised around ONE WARP PER 32 STATE ROWS
// (a "unit"), with no barrier between compute warps.  One persistent CTA per SM:
//
//   head warps      what depends on a head's inputs but on no state row.  A head warp
//                   loads the head's dt, B and C rows from global memory straight into
//                   matrix-instruction fragments and forms: the decay products of the
//                   on-the-fly discretisation (Sec. 2.2), the T x T table of the unrolled
//                   recurrence, fp32 copies of the C rows and of the B rows that the new
//                   state needs.  Each head warp owns one table slot; they run ahead of
//                   the compute warps.
//   compute warps   each owns one or two state stages and takes every AW-th unit of the CTA's work
//                   list through them: it requests the unit's 32 state rows itself, with one TMA
//                   request (a 3-D tiled tensor map that lays the rows down as swizzled 32-column
//                   quarters), as soon as the stage is free.  Nothing else goes through the TMA
//                   unit: a request costs it several hundred cycles whatever its size, and the small
//                   inputs would take most of it.  For the streaming part a lane holds 4 rows x 4 columns
//                   of the state at a time (lane = (row mod 8, column quarter)), so that one
//                   16-byte read of C_t feeds eight packed multiply-adds; the column quarters
//                   are summed by two shuffles per value.  Where tokens were accepted the
//                   state at the verified position is formed in the same registers, put back
//                   into the stage and stored by one TMA request (Sec. 4.3 iii).  For the rest
//                   lane = row: causal conv + SiLU from the rolling window (Sec. 4.3,
//                   footnote; inputs read directly from global memory while the state rows
//                   are in flight), outputs with skip term and gate, conv window at position j.
//
// Stages and table slots are handed over through mbarriers and monotonic counters; every
// wait is bounded.  The kernel is launched with programmatic stream serialisation: its
// on-chip set-up overlaps the tail of the previous kernel.
//
// The recurrence (Eq. 1, discretised on the fly) is evaluated in its unrolled
// form, the same sum in another order.  With a_t = exp(dt_t A_h), the cached
// state h and xc the post-conv input:
//     y_t[p]   = alpha_t (C_t . h[p,:]) + sum_{s<=t} G[t][s] xc_s[p],
//     G[t][s]  = (C_t . B_s) dt_s prod_{s<r<=t} a_r  (+ D_h on the diagonal),
//     alpha_t  = prod_{r<=t} a_r,
//     h_j[p,:] = alpha_{j-1} h[p,:] + sum_{s<j} (dt_s prod_{s<r<j} a_r) xc_s[p] B_s.
// Each state element is touched by T multiply-adds for the outputs and j+1 for
// the new state; the per-token states never exist (Sec. 4.2) and the state at
// the verified position is formed and stored once.  Multiply-adds on the state
// are packed f32x2 operations, no tensor cores (fp32 state, exact products
// wanted); only the small T x T table of bf16 dot products C_t . B_s, exact in
// fp32, is formed with warp-level matrix instructions.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace mspec {
namespace {

constexpr int kComputeWarps = 10, kHeadWarps = 2, kSlots = 4;   // twelve warps leave each thread 168 registers
constexpr int kThreads = (kComputeWarps + kHeadWarps) * 32;
static_assert(kSlots % kHeadWarps == 0, "a table slot is always filled by the same head warp");
constexpr int kUnitRows = 32;   // state rows of a unit
constexpr int kMaxS = 2 * kComputeWarps;
constexpr int kJTable = 1024;   // sequences whose pending length is kept in shared memory
constexpr int kW = 4;           // conv width handled here
constexpr int kMaxT = 16;       // token rows per sequence handled here
constexpr int kMaxJ = 8;
constexpr int kTB = 4;          // tokens whose sums a lane accumulates at a time (the state rows are re-read per block)
#ifndef MSPEC_WAIT_LIMIT_CYCLES
#define MSPEC_WAIT_LIMIT_CYCLES 4000000000ll   // a wait that lasts about 2 s is reported, not sat out
#endif
constexpr long long kWaitLimitCycles = MSPEC_WAIT_LIMIT_CYCLES;

struct Ctrl {
    unsigned long long state_full[kMaxS];
    unsigned long long slot_empty[kSlots], slot_full[kSlots];
    int abort;
    // heads published in each table slot, as (item index + 1): monotonic, so a reader that is several
    // uses of a slot behind cannot mistake one use for another the way a phase parity could
    int slot_ready[kSlots];
    int state_par[kMaxS];   // parity of the last fill of each state stage, -1 before any
    int work[16];           // the CTA's Work (see below), computed once
    int jarr[kJTable];
};
constexpr int kCtrlBytes = (sizeof(Ctrl) + 1023) / 1024 * 1024;   // the swizzled stages behind it need 1024-byte alignment

// Per-head scalars, written by the head warp.
struct HeadConst {
    float alpha[kMaxT];  // prod_{r<=t} a_r
    float wsp[kMaxT];    // dt_s prod_{s<r<j} a_r, s < j
    float wspT[kMaxT];   // dt_s prod_{s<r<T} a_r, s >= j  (second snapshot only)
    float alpha_j;       // prod_{r<j} a_r
    float alpha_jT;      // prod_{j<=r<T} a_r             (second snapshot only)
    float pad[2];
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
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
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
// Slow path of a wait, kept out of line so that the wait sites stay small.  Waiting threads are
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
// Waits until a monotonic counter in shared memory has reached `want` (acquire), with the same limits.
__device__ __forceinline__ int ld_acquire_shared(uint32_t addr) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __noinline__ bool counter_wait_slow(uint32_t addr, int want, const volatile int *abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        __nanosleep(64);
        if (ld_acquire_shared(addr) >= want) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitLimitCycles) return false;
    }
}
__device__ __forceinline__ bool counter_wait(uint32_t addr, int want, const volatile int *abort_flag) {
    if (ld_acquire_shared(addr) >= want) return true;
    return counter_wait_slow(addr, want, abort_flag);
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

// ---------------------------------------------------------------- work list of a CTA
// Heads (a head = one (sequence, head) pair, P state rows = P/32 units) are dealt to the CTAs whole as
// long as every CTA gets the same number: CTA i owns heads i, i + G, ..., i + (F-1) G.  The R = heads
// mod G heads that are left are cut into units, and CTA i takes the i-th of G nearly equal contiguous
// runs of them, so that no CTA has more than one unit more than another.  An "item" is what a CTA has
// of one head: all its units, or a run of them.
struct Work {
    int G, i, H, uph;          // CTAs, this CTA, heads per sequence, units per head
    unsigned H_mul, uph_mul;   // ceil(2^32 / H), ceil(2^32 / uph): x / d = umulhi(x, mul) for the x that occur here
    int F;                     // whole heads of this CTA
    int ra, rb, rh0;           // its run [ra, rb) of the left-over units, and the left-over head that ra falls in
    int nitems, nunits;
};
struct Item {
    int head, u0, nu, n0;      // global head index, first unit of the head, units, sequence number of the first unit
};
// Computed once per CTA (by one thread, into shared memory): the divisions are not cheap.
__device__ __forceinline__ void make_work(const VerifyParams &p, const StreamLayout &L, Work &w) {
    w.G = (int)gridDim.x;
    w.i = (int)blockIdx.x;
    w.H = p.H;
    w.uph = p.P / kUnitRows;
    w.H_mul = L.H_mul;
    w.uph_mul = L.uph_mul;
    const int nheads = p.batch * p.H;
    w.F = nheads / w.G;
    const long long rem_units = (long long)(nheads - w.F * w.G) * w.uph;
    w.ra = (int)(rem_units * w.i / w.G);
    w.rb = (int)(rem_units * (w.i + 1) / w.G);
    w.rh0 = w.ra / w.uph;
    const int npart = w.rb > w.ra ? (w.rb - 1) / w.uph - w.rh0 + 1 : 0;
    w.nitems = w.F + npart;
    w.nunits = w.F * w.uph + (w.rb - w.ra);
}
__device__ __forceinline__ int div_uph(const Work &w, int x) { return (int)__umulhi((unsigned)x, w.uph_mul); }
__device__ __forceinline__ int div_H(const Work &w, int x) { return (int)__umulhi((unsigned)x, w.H_mul); }
__device__ __forceinline__ Item item_of(const Work &w, int m) {
    Item it;
    if (m < w.F) {
        it.head = w.i + m * w.G;
        it.u0 = 0;
        it.nu = w.uph;
        it.n0 = m * w.uph;
    } else {
        const int rh = w.rh0 + (m - w.F);
        const int lo = max(w.ra, rh * w.uph), hi = min(w.rb, (rh + 1) * w.uph);
        it.head = w.F * w.G + rh;
        it.u0 = lo - rh * w.uph;
        it.nu = hi - lo;
        it.n0 = w.F * w.uph + (lo - w.ra);
    }
    return it;
}
// Unit number n of the CTA -> its item, head and unit of the head.
__device__ __forceinline__ void unit_of(const Work &w, int n, int &m, int &head, int &u) {
    if (n < w.F * w.uph) {
        m = div_uph(w, n);
        u = n - m * w.uph;
        head = w.i + m * w.G;
    } else {
        const int r = w.ra + (n - w.F * w.uph), rh = div_uph(w, r);
        m = w.F + rh - w.rh0;
        u = r - rh * w.uph;
        head = w.F * w.G + rh;
    }
}
__device__ __forceinline__ int pending_of(const VerifyParams &p, const Ctrl &ctl, int b) {
    return b < kJTable ? ctl.jarr[b] : load_n_prev(p, b);
}
__device__ __forceinline__ void give_up(const VerifyParams &p, Ctrl &ctl) {
    atomicOr(p.status, kStatusCopyTimeout);
    ctl.abort = 1;
}


static_assert(sizeof(Work) <= sizeof(int) * 16, "Ctrl::work too small");

// ---------------------------------------------------------------- state requests
// One TMA request for the 32 state rows of unit n into a stage (issued by one lane of the warp that owns the stage).
template <int N>
__device__ __forceinline__ void request_state(const VerifyParams &p, const StreamLayout &L, unsigned char *smem, Ctrl &ctl,
                                              const InputMaps &tm, const Work &w, int n, int ss, int sp) {
    constexpr uint32_t kStateBytes = kUnitRows * N * 4;
    int m, head, u;
    unit_of(w, n, m, head, u);
    const uint32_t sbar = smem_u32(&ctl.state_full[ss]);
    ctl.state_par[ss] = sp;
    mbar_arrive_expect_tx(sbar, kStateBytes);
    tma_load_3d(smem_u32(smem) + L.state_off + ss * L.state_stride, as_map(&tm.state), 0, head * p.P + u * kUnitRows, 0, sbar);
}

// ---------------------------------------------------------------- head warps
// The fragments of one head's C and B rows for the matrix instruction (16 x 8 x 16 per instruction; thread
// (g, tq) = (lane / 4, lane % 4) supplies rows g and g + 8 of C, row g of a block of eight B rows, and of
// every 32 columns the eight columns 8 tq .. 8 tq + 7 -- the order in which the instruction walks the columns
// does not matter as long as both operands use the same one): 16-byte loads straight from global memory.
template <int N, int TC>
struct HeadFrags {
    uint4 a_lo[N / 32], b_lo[N / 32];
    uint4 a_hi[TC > 8 ? N / 32 : 1], b_hi[TC > 8 ? N / 32 : 1];
    float dtv, A, D;
};
template <int N, int TC>
__device__ __forceinline__ void load_head(const VerifyParams &p, const StreamLayout &L, const Work &w, int head, int lane,
                                          HeadFrags<N, TC> &f) {
    constexpr int NC = N / 32;
    const int b = div_H(w, head), h = head - b * w.H;
    const int g = lane >> 2, tq = lane & 3;
    const size_t trow = (size_t)b * p.t_max;
    const int rmax = p.t_max - 1;   // rows past the sequence's tokens are read (they exist) but never used
    const int r0 = g < rmax ? g : rmax, r1 = g + 8 < rmax ? g + 8 : rmax;
    f.A = p.A[h];
    f.D = p.D[h];
    f.dtv = lane <= rmax ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p.dt)[(trow + lane) * p.H + h]) : 0.f;
    const uint4 *Cg = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(p.C) + ((trow * p.GC) + h / L.hpg_c) * N) + tq;
    const uint4 *Bg = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(p.B) + ((trow * p.GB) + h / L.hpg_b) * N) + tq;
    const size_t cstr = (size_t)p.GC * N / 8, bstr = (size_t)p.GB * N / 8;   // row stride in 16-byte pieces
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        f.a_lo[c] = Cg[r0 * cstr + c * 4];
        f.b_lo[c] = Bg[r0 * bstr + c * 4];
        if (TC > 8) {
            f.a_hi[c] = Cg[r1 * cstr + c * 4];
            f.b_hi[c] = Bg[r1 * bstr + c * 4];
        }
    }
}

// Everything of one head that needs no state row, left in the head warp's table slot:
//   pairs   G[t][s] = (C_t . B_s) dt_s prod_{s<r<=t} a_r for s <= t (+ D_h on the diagonal): the T x T products
//           are a small bf16 matrix product, exact in fp32; the decay product is one exp of a difference of
//           prefix sums of dt (Sec. 2.2: a_r = exp(dt_r A_h))
//   decay   alpha_t, wsp_s, alpha_j from the same prefix sums (lane t holds dt_t)
//   rows    fp32 copies of the C rows (all tokens) and of the B rows s < j, from the same fragments; the
//           compute warps read them as broadcasts
template <int N, int TC, bool SNAP>
__device__ __forceinline__ void head_tables(const StreamLayout &L, unsigned char *slot, const HeadFrags<N, TC> &f, int j, int T,
                                            int lane) {
    constexpr int NC = N / 32;
    HeadConst *hc = reinterpret_cast<HeadConst *>(slot + L.c_hc);
    float *Gm = reinterpret_cast<float *>(slot + L.c_G);    // [kMaxT][kMaxT], entries s <= t < T
    float *Cf = reinterpret_cast<float *>(slot + L.c_Cf), *Bf = reinterpret_cast<float *>(slot + L.c_Bf);
    const int g = lane >> 2, tq = lane & 3;
    const bool two = TC > 8 && T > 8;
    const float A_of_head = f.A, D_of_head = f.D;
    const float dtv = lane < T ? f.dtv : 0.f;
    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i >> 2][i & 3] = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const uint4 a_hi = TC > 8 ? f.a_hi[c] : make_uint4(0u, 0u, 0u, 0u);
        mma_bf16_16816(acc[0], f.a_lo[c].x, a_hi.x, f.a_lo[c].y, a_hi.y, f.b_lo[c].x, f.b_lo[c].y);
        mma_bf16_16816(acc[0], f.a_lo[c].z, a_hi.z, f.a_lo[c].w, a_hi.w, f.b_lo[c].z, f.b_lo[c].w);
        if (TC > 8) {
            if (two) {
                mma_bf16_16816(acc[1], f.a_lo[c].x, a_hi.x, f.a_lo[c].y, a_hi.y, f.b_hi[c].x, f.b_hi[c].y);
                mma_bf16_16816(acc[1], f.a_lo[c].z, a_hi.z, f.a_lo[c].w, a_hi.w, f.b_hi[c].z, f.b_hi[c].w);
            }
        }
    }
    // lane r holds dt_r and E_r = sum_{r' <= r} dt_r'
    float E = dtv;
#pragma unroll
    for (int d = 1; d < kMaxT; d <<= 1) {
        const float up = __shfl_up_sync(0xffffffffu, E, d);
        if (lane >= d) E += up;
    }
    const float Et0 = __shfl_sync(0xffffffffu, E, g), Et1 = __shfl_sync(0xffffffffu, E, g + 8);
#pragma unroll
    for (int nt = 0; nt < (TC > 8 ? 2 : 1); ++nt) {
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
        if (nt == 0 || two) {
            *reinterpret_cast<float2 *>(Gm + g * kMaxT + s0) = lo;
            if (two) *reinterpret_cast<float2 *>(Gm + (g + 8) * kMaxT + s0) = hi;
        }
    }
    // ---- decay products: lane t: alpha_t = exp(A_h E_t); t < j: wsp_t = dt_t exp(A_h (E_{j-1} - E_t));
    //      alpha_j = exp(A_h E_{j-1}); for the second snapshot the same towards the end of the block
    {
        const float Ej = __shfl_sync(0xffffffffu, E, j > 0 ? j - 1 : 0), ET = __shfl_sync(0xffffffffu, E, T > 0 ? T - 1 : 0);
        const float Ejj = j > 0 ? Ej : 0.f, ETT = T > 0 ? ET : 0.f;
        if (lane < T) hc->alpha[lane] = expf(A_of_head * E);
        if (lane < j) hc->wsp[lane] = dtv * expf(A_of_head * (Ejj - E));
        if (lane == 0) hc->alpha_j = expf(A_of_head * Ejj);
        if (SNAP) {
            if (lane >= j && lane < T) hc->wspT[lane] = dtv * expf(A_of_head * (ETT - E));
            if (lane == 0) hc->alpha_jT = expf(A_of_head * (ETT - Ejj));
        }
    }
    // ---- fp32 copies of the rows this lane holds fragments of: C rows g (and g + 8) up to a multiple of
    //      four (the compute warps take tokens in pairs), B rows below j up to an even count (all rows for the
    //      second snapshot); rows past T hold padding that meets only zero coefficients or unused sums --
    //      except that a B row past j must be finite, so it is written as zeros
    {
        const int nC = (T + 3) & ~3, nB = SNAP ? T : j, nBz = (nB + 1) & ~1;
        auto put = [&](float *dst, const uint4 &v, bool zero) {
            const uint4 q = zero ? make_uint4(0u, 0u, 0u, 0u) : v;
            reinterpret_cast<float4 *>(dst)[0] = make_float4(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u),
                                                             __uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u));
            reinterpret_cast<float4 *>(dst)[1] = make_float4(__uint_as_float(q.z << 16), __uint_as_float(q.z & 0xffff0000u),
                                                             __uint_as_float(q.w << 16), __uint_as_float(q.w & 0xffff0000u));
        };
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int col = c * 32 + tq * 8;
            if (g < nC) put(Cf + g * N + col, f.a_lo[c], false);
            if (g < nBz && g < L.JB) put(Bf + g * N + col, f.b_lo[c], g >= nB);
            if (TC > 8) {
                if (g + 8 < nC) put(Cf + (g + 8) * N + col, f.a_hi[c], false);
                if (g + 8 < nBz && g + 8 < L.JB) put(Bf + (g + 8) * N + col, f.b_hi[c], g + 8 >= nB);
            }
        }
    }
}

template <int N, int TC, bool SNAP>
__device__ __forceinline__ void head_role(const VerifyParams &p, const StreamLayout &L, unsigned char *smem, Ctrl &ctl,
                                          const Work &w, int hw, int lane, HeadFrags<N, TC> &f) {
    for (int m = hw; m < w.nitems; m += kHeadWarps) {
        const int hs = m % kSlots, use = m / kSlots;   // slot hs is always this head warp's: kSlots is a multiple of kHeadWarps
        unsigned char *slot = smem + L.tab_off + (size_t)hs * L.tab_stride;
        const Item it = item_of(w, m);
        if (m != hw) load_head<N, TC>(p, L, w, it.head, lane, f);   // (the first head's loads went out at the start of the kernel)
        const int b = div_H(w, it.head);
        const int j = pending_of(p, ctl, b), T = j + p.k;
        // the slot is free once every unit of the head that had it has handed it back
        if (use > 0 && !mbar_wait(smem_u32(&ctl.slot_empty[hs]), (uint32_t)((use - 1) & 1), &ctl.abort)) return give_up(p, ctl);
        head_tables<N, TC, SNAP>(L, slot, f, j, T, lane);
        __syncwarp();
        if (lane == 0) {
            asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(&ctl.slot_ready[hs])), "r"(m + 1) : "memory");
            mbar_arrive(smem_u32(&ctl.slot_full[hs]));
            // the slot is handed back by the head's units, one arrival each; units of this head that other
            // CTAs have are made up for here
            if (it.nu < w.uph) mbar_arrive_n(smem_u32(&ctl.slot_empty[hs]), (uint32_t)(w.uph - it.nu));
        }
    }
}

// ---------------------------------------------------------------- compute warps
// What a lane needs of its own row (lane = row outside the streaming part): straight from global memory.
template <int TC>
struct RowIn {
    unsigned short xr[TC + kW - 1];   // the cached window, then x_t
    unsigned short zr[TC];
    float4 wv;
    float bias;
};
template <int TC>
__device__ __forceinline__ void load_row(const VerifyParams &p, int b, int h, int row, int tlim, RowIn<TC> &in) {
    const int HP = p.H * p.P;   // tlim: token rows to load (at most the rows of the slab)
    const unsigned short *xg = reinterpret_cast<const unsigned short *>(p.x) + ((size_t)b * p.t_max * p.H + h) * p.P + row;
    const unsigned short *zg = reinterpret_cast<const unsigned short *>(p.z) + ((size_t)b * p.t_max * p.H + h) * p.P + row;
    const unsigned short *cg = reinterpret_cast<const unsigned short *>(p.conv_state) + (size_t)b * (kW - 1) * HP + h * p.P + row;
#pragma unroll
    for (int wi = 0; wi < kW - 1; ++wi) in.xr[wi] = cg[wi * HP];
#pragma unroll
    for (int t = 0; t < TC; ++t) in.xr[kW - 1 + t] = t < tlim ? xg[t * HP] : (unsigned short)0;
#pragma unroll
    for (int t = 0; t < TC; ++t) in.zr[t] = (p.z != nullptr && t < tlim) ? zg[t * HP] : (unsigned short)0;
    in.wv = reinterpret_cast<const float4 *>(p.conv_w)[h * p.P + row];
    in.bias = p.conv_b[h * p.P + row];
}

// The same addresses as load_row / load_head, as L2 prefetches: they have no architectural effect, so they may go
// out before the previous kernel of the stream has completed, and they take the cold misses (address translation,
// first DRAM access) off the path of the real loads.
__device__ __forceinline__ void prefetch_l2(const void *ptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr)); }
template <int TC>
__device__ __forceinline__ void prefetch_row(const VerifyParams &p, int b, int h, int row, int tlim) {
    const int HP = p.H * p.P;
    const unsigned short *xg = reinterpret_cast<const unsigned short *>(p.x) + ((size_t)b * p.t_max * p.H + h) * p.P + row;
    const unsigned short *zg = reinterpret_cast<const unsigned short *>(p.z) + ((size_t)b * p.t_max * p.H + h) * p.P + row;
    const unsigned short *cg = reinterpret_cast<const unsigned short *>(p.conv_state) + (size_t)b * (kW - 1) * HP + h * p.P + row;
    if ((row & 15) == 0) {   // one lane per 32-byte sector
#pragma unroll
        for (int wi = 0; wi < kW - 1; ++wi) prefetch_l2(cg + wi * HP);
#pragma unroll
        for (int t = 0; t < TC; ++t) {
            if (t < tlim) {
                prefetch_l2(xg + t * HP);
                if (p.z != nullptr) prefetch_l2(zg + t * HP);
            }
        }
    }
    if ((row & 1) == 0) prefetch_l2(reinterpret_cast<const float4 *>(p.conv_w) + h * p.P + row);
    if ((row & 7) == 0) prefetch_l2(p.conv_b + h * p.P + row);
}
template <int N, int TC>
__device__ __forceinline__ void prefetch_head(const VerifyParams &p, const StreamLayout &L, const Work &w, int head, int lane) {
    const int b = div_H(w, head), h = head - b * w.H;
    const size_t trow = (size_t)b * p.t_max;
    const int rows = p.t_max < TC ? p.t_max : TC, r = lane >> 1;   // lane -> (row, half of a 256-byte row)
    const __nv_bfloat16 *Cg = reinterpret_cast<const __nv_bfloat16 *>(p.C) + ((trow * p.GC) + h / L.hpg_c) * N;
    const __nv_bfloat16 *Bg = reinterpret_cast<const __nv_bfloat16 *>(p.B) + ((trow * p.GB) + h / L.hpg_b) * N;
    if (r < rows) {
        if ((lane & 1) * 64 < N) {
            prefetch_l2(Cg + (size_t)r * p.GC * N + (lane & 1) * 64);
            prefetch_l2(Bg + (size_t)r * p.GB * N + (lane & 1) * 64);
        }
        if ((lane & 1) == 0) prefetch_l2(reinterpret_cast<const __nv_bfloat16 *>(p.dt) + (trow + r) * p.H + h);
    }
    if (lane == 0) { prefetch_l2(p.A + h); prefetch_l2(p.D + h); }
}

// The streaming part over one block of NT tokens.  The rows sit in the stage as the TMA engine wrote them:
// 32-column quarters, quarter-major ([quarter][row][32 floats], 128 bytes per line) with the 128-byte
// swizzle, so that eight lanes read 16-byte pieces of eight consecutive rows without bank conflicts.
// Lane (g, cq) = (lane % 8, lane / 8) owns rows g, g+8, g+16, g+24 and the cq-th quarter of the columns,
// one 16-byte piece (4 columns) of each of its rows at a time; `rb` is row g's line in the lane's quarter,
// `gx` the swizzled byte offset of the lane's first piece.  With FORM the state at the verified position
// (Sec. 4.3 iii) is formed in the same registers and put back in place.
template <int N, int NT, bool FORM, int JC>
__device__ __forceinline__ void stream_block(unsigned char *rb, uint32_t gx, const float *cbase, const float *bbase,
                                             float2 (&acc)[kTB][4], int j, float aj, const float (&cx)[JC],
                                             const float (&cfr)[JC <= 4 ? JC : 1][4], int g) {
    constexpr bool HOIST = JC <= 4;   // few replayed tokens: the rows' coefficients are kept in registers
    constexpr int PPL = N / 16;   // 16-byte pieces of a row that a lane goes through
#pragma unroll 1
    for (int ps = 0; ps < PPL; ++ps) {

        unsigned char *a = rb + (gx ^ (uint32_t)(ps << 4));
        float4 hv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) hv[i] = *reinterpret_cast<const float4 *>(a + 1024 * i);   // row g + 8 i
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const float4 cv = *reinterpret_cast<const float4 *>(cbase + t * N + ps * 4);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t][i] = ffma2(lo2(hv[i]), lo2(cv), acc[t][i]);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t][i] = ffma2(hi2(hv[i]), hi2(cv), acc[t][i]);
        }
        if (FORM) {
            const float2 aj2 = make_float2(aj, aj);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 l = __fmul2_rn(lo2(hv[i]), aj2), h2 = __fmul2_rn(hi2(hv[i]), aj2);
                hv[i] = make_float4(l.x, l.y, h2.x, h2.y);
            }
#pragma unroll
            for (int s = 0; s < JC; s += 2) {
                if (s < j) {   // two at a time: a coefficient past j is zero and its B row is zeros
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        if (s + e < JC) {
                            const float4 bv = *reinterpret_cast<const float4 *>(bbase + (s + e) * N + ps * 4);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float c = HOIST ? cfr[HOIST ? s + e : 0][i] : __shfl_sync(0xffffffffu, cx[s + e], g + 8 * i);
                                const float2 c2 = make_float2(c, c);
                                const float2 l = ffma2(c2, lo2(bv), lo2(hv[i])), h2 = ffma2(c2, hi2(bv), hi2(hv[i]));
                                hv[i] = make_float4(l.x, l.y, h2.x, h2.y);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) *reinterpret_cast<float4 *>(a + 1024 * i) = hv[i];
        }
    }
}

// One unit: the 32 state rows [u*32, u*32+32) of a head.
template <int N, int TC, int JC, bool SNAP>
__device__ __forceinline__ bool compute_unit(const VerifyParams &p, const StreamLayout &L, const InputMaps &tm, Ctrl &ctl,
                                             unsigned char *st, const unsigned char *slot, uint32_t full_bar, uint32_t full_par,
                                             int hs, int m, int ss, int n_next, unsigned char *smem, const Work &w, int head,
                                             int b, int h, int u, int j, int T, int lane, const RowIn<TC> &in) {
    // the stage is free: request the rows of the next unit that goes through it (one lane)
    auto refill = [&]() {
        if (n_next < w.nunits) request_state<N>(p, L, smem, ctl, tm, w, n_next, ss, (int)(full_par ^ 1u));
    };
    constexpr int PPL = N / 16;
    constexpr unsigned FULL = 0xffffffffu;
    const int P = p.P, HP = p.H * p.P, row = u * kUnitRows + lane;
    const int g = lane & 7, cq = lane >> 3;
    const bool gate = p.z != nullptr, y_f32 = (p.flags & kFlagYF32) != 0, conv_silu = (p.flags & kFlagConvSilu) != 0;
    const HeadConst *hc = reinterpret_cast<const HeadConst *>(slot + L.c_hc);

    // ---- causal conv + SiLU of this row over the token block, from the rolling window
    float xc[TC];
#pragma unroll
    for (int t2 = 0; t2 < TC; t2 += 2) {
        xc[t2] = xc[t2 + 1] = 0.f;
        if (t2 < T) {   // tokens in pairs; a token past T gives a value that is never used
#pragma unroll
            for (int t = t2; t < t2 + 2; ++t) {
                const float v = fmaf(in.wv.w, bf16_bits_to_f32(in.xr[t + 3]), fmaf(in.wv.z, bf16_bits_to_f32(in.xr[t + 2]),
                                fmaf(in.wv.y, bf16_bits_to_f32(in.xr[t + 1]), fmaf(in.wv.x, bf16_bits_to_f32(in.xr[t]), in.bias))));
                xc[t] = conv_silu ? silu_fast(v) : v;
            }
        }
    }

    // ---- the head's tables: published by the slot's head warp.  The counter tells which use of the slot is
    //      in; once the previous use is known to be over, the slot's barrier is at most one phase ahead and
    //      can be waited on.
    {
        const uint32_t ready = smem_u32(&ctl.slot_ready[hs]);
        if (ld_acquire_shared(ready) < m + 1) {
            if (!counter_wait(ready, m + 1 - kSlots, &ctl.abort)) return false;
            if (!mbar_wait(smem_u32(&ctl.slot_full[hs]), (uint32_t)((m / kSlots) & 1), &ctl.abort)) return false;
        }
    }
    // ---- everything of the outputs that needs no state: y_t = ya_t (C_t . h) + yw_t with
    //      ya_t = alpha_t gate_t, yw_t = gate_t sum_{s<=t} G[t][s] xc_s (D on the diagonal of G)
    float ya[TC], yw[TC];
    {
        const float *Gm = reinterpret_cast<const float *>(slot + L.c_G);
#pragma unroll
        for (int t = 0; t < TC; ++t) {
            ya[t] = yw[t] = 0.f;
            if ((t & ~1) >= T) continue;   // tokens in pairs, as above
            float wsum = 0.f;
#pragma unroll
            for (int s4 = 0; s4 <= t; s4 += 4) {
                const float4 g4 = *reinterpret_cast<const float4 *>(Gm + t * kMaxT + s4);
                wsum = fmaf(g4.x, xc[s4], wsum);
                if (s4 + 1 <= t) wsum = fmaf(g4.y, xc[s4 + 1], wsum);
                if (s4 + 2 <= t) wsum = fmaf(g4.z, xc[s4 + 2], wsum);
                if (s4 + 3 <= t) wsum = fmaf(g4.w, xc[s4 + 3], wsum);
            }
            const float gz = gate ? silu_fast(bf16_bits_to_f32(in.zr[t])) : 1.f;
            ya[t] = hc->alpha[t] * gz;
            yw[t] = wsum * gz;
        }
    }
    // ---- the coefficients of B_s in the new state of the lane's four rows: wsp_s xc_s[row g + 8 i]
    const bool stored = j > 0;
    float cx[JC], cfr[JC <= 4 ? JC : 1][4];
#pragma unroll
    for (int s = 0; s < JC; ++s) {
        cx[s] = s < j ? hc->wsp[s] * xc[s] : 0.f;
        if (JC <= 4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) cfr[JC <= 4 ? s : 0][i] = __shfl_sync(FULL, cx[s], g + 8 * i);
        }
    }
    const float aj = hc->alpha_j;
    const float *Cf = reinterpret_cast<const float *>(slot + L.c_Cf) + cq * (N / 4);
    const float *Bf = reinterpret_cast<const float *>(slot + L.c_Bf) + cq * (N / 4);
    const int pc0 = cq * PPL;   // the lane's first piece of the row: quarter pc0 / 8, piece pc0 % 8 of the quarter
    unsigned char *rb = st + (size_t)((pc0 >> 3) * kUnitRows + g) * 128;
    const uint32_t gx = (uint32_t)(((pc0 & 7) ^ g) << 4);
    const size_t y0 = (((size_t)b * p.t_max) * p.H + h) * P + row;

    // ---- the state rows
    if (!mbar_wait(full_bar, full_par, &ctl.abort)) return false;
#pragma unroll 1
    for (int tb0 = 0; tb0 < T; tb0 += kTB) {
        const bool form = stored && tb0 + kTB >= T;   // the last token block also forms the new state
        const bool four = tb0 + 2 < T;                // tokens are taken in pairs
        float2 acc[kTB][4];
#pragma unroll
        for (int t = 0; t < kTB; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t][i] = make_float2(0.f, 0.f);
        const float *cb = Cf + tb0 * N;
        if (form) {
            if (four) stream_block<N, 4, true, JC>(rb, gx, cb, Bf, acc, j, aj, cx, cfr, g);
            else stream_block<N, 2, true, JC>(rb, gx, cb, Bf, acc, j, aj, cx, cfr, g);
            fence_proxy_async();   // the TMA store below reads what the lanes just wrote
            __syncwarp();
            if (lane == 0) {
                tma_store_3d(as_map(&tm.state), smem_u32(st), 0, head * P + u * kUnitRows, 0);
                bulk_commit_group();
            }
        } else {
            if (four) stream_block<N, 4, false, JC>(rb, gx, cb, Bf, acc, j, aj, cx, cfr, g);
            else stream_block<N, 2, false, JC>(rb, gx, cb, Bf, acc, j, aj, cx, cfr, g);
            if (!stored && !SNAP && tb0 + kTB >= T) {   // nothing is written back: the stage is free once the rows have been read
                __syncwarp();
                if (lane == 0) refill();
            }
        }
        // ---- outputs of this token block.  The four column quarters of a sum meet by a reduce-scatter over
        //      the lanes (g, 0..3): two exchanges, after which lane (g, cq) holds row g + 8 cq = lane.
#pragma unroll
        for (int t = 0; t < kTB; ++t) {
            const int tt = tb0 + t;
            if (tt < T) {
                const float v0 = acc[t][0].x + acc[t][0].y, v1 = acc[t][1].x + acc[t][1].y;
                const float v2 = acc[t][2].x + acc[t][2].y, v3 = acc[t][3].x + acc[t][3].y;
                const bool up = (cq & 2) != 0, odd = (cq & 1) != 0;
                const float r0 = (up ? v2 : v0) + __shfl_xor_sync(FULL, up ? v0 : v2, 16);
                const float r1 = (up ? v3 : v1) + __shfl_xor_sync(FULL, up ? v1 : v3, 16);
                const float mine = (odd ? r1 : r0) + __shfl_xor_sync(FULL, odd ? r0 : r1, 8);
                float yat = ya[0], ywt = yw[0];   // ya[tt], yw[tt]: tt is tb0 + t with t known at compile time
#pragma unroll
                for (int q = 1; q < TC / kTB; ++q)
                    if (tb0 == q * kTB) { yat = ya[q * kTB + t]; ywt = yw[q * kTB + t]; }
                if (TC / kTB >= 1 && tb0 == 0) { yat = ya[t]; ywt = yw[t]; }
                const float y = fmaf(yat, mine, ywt);
                if (y_f32) reinterpret_cast<float *>(p.y)[y0 + (size_t)tt * HP] = y;
                else reinterpret_cast<__nv_bfloat16 *>(p.y)[y0 + (size_t)tt * HP] = __float2bfloat16_rn(y);
            }
        }
    }
    if (T == 0 && !SNAP) {   // no token at all: nothing to do with the rows
        if (lane == 0) refill();
    }

    const float *Bfull = reinterpret_cast<const float *>(slot + L.c_Bf);
    if (SNAP) {
        // Second snapshot (Algorithm 2 caches h_j and h_k): carry the rows on from position j to the end of
        // the block, h_T = (prod_{j<=r<T} a_r) h_j + sum_{j<=s<T} (dt_s prod_{s<r<T} a_r) xc_s B_s, in the
        // stage once the first store has read it, and store the result to the second buffer.
        if (stored) {
            if (lane == 0) bulk_wait_group_read0();
            __syncwarp();
        }
        const float aT = hc->alpha_jT;
        const float2 aT2 = make_float2(aT, aT);
        float cT[TC];
#pragma unroll
        for (int s = 0; s < TC; ++s) cT[s] = (s >= j && s < T) ? hc->wspT[s] * xc[s] : 0.f;
#pragma unroll 1
        for (int ps = 0; ps < PPL; ++ps) {
            const int pc = pc0 + ps;
            unsigned char *a = rb + (gx ^ (uint32_t)(ps << 4));
            float4 hv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 v = *reinterpret_cast<const float4 *>(a + 1024 * i);
                const float2 l = __fmul2_rn(lo2(v), aT2), h2 = __fmul2_rn(hi2(v), aT2);
                hv[i] = make_float4(l.x, l.y, h2.x, h2.y);
            }
#pragma unroll
            for (int s = 0; s < TC; ++s) {
                if (s >= j && s < T) {
                    const float4 bv = *reinterpret_cast<const float4 *>(Bfull + (size_t)s * N + pc * 4);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float c = __shfl_sync(FULL, cT[s], g + 8 * i);
                        const float2 c2 = make_float2(c, c);
                        const float2 l = ffma2(c2, lo2(bv), lo2(hv[i])), h2 = ffma2(c2, hi2(bv), hi2(hv[i]));
                        hv[i] = make_float4(l.x, l.y, h2.x, h2.y);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) *reinterpret_cast<float4 *>(a + 1024 * i) = hv[i];
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
            tma_store_3d(as_map(&tm.state_k), smem_u32(st), 0, head * P + u * kUnitRows, 0);
            bulk_commit_group();
        }
    }

    // ---- hand back the table slot (all lanes are done with it) and the stage (once the store has read it)
    __syncwarp();
    if (lane == 0) {
        mbar_arrive(smem_u32(&ctl.slot_empty[hs]));
        if (stored || SNAP) {
            bulk_wait_group_read0();
            refill();
        }
    }
    // ---- the conv window at the verified position: the last W-1 inputs up to token j-1 (Sec. 4.3 iii); for
    //      the second snapshot also the window after all T tokens.  Re-read from global memory (cache hits);
    //      every read of the old window comes before the first write.
    if (stored || SNAP) {
        const unsigned short *xg = reinterpret_cast<const unsigned short *>(p.x) + ((size_t)b * p.t_max * p.H + h) * P + row;
        const unsigned short *cg = reinterpret_cast<const unsigned short *>(p.conv_state) + (size_t)b * (kW - 1) * HP + h * P + row;
        unsigned short vj[kW - 1], vT[kW - 1];
#pragma unroll
        for (int wi = 0; wi < kW - 1; ++wi) {
            const int tj = j - (kW - 1) + wi, tT = T - (kW - 1) + wi;
            vj[wi] = tj < 0 ? cg[(kW - 1 + tj) * HP] : xg[tj * HP];
            vT[wi] = SNAP ? (tT < 0 ? cg[(kW - 1 + tT) * HP] : xg[tT * HP]) : (unsigned short)0;
        }
        if (stored) {
            unsigned short *out = reinterpret_cast<unsigned short *>(p.conv_state) + (size_t)b * (kW - 1) * HP + h * P + row;
#pragma unroll
            for (int wi = 0; wi < kW - 1; ++wi) out[wi * HP] = vj[wi];
        }
        if (SNAP) {
            unsigned short *out = reinterpret_cast<unsigned short *>(p.conv_state_k) + (size_t)b * (kW - 1) * HP + h * P + row;
#pragma unroll
            for (int wi = 0; wi < kW - 1; ++wi) out[wi * HP] = vT[wi];
        }
    }
    return true;
}

template <int N, int TC, int JC, bool SNAP>
__device__ __forceinline__ void compute_role(const VerifyParams &p, const StreamLayout &L, unsigned char *smem, Ctrl &ctl,
                                             const InputMaps &tm, const Work &w, int warp, int lane, RowIn<TC> &in) {
    // Warp w takes units w, w + AW, ... through its own stages w, w + AW, ... (S / AW of them, in turn): every
    // use of a stage is requested and waited for by the same warp, in order, so a wait is never more than one
    // phase behind its barrier, and no "empty" barrier is needed.
    int k = 0, ss = warp, sp = 0;
    for (int n = warp; n < w.nunits; n += L.AW, ++k) {
        int m, head, u;
        unit_of(w, n, m, head, u);
        const int hs = m % kSlots;
        const int b = div_H(w, head), h = head - b * w.H;
        const int j = pending_of(p, ctl, b), T = j + p.k;
        if (k > 0) load_row<TC>(p, b, h, u * kUnitRows + lane, T, in);   // (the first unit's loads went out at the start of the kernel)
        const bool ok = compute_unit<N, TC, JC, SNAP>(p, L, tm, ctl, smem + L.state_off + (size_t)ss * L.state_stride,
                                                       smem + L.tab_off + (size_t)hs * L.tab_stride, smem_u32(&ctl.state_full[ss]),
                                                       (uint32_t)sp, hs, m, ss, n + L.S, smem, w, head, b, h, u, j, T, lane, in);
        if (!ok) {   // a wait gave up
            if (lane == 0) {
                bulk_wait_group_read0();
                give_up(p, ctl);
            }
            return;
        }
        ss += L.AW;
        if (ss >= L.S) { ss = warp; sp ^= 1; }
    }
}

// ---------------------------------------------------------------- the kernel
template <int N, int TC, int JC, bool SNAP>
__global__ void __launch_bounds__(kThreads, 1)
verify_stream_kernel(const __grid_constant__ VerifyParams p, const __grid_constant__ StreamLayout L,
                     const __grid_constant__ InputMaps tm) {
    extern __shared__ __align__(1024) unsigned char smem[];
    Ctrl &ctl = *reinterpret_cast<Ctrl *>(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        make_work(p, L, *reinterpret_cast<Work *>(ctl.work));
        for (int s = 0; s < L.S; ++s) {
            mbar_init(smem_u32(&ctl.state_full[s]), 1);
            ctl.state_par[s] = -1;
        }
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&ctl.slot_empty[s]), (uint32_t)(p.P / kUnitRows));
            mbar_init(smem_u32(&ctl.slot_full[s]), 1);
            ctl.slot_ready[s] = 0;
        }
        ctl.abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const Work &w = *reinterpret_cast<const Work *>(ctl.work);   // left in shared memory: read where needed
    // Programmatic dependent launch.  Nothing touches global memory before everything launched earlier in the
    // stream has completed -- except, where the caller has promised that the kernel before this one does not
    // write this call's state, the first state requests: the rows then stream in while the previous kernel's
    // last CTAs finish.  The next kernel is let in only after the wait, so that its own early requests can
    // overlap with this kernel but with nothing older.
    const bool early = (p.flags & kFlagEarlyState) != 0;
    auto first_requests = [&]() {
        if (warp < L.AW && lane == 0)
            for (int n = warp, ss = warp; n < w.nunits && ss < L.S; n += L.AW, ss += L.AW) request_state<N>(p, L, smem, ctl, tm, w, n, ss, 0);
    };
    if (early) first_requests();
    {   // what every warp will load first, as prefetches
        const int tl = p.t_max < TC ? p.t_max : TC;
        if (tid < (p.batch < kJTable ? p.batch : kJTable)) prefetch_l2(p.n_prev + tid);
        if (warp >= kComputeWarps) {
            const int hw = warp - kComputeWarps;
            if (hw < w.nitems) prefetch_head<N, TC>(p, L, w, item_of(w, hw).head, lane);
            if (hw + kHeadWarps < w.nitems) prefetch_head<N, TC>(p, L, w, item_of(w, hw + kHeadWarps).head, lane);
        } else if (warp < L.AW && warp < w.nunits) {
            int m, head, u;
            unit_of(w, warp, m, head, u);
            const int b = div_H(w, head);
            prefetch_row<TC>(p, b, head - b * w.H, u * kUnitRows + lane, tl);
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Every warp sends its small loads first and the state requests behind them: behind the state requests of
    // 148 CTAs the small loads would wait for microseconds.
    const int ntab = p.batch < kJTable ? p.batch : kJTable;
    if (warp >= kComputeWarps) {
        const int hw = warp - kComputeWarps;
        HeadFrags<N, TC> f;
        if (hw < w.nitems) load_head<N, TC>(p, L, w, item_of(w, hw).head, lane, f);
#pragma unroll 1
        for (int i = tid; i < ntab; i += kThreads) ctl.jarr[i] = load_n_prev(p, i);
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
        head_role<N, TC, SNAP>(p, L, smem, ctl, w, hw, lane, f);
    } else {
        RowIn<TC> in;
        if (warp < L.AW && warp < w.nunits) {
            int m, head, u;
            unit_of(w, warp, m, head, u);
            const int b = div_H(w, head);
            // (the pending length is not known yet: all rows of the slab, those past the sequence's tokens are never used)
            load_row<TC>(p, b, head - b * w.H, u * kUnitRows + lane, p.t_max < TC ? p.t_max : TC, in);
            if (!early) first_requests();
        }
#pragma unroll 1
        for (int i = tid; i < ntab; i += kThreads) ctl.jarr[i] = load_n_prev(p, i);
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
        if (warp < L.AW) compute_role<N, TC, JC, SNAP>(p, L, smem, ctl, tm, w, warp, lane, in);
    }

    __syncthreads();
    if (ctl.abort && tid == 0) {
        // Some wait gave up.  Give every state load that was started a bounded chance to land before the
        // CTA's shared memory is released.
        for (int s = 0; s < L.S; ++s) {
            const long long t0 = clock64();
            if (ctl.state_par[s] >= 0)
                while (!mbar_try_park(smem_u32(&ctl.state_full[s]), (uint32_t)ctl.state_par[s], 20000u) &&
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

// fp32 state [rows][N] as [32 columns][rows][N/32 quarters], boxes of one unit's rows, 128-byte swizzle
bool encode_state(EncodeTiledFn fn, TensorMapBytes *map, const void *base, size_t rows, int N) {
    const cuuint64_t dims[3] = {32, (cuuint64_t)rows, (cuuint64_t)(N / 32)};
    const cuuint64_t strides[2] = {(cuuint64_t)N * 4, 128};
    const cuuint32_t box[3] = {32, (cuuint32_t)kUnitRows, (cuuint32_t)(N / 32)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(reinterpret_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int N, int TC, int JC, bool SNAP>
cudaError_t launch_variant(const VerifyParams &p, const StreamPlan &plan, const InputMaps &tm, cudaStream_t stream) {
    auto kern = verify_stream_kernel<N, TC, JC, SNAP>;
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
    if (p.W != kW) return reject("conv width is not 4");
    if (p.N != 64 && p.N != 128) return reject("state dim is not 64 or 128");
    if (p.P % kUnitRows || p.P > 256) return reject("head dim is not a multiple of 32 up to 256");
    if (p.H % 8) return reject("head count is not a multiple of 8");
    const int t_cap = p.j_cap + p.k;
    if (t_cap > kMaxT || p.j_cap > kMaxJ) return reject("more than 16 token rows or more than 8 replayed tokens");
    const int N = p.N, P = p.P;
    StreamLayout &L = plan.layout;
    L.TCAP = t_cap <= 8 ? 8 : 16;
    const bool snap = p.state_k != nullptr;
    L.JB = snap ? L.TCAP : (p.j_cap < 1 ? 1 : p.j_cap);
    L.hpg_b = p.H / p.GB;
    L.hpg_c = p.H / p.GC;
    L.H_mul = (unsigned)((0x100000000ull + (unsigned)p.H - 1) / (unsigned)p.H);
    L.uph_mul = (unsigned)((0x100000000ull + (unsigned)(P / kUnitRows) - 1) / (unsigned)(P / kUnitRows));
    // a table slot: what a head warp leaves for the compute warps
    int o = 0;
    L.c_Cf = o;  o += L.TCAP * N * 4;
    L.c_Bf = o;  o += L.JB * N * 4;
    L.c_G = o;   o += kMaxT * kMaxT * 4;
    L.c_hc = o;  o += (int)sizeof(HeadConst);
    L.tab_stride = align128(o);
    L.state_stride = kUnitRows * N * 4;
    L.state_off = kCtrlBytes;

    const long long uph = P / kUnitRows, nunits = (long long)p.batch * p.H * uph;
    if (nunits >= (1ll << 30)) return reject("more than 2^30 units");
    if ((long long)p.batch * p.H * p.H >= (1ll << 31)) return reject("batch x heads^2 beyond the range of the index arithmetic");
    if (nunits < 1) return reject("empty problem");
    long long grid = sm_count < nunits ? sm_count : nunits;
    const long long per_cta = (nunits + grid - 1) / grid;
    // Shared memory: the table slots, the rest for state stages -- as many as fit, but no
    // more than the CTA has units; every stage belongs to one compute warp, so there are as many warps in use
    // as stages, or two stages per warp.
    const long long left = (long long)smem_per_block_optin - kCtrlBytes - (long long)kSlots * L.tab_stride;
    int S = left > 0 ? (int)(left / L.state_stride) : 0;
    if (S < 2) return reject("not enough shared memory for two state stages");
    if (S > per_cta) S = per_cta < 2 ? 2 : (int)per_cta;
    if (S > kComputeWarps) S = S >= 2 * kComputeWarps ? 2 * kComputeWarps : kComputeWarps;
    L.S = S;
    L.AW = S < kComputeWarps ? S : kComputeWarps;
    L.tab_off = L.state_off + S * L.state_stride;

    plan.ok = true;
    plan.grid = (int)grid;
    const int JC = p.j_cap <= 4 ? 4 : 8;
    plan.variant = (N == 128 ? 0 : 8) + (L.TCAP == 8 ? 0 : 4) + (JC == 4 ? 0 : 2) + (snap ? 1 : 0);
    plan.smem_bytes = (size_t)L.tab_off + (size_t)kSlots * L.tab_stride;
    snprintf(plan.name, sizeof plan.name, "stream<N=%d,TC=%d,JC=%d,snap=%d,S=%d,AW=%d,grid=%d>", N, L.TCAP, JC, snap ? 1 : 0, L.S, L.AW, (int)grid);
    return plan;
}

bool encode_stream_maps(const VerifyParams &p, const StreamPlan &plan, InputMaps *tm) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    (void)plan;
    const size_t srows = (size_t)p.batch * p.H * p.P;
    memset(tm, 0, sizeof *tm);
    bool ok = encode_state(fn, &tm->state, p.state, srows, p.N);
    if (p.state_k) ok = ok && encode_state(fn, &tm->state_k, p.state_k, srows, p.N);
    else memcpy(&tm->state_k, &tm->state, sizeof(TensorMapBytes));
    return ok;
}

cudaError_t launch_verify_stream(const VerifyParams &p, const StreamPlan &plan, const InputMaps &tm, cudaStream_t stream) {
    switch (plan.variant) {   // bit 3: N = 64; bit 2: 16 token rows; bit 1: up to 8 replayed tokens; bit 0: second snapshot
        case 0: return launch_variant<128, 8, 4, false>(p, plan, tm, stream);
        case 1: return launch_variant<128, 8, 4, true>(p, plan, tm, stream);
        case 2: return launch_variant<128, 8, 8, false>(p, plan, tm, stream);
        case 3: return launch_variant<128, 8, 8, true>(p, plan, tm, stream);
        case 4: return launch_variant<128, 16, 4, false>(p, plan, tm, stream);
        case 5: return launch_variant<128, 16, 4, true>(p, plan, tm, stream);
        case 6: return launch_variant<128, 16, 8, false>(p, plan, tm, stream);
        case 7: return launch_variant<128, 16, 8, true>(p, plan, tm, stream);
        case 8: return launch_variant<64, 8, 4, false>(p, plan, tm, stream);
        case 9: return launch_variant<64, 8, 4, true>(p, plan, tm, stream);
        case 10: return launch_variant<64, 8, 8, false>(p, plan, tm, stream);
        case 11: return launch_variant<64, 8, 8, true>(p, plan, tm, stream);
        case 12: return launch_variant<64, 16, 4, false>(p, plan, tm, stream);
        case 13: return launch_variant<64, 16, 4, true>(p, plan, tm, stream);
        case 14: return launch_variant<64, 16, 8, false>(p, plan, tm, stream);
        case 15: return launch_variant<64, 16, 8, true>(p, plan, tm, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace mspec
