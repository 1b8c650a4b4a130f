#pragma once
// AdaScale SGD gain-ratio step for sm_100a: device code (the host glue is in adascale.cu).
//
// Two kernels make up one iteration (paper: Sec. 3.2, App. B.3, Eq. 2-3):
//   reduce  - streams the S x P gradient matrix once through shared memory (bulk asynchronous
//             copies completed on mbarriers, a producer warp and eight consumer warps), writes
//             the mean gradient and pairs (sum of squared deviations, squared norm of the mean)
//             per block or per run of tiles, and prepares the part of the scalar step that
//             depends only on the state the iteration starts from.
//   update  - every block adds up the pairs (for large jobs a 64-block kernel, k_sum, has brought
//             them down to a few dozen first) and completes the scalar part (estimates, clamps,
//             moving averages, r_t, eta_t, tau_{t+1}); then v <- rho v + (gbar + lambda w),
//             w <- w - eta_t v.
// Where no update kernel follows (one-pass form, sharded form, a reduce call on its own) the
// pairs are added up and the scalar part completed by the reduce kernel's last block or by the
// one-block kernels k_finish / k_scalar.
// Three trivial streaming kernels calibrate the bandwidth ceiling.
// The path is bound by HBM bandwidth; there is no contraction, hence no tensor-core work.
//
// Work distribution: every tensor is cut into tiles.  Small jobs: tile t belongs to block
// t mod gridDim.  Large jobs: runs of consecutive tiles (reduce) or single tiles (update) are
// handed to the blocks from a device counter as they become free.  Either way all blocks
// advance through each array as one narrow front, which keeps DRAM pages hot, and the sums are
// added up in an order that does not depend on how the hardware schedules blocks, so they are
// reproducible from run to run.
#include "../../include/adascale.h"

#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

namespace {

constexpr int kThreads = 256;             // consumer threads of the reduce kernel, all threads of the update kernel
constexpr int kWarps = kThreads / 32;
constexpr int kStagedThreads = kThreads + 32;  // + 1 producer warp
constexpr int kStagedWarps = kStagedThreads / 32;
constexpr int kStages = 3;                // most shared-memory stages per block (a launch uses 2 or 3)
// Rows of one stage; larger S goes through in row chunks.  Eight rows of up to 4 KB measured
// fastest for both element types (bf16: 8 rows of 4 KB beat 16 rows of 2 KB once tiles were
// handed out dynamically).
__host__ __device__ constexpr int max_rows_per_stage(int) { return 8; }
constexpr int kStageBytes = 32 * 1024;    // upper bound of one stage
constexpr int kReduceBlocksPerSM = 2;
constexpr int kUpdateVecs = 2;            // 128-bit accesses per array, thread and tile of the update kernel
constexpr int kUpdateBlocksPerSM = 4;
constexpr long long kDynamicMinTiles = 32768;  // staged tiles from which they are handed out from a counter
constexpr int kSlots = kStages + 1;       // tiles of a block whose sums can be on their way at once
static_assert(kSlots == 4, "the producer keeps the tile index of each slot in four named registers");
constexpr int kSumBlocks = 64;            // blocks of the kernel that adds up the run pairs of a large job
constexpr int kScalarTile = 2048;         // elements per tile on the unaligned / ragged-tail path
constexpr int kUpdateTile = 1024 * kUpdateVecs;  // elements per tile of the update kernel
constexpr int kGbarAlign = 64;            // every tensor's mean gradient starts on a 256-byte boundary
constexpr int kRing = 4;                  // pinned staging slots for pointer-table uploads
constexpr int kMaxS = 4096;
constexpr unsigned kSpinLimit = 1u << 22; // bounded waits: give up, flag, leave (default of the handshake waits,
                                          // fixed bound of the wait for copies that are already in flight)
constexpr unsigned long long kWaitNs = 2000000000ull;  // and no wait lasts longer than two seconds
constexpr unsigned kWaitHintNs = 20000;   // how long one poll of a barrier may sleep (it wakes on completion)

typedef unsigned long long u64;

// Scalar state kept on the device between iterations.
struct DevState {
    double tau;    // scale-invariant iteration tau_t
    double avg_a;  // sigma_bar^2 (ratio estimator: m1)
    double avg_b;  // mu_bar^2    (ratio estimator: m2)
    long long n;   // samples absorbed by the averages
    long long t;   // iterations applied
    long long skipped;
    double r, eta, lr;
    double sigma2_raw, mu2_raw;
    double N, D;
    unsigned status;
    unsigned fault;  // sticky: a bounded device-side wait gave up
};
static_assert(sizeof(DevState) == 112, "the snapshot copied to the host is 112 bytes");

// What an iteration's scalar part reads of the state it starts from.
struct RawState {
    double tau, avg_a, avg_b;
    long long n, t, skipped;
};

// What the second half of the scalar part needs of the first (see scalar_prepare).
struct ScalarPrep {
    RawState s;
    double lr;       // lr(floor(tau_t)), App. B.1
    double th;       // weight of the old average: min(theta, 1 - 1/n), plain mean of the first samples (App. B.3)
    double r_prior;  // gain from the averages of prior iterations (r_0 = 1)
    double inv_S, inv_Sm1;  // 1/S and 1/(S-1): the second half multiplies where the formulas divide
};

struct ScalarCfg {
    double eps, theta;  // theta already resolved on the host (the paper's rule follows S)
    unsigned flags;
    int S;
};

struct Sched {
    int kind, n;
    double eta0, decay, t_s1;
    double w[ADASCALE_MAX_MILESTONES];
};

// One tile of work: `len` elements of tensor `tensor` starting at element `first`; `goff` is
// where the tile's mean gradient lives in the library's workspace.  The descriptors hold no
// pointers, so they change only with the tiling.
struct __align__(16) TileDesc {
    long long first;
    long long goff;
    int tensor;
    int len;
    int pad[2];
};

// What the producer warp tells the consumers about the contents of a stage.
struct StageInfo {
    long long first;  // first element within its tensor
    long long goff;   // where its mean gradient lives
    float *w, *v;     // fused mode: the tensor's parameters and momentum
    unsigned wflag;   // fused mode: bit0: both 16-byte aligned
    int len;          // columns; < 0: no tile follows
};

// Reduce kernel: a tensor whose S row pointers are 16-byte aligned contributes staged tiles of
// kThreads * CPT columns for its first numel & ~7 elements and one scalar tile for the ragged
// rest; any other tensor contributes only scalar tiles of kScalarTile elements.
struct ReduceArgs {
    const u64 *gptr;          // [S * T] row pointers
    const TileDesc *tiles;    // staged tiles
    const TileDesc *stiles;   // scalar-path tiles
    long long n_tiles, n_stiles;
    float *gbar;
    const u64 *wv;            // fused mode only: [2 * T] parameters then momentum
    const unsigned *wflags;   // fused mode only: [T] bit0: both pointers 16-byte aligned
    float rho, lambda;        // fused mode only
    double2 *partials;        // [grid] sums over each block's scalar-path tiles
    double2 *run_partials;    // sums of the staged tiles, one pair per run (run_tiles > 0)
    long long run_tiles;      // consecutive staged tiles handed out together; 0: static assignment
    long long long_runs;      // the first long_runs runs have run_tiles tiles, every later run a single tile
    unsigned stages;          // shared-memory stages in use, 2 .. kStages
    unsigned *ticket;
    u64 *tile_counter;        // runs handed out beyond each block's first; zero between launches
    DevState *st;
    double *sums_out;         // not null: write (D, N) there and leave the scalar part to k_scalar
    ScalarPrep *prepared;     // block 0 leaves the first half of the scalar part here, for whoever runs the second
    unsigned leave_open;      // non-zero: that is the next kernel (see k_update), and no block stays behind at the end
    unsigned spin_limit;      // bound of the producer / consumer handshake waits
    unsigned early_rows;      // non-zero: the gradient rows may be read before griddepcontrol.wait
    int S, T;
    float invS, fS;
    ScalarCfg sc;
    Sched sched;
};

// Scalar part on its own, for sums that were completed outside the reduce kernel.
struct ScalarArgs {
    DevState *st;
    const double *sums;       // [0] = sum_i ||g_i - gbar||^2, [1] = ||gbar||^2, over ALL shards
    ScalarCfg sc;
    Sched sched;
};

struct UpdateArgs {
    const u64 *wv;            // [2 * T]: parameters then momentum
    const unsigned *wflags;   // [T] bit0: both pointers 16-byte aligned
    const TileDesc *tiles;    // tiles of kUpdateTile elements
    long long n_tiles;
    const float *gbar;
    DevState *st;
    unsigned *next_tile;      // tiles handed out beyond each block's first; wraps to zero by itself
    int T;
    float rho, lambda;
    // only when the reduce kernel left the scalar part of the iteration to this one
    const double2 *partials;  // one pair per block of the reduce launch
    int n_partials;
    const ScalarPrep *prepared;  // first half of the scalar part, left by the reduce launch
    ScalarCfg sc;
};

// First level of the sum over the run pairs of a large job (see k_sum).
struct SumArgs {
    const double2 *run_partials;
    long long n_pairs;
    double2 *out;        // one pair per block of the launch
    u64 *tile_counter;   // the reduce launch's run counter, put back to zero here
};

// The scalar part as a kernel of one block, when no update follows a reduce launch that left it open.
struct FinishArgs {
    DevState *st;
    const double2 *partials;
    int n_partials;
    const ScalarPrep *prepared;
    ScalarCfg sc;
};

// Streaming 128-bit load (read once, evict first): used by the bandwidth probes.
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 r;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// Element types of the gradient rows.  A bf16 is the upper half of an fp32, so widening is a
// shift and exact.
template <int DT> struct Elem;
template <> struct Elem<ADASCALE_F32> {
    static constexpr int kBytes = 4;
    static __device__ __forceinline__ float load1(const void *p) { return __ldcs((const float *)p); }
};
template <> struct Elem<ADASCALE_BF16> {
    static constexpr int kBytes = 2;
    static __device__ __forceinline__ float load1(const void *p)
    {
        return __uint_as_float((unsigned)__ldcs((const unsigned short *)p) << 16);
    }
};

// d = x - c, blocked first moment, running second moment, for V columns of one row.
template <int V>
__device__ __forceinline__ void accumulate_row(const float *x, const float *c, float *p1, float *s2)
{
#pragma unroll
    for (int k = 0; k < V; ++k) {
        const float d = x[k] - c[k];
        p1[k] += d;
        s2[k] = fmaf(d, d, s2[k]);
    }
}

// One column, any alignment, any S: plain two-pass with a residual correction of the mean.
// Row pointers come straight from the device table.
template <int DT>
__device__ __forceinline__ void column_scalar(const u64 *gptr, int T, int tensor, size_t boff, int S,
                                                     float fS, float *gb, float &dsum, float &nsum)
{
    float sum = 0.f;
    for (int i = 0; i < S; ++i) sum += Elem<DT>::load1((const char *)gptr[(size_t)i * T + tensor] + boff);
    const float m0 = sum / fS;
    float e = 0.f, qq = 0.f;
    for (int i = 0; i < S; ++i) {
        const float d = Elem<DT>::load1((const char *)gptr[(size_t)i * T + tensor] + boff) - m0;
        e += d;
        qq = fmaf(d, d, qq);
    }
    const float corr = e / fS;
    const float m = m0 + corr;
    *gb = m;
    dsum = fmaf(-corr, e, qq);
    nsum = m * m;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// Fixed-shape block sum of two doubles over NW warps; result valid in thread 0.
template <int NW = kWarps>
__device__ __forceinline__ void block_sum2(double &a, double &b, double *sa, double *sb)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    a = warp_sum(a);
    b = warp_sum(b);
    __syncthreads();  // scratch may still be in use by a previous call
    if (lane == 0) {
        sa[warp] = a;
        sb[warp] = b;
    }
    __syncthreads();
    if (warp == 0) {
        a = lane < NW ? sa[lane] : 0.0;
        b = lane < NW ? sb[lane] : 0.0;
        a = warp_sum(a);
        b = warp_sum(b);
    }
}

// App. B.1
__device__ double lr_eval(const Sched &s, double t)
{
    if (s.kind == ADASCALE_LR_EXP) return s.eta0 * pow(s.decay, t / s.t_s1);
    if (s.kind == ADASCALE_LR_STEP) {
        double f = 1.0;  // decay^(milestones passed), by repeated multiplication
        for (int i = 0; i < s.n; ++i) f = (t > s.w[i]) ? f * s.decay : f;
        return s.eta0 * f;
    }
    return s.eta0;
}

// The scalar part of an iteration in two halves.  Everything that depends only on the state the
// iteration starts from (the schedule's value at tau_t, the averaging weight, the gain of the lagged
// form) can be worked out while the gradient rows are still being read; what is left once the two
// sums are known is a handful of operations and one division.  Every path (the last block of the
// reduce kernel, the update kernel, the scalar kernels) runs these same two functions.

__device__ __forceinline__ RawState raw_state(const DevState *st)
{
    RawState s;
    s.tau = st->tau;
    s.avg_a = st->avg_a;
    s.avg_b = st->avg_b;
    s.n = st->n;
    s.t = st->t;
    s.skipped = st->skipped;
    return s;
}

// What another kernel left for this one, read from L2.
__device__ __forceinline__ ScalarPrep load_prepared(const ScalarPrep *q)
{
    static_assert(sizeof(ScalarPrep) == 11 * 8, "eleven 8-byte fields");
    ScalarPrep p;
    const long long *src = reinterpret_cast<const long long *>(q);
    long long *dst = reinterpret_cast<long long *>(&p);
#pragma unroll
    for (int i = 0; i < 11; ++i) dst[i] = __ldcg(src + i);
    return p;
}

__device__ ScalarPrep scalar_prepare(const RawState &s, const ScalarCfg &c, const Sched &sched)
{
    ScalarPrep p;
    p.s = s;
    const double t_arg = (c.flags & ADASCALE_FLAG_CONT_TAU) ? s.tau : floor(s.tau);
    p.lr = lr_eval(sched, t_arg);
    const double S = (double)c.S;
    const double warm = 1.0 - 1.0 / (double)(s.n + 1);
    p.th = c.theta < warm ? c.theta : warm;
    p.inv_S = 1.0 / S;
    p.inv_Sm1 = c.S > 1 ? 1.0 / (S - 1.0) : 0.0;
    p.r_prior = 1.0;  // wanted by the lagged form only
    if ((c.flags & ADASCALE_FLAG_LAGGED) && c.S > 1 && s.n > 0)
        p.r_prior = (c.flags & ADASCALE_FLAG_RATIO) ? (s.avg_a + c.eps) / (s.avg_b + c.eps)
                                                    : (s.avg_a + s.avg_b) / fma(s.avg_a, p.inv_S, s.avg_b);
    return p;
}

// explicit roundings here and explicit fused operations below: the same value whichever kernel
// the function is compiled into
__device__ __forceinline__ double ema(double prev, double sample, double th)
{
    return __dadd_rn(__dmul_rn(th, prev), __dmul_rn(__dsub_rn(1.0, th), sample));
}

// Second half: from the two sums to r_t, eta_t, tau_{t+1}.  Returns eta_t (0 when the iteration is
// skipped); writes the state when st is given.  One thread, fp64, no host involvement.
__device__ double scalar_finish(DevState *st, const ScalarPrep &p, const ScalarCfg &c, double D, double N,
                                             unsigned fault, bool &skip)
{
    if (st) {
        st->D = D;
        st->N = N;
    }
    skip = true;
    if (fault) {  // a bounded wait gave up somewhere: the sums are incomplete, nothing is applied
        if (st) {
            st->skipped = p.s.skipped + 1;
            st->eta = 0.0;
        }
        return 0.0;
    }
    if (!isfinite(D) || !isfinite(N)) {  // skip the iteration, leave every average and tau alone
        if (st) {
            st->status = ADASCALE_STATUS_NONFINITE;
            st->skipped = p.s.skipped + 1;
            st->eta = 0.0;
        }
        return 0.0;
    }
    skip = false;
    double r, sigma2_raw, mu2_raw, na = p.s.avg_a, nb = p.s.avg_b;
    long long n = p.s.n;
    if (c.S == 1) {  // App. A.2: unit gain at scale one
        sigma2_raw = 0.0;
        mu2_raw = N;
        r = 1.0;
    } else {
        double a, b;
        const bool ratio = (c.flags & ADASCALE_FLAG_RATIO) != 0;
        if (ratio) {
            // Sec. 3.4: (1/S) sum_i ||g_i||^2 = D/S + N  and ||gbar||^2
            a = fma(D, p.inv_S, N);
            b = N;
            sigma2_raw = a;
            mu2_raw = b;
        } else {
            // App. B.3: sigma^2 = D/(S-1) equals 1/(S-1) sum||g_i||^2 - S/(S-1)||gbar||^2
            const double sigma2 = D * p.inv_Sm1;
            const double mu2 = fma(-sigma2, p.inv_S, N);
            sigma2_raw = sigma2;
            mu2_raw = mu2;
            a = sigma2 > c.eps ? sigma2 : c.eps;
            b = mu2 > 0.0 ? mu2 : 0.0;
        }
        n = p.s.n + 1;
        na = ema(p.s.avg_a, a, p.th);
        nb = ema(p.s.avg_b, b, p.th);
        if (c.flags & ADASCALE_FLAG_LAGGED)
            r = p.r_prior;
        else
            r = ratio ? (na + c.eps) / (nb + c.eps) : (na + nb) / fma(na, p.inv_S, nb);  // Eq. 3
    }
    const double eta = r * p.lr;  // Sec. 3.2
    if (st) {
        st->status = 0;
        st->sigma2_raw = sigma2_raw;
        st->mu2_raw = mu2_raw;
        st->n = n;
        st->avg_a = na;
        st->avg_b = nb;
        st->r = r;
        st->lr = p.lr;
        st->eta = eta;
        st->tau = p.s.tau + r;
        st->t = p.s.t + 1;
    }
    return eta;
}

// Both halves in one go, on the state in place.
__device__ void scalar_step(DevState *st, const ScalarCfg &c, const Sched &sched, double D, double N)
{
    const ScalarPrep p = scalar_prepare(raw_state(st), c, sched);
    bool skip;
    scalar_finish(st, p, c, D, N, __ldcg(&st->fault), skip);
}

// Programmatic dependent launch: a kernel lets its successor in the stream be scheduled
// early, and waits for its predecessor (completion and visibility of its writes) only where
// it first depends on it.  Both are no-ops for a launch without the attribute.
//
// Ordering rule of this library: a kernel triggers its dependents only AFTER its own
// griddepcontrol.wait has returned.  A kernel can start no earlier than its predecessor's
// trigger, so by induction, when a kernel of this library starts, every kernel that precedes
// its predecessor in the stream has completed and its writes are visible.  What a kernel
// touches before its own wait must therefore be data that its immediate predecessor does not
// write: the update kernel's first w and v values (last written by the update before the
// preceding reduce), and, only when the caller vouches for them, the gradient rows.
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u64 *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u64 *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(u64 *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ u64 global_ns()
{
    u64 t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Returns false if the phase did not complete within `limit` polls or within kWaitNs of wall
// time, whichever comes first (one poll can itself suspend the thread for a while, so a poll
// count alone does not bound the time).  Each poll may sleep up to kWaitHintNs and wakes when
// the phase completes: with the default (much shorter) sleep a third of all instructions the
// reduce kernel issued were polls of waiting warps, and it ran 0.4 % slower.
__device__ __forceinline__ bool mbar_wait(u64 *bar, unsigned parity, unsigned limit)
{
    const unsigned addr = smem_u32(bar);
    u64 t0 = 0;
    for (unsigned spin = 0; spin < limit; ++spin) {
        unsigned done;
asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done)
                     : "r"(addr), "r"(parity), "r"(kWaitHintNs)
                     : "memory");
        if (done) return true;
        if ((spin & 63u) == 63u) {
            const u64 now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNs) return false;
        }
    }
    return false;
}
// global -> shared bulk copy; bytes and both addresses are multiples of 16.  The rows are read
// once: evict-first in L2 leaves the cache to the mean gradient that the update reads next.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned bytes, u64 *bar, u64 policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
                 : "memory");
}

// ---- packed fp32 pairs -------------------------------------------------------------------
// sm_100 adds, subtracts and multiply-adds two fp32 values with one instruction (f32x2).  The
// consumer loop of the reduce kernel keeps its per-column state in such pairs: same IEEE
// operations in the same order as scalar code, half the instruction issue.
typedef unsigned long long f2;

__device__ __forceinline__ f2 pack2(float lo, float hi)
{
    f2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f2 v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f2 add2(f2 a, f2 b)
{
    f2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f2 sub2(f2 a, f2 b)
{
    f2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c)
{
    f2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// a bf16 pair in one 32-bit word -> two fp32 (widening is a shift / a mask, exact)
__device__ __forceinline__ f2 widen2(unsigned u)
{
    f2 r;
    asm("{\n\t.reg .b32 lo, hi;\n\tshl.b32 lo, %1, 16;\n\tand.b32 hi, %1, 0xffff0000;\n\tmov.b64 %0, {lo, hi};\n\t}"
        : "=l"(r)
        : "r"(u));
    return r;
}

// CPT columns of one staged row, from shared memory (32-bit shared address plus a
// compile-time byte offset), as CPT/2 packed pairs.
template <int DT, int CPT> struct PairLoad;
template <int CPT> struct PairLoad<ADASCALE_F32, CPT> {
    template <int OFF>
    static __device__ __forceinline__ void load(unsigned addr, f2 *x)
    {
        if constexpr (CPT == 2) {
            asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(x[0]) : "r"(addr), "n"(OFF));
        } else {
#pragma unroll
            for (int k = 0; k < CPT / 4; ++k)
                asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];"
                             : "=l"(x[2 * k]), "=l"(x[2 * k + 1])
                             : "r"(addr + 16 * k), "n"(OFF));
        }
    }
};
template <int CPT> struct PairLoad<ADASCALE_BF16, CPT> {
    template <int OFF>
    static __device__ __forceinline__ void load(unsigned addr, f2 *x)
    {
        if constexpr (CPT == 4) {
            unsigned u0, u1;
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2+%3];" : "=r"(u0), "=r"(u1) : "r"(addr), "n"(OFF));
            x[0] = widen2(u0);
            x[1] = widen2(u1);
        } else {
            unsigned u0, u1, u2, u3;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+%5];"
                         : "=r"(u0), "=r"(u1), "=r"(u2), "=r"(u3)
                         : "r"(addr), "n"(OFF));
            x[0] = widen2(u0);
            x[1] = widen2(u1);
            x[2] = widen2(u2);
            x[3] = widen2(u3);
        }
    }
};

// What a thread holds of two adjacent columns of a row before the shift is subtracted.
template <int DT> struct Held { typedef f2 type; };                       // fp32: the packed pair
template <> struct Held<ADASCALE_BF16> { typedef unsigned type; };       // bf16: the raw word

// CPT bf16 columns of one staged row as CPT/2 raw 32-bit words (two elements each).
template <int CPT, int OFF>
__device__ __forceinline__ void load_words(unsigned addr, unsigned *u)
{
    if constexpr (CPT == 4)
        asm volatile("ld.shared.v2.b32 {%0, %1}, [%2+%3];" : "=r"(u[0]), "=r"(u[1]) : "r"(addr), "n"(OFF));
    else
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+%5];"
                     : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3])
                     : "r"(addr), "n"(OFF));
}
// Median of three, on both bf16 elements of a word at once.  The median of three bf16 values is
// one of them, so taking it before widening is exact; like fminf / fmaxf, the packed min / max
// return the other operand when one is NaN.
__device__ __forceinline__ unsigned median3_bf16x2(unsigned a, unsigned b, unsigned e)
{
    unsigned r;
    asm("{\n\t.reg .b32 lo, hi, t;\n\t"
        "min.bf16x2 lo, %1, %2;\n\tmax.bf16x2 hi, %1, %2;\n\t"
        "min.bf16x2 t, hi, %3;\n\tmax.bf16x2 %0, lo, t;\n\t}"
        : "=r"(r)
        : "r"(a), "r"(b), "r"(e));
    return r;
}
// x - c for the two bf16 elements of one 32-bit word.  sm_100 subtracts an fp32 from a bf16
// operand in one instruction (the operand is widened exactly, the difference rounded once: the
// same result as widening first), so no shift or mask is spent per element.
__device__ __forceinline__ f2 sub2_bf16(unsigned u, f2 c)
{
    f2 r;
    asm("{\n\t.reg .b16 xl, xh;\n\t.reg .f32 cl, ch, dl, dh;\n\t"
        "mov.b32 {xl, xh}, %1;\n\tmov.b64 {cl, ch}, %2;\n\t"
        "sub.rn.f32.bf16 dl, xl, cl;\n\tsub.rn.f32.bf16 dh, xh, ch;\n\t"
        "mov.b64 %0, {dl, dh};\n\t}"
        : "=l"(r)
        : "r"(u), "l"(c));
    return r;
}

// A row that is already in registers (raw words for bf16, packed pairs for fp32) into the running sums.
template <int DT, int CPT>
__device__ __forceinline__ void consume_held(const typename Held<DT>::type *x, const f2 *c, f2 *p1, f2 *s2)
{
#pragma unroll
    for (int j = 0; j < CPT / 2; ++j) {
        f2 d;
        if constexpr (DT == ADASCALE_BF16) d = sub2_bf16(x[j], c[j]);
        else d = sub2(x[j], c[j]);
        p1[j] = add2(p1[j], d);
        s2[j] = fma2(d, d, s2[j]);
    }
}

// One staged row into the running sums: d = x - c, p1 += d, s2 += d * d.
template <int DT, int CPT, int OFF>
__device__ __forceinline__ void consume_row(unsigned addr, const f2 *c, f2 *p1, f2 *s2)
{
    f2 d[CPT / 2];
    if constexpr (DT == ADASCALE_BF16) {
        unsigned u[CPT / 2];
        load_words<CPT, OFF>(addr, u);
#pragma unroll
        for (int j = 0; j < CPT / 2; ++j) d[j] = sub2_bf16(u[j], c[j]);
    } else {
        f2 x[CPT / 2];
        PairLoad<DT, CPT>::template load<OFF>(addr, x);
#pragma unroll
        for (int j = 0; j < CPT / 2; ++j) d[j] = sub2(x[j], c[j]);
    }
#pragma unroll
    for (int j = 0; j < CPT / 2; ++j) {
        p1[j] = add2(p1[j], d[j]);
        s2[j] = fma2(d[j], d[j], s2[j]);
    }
}

template <int DT, int CPT> struct Cols;
template <int CPT> struct Cols<ADASCALE_F32, CPT> {
    static __device__ __forceinline__ void load(const char *p, float *x)
    {
        if constexpr (CPT == 1) {
            x[0] = *(const float *)p;
        } else if constexpr (CPT == 2) {
            const float2 t = *(const float2 *)p;
            x[0] = t.x; x[1] = t.y;
        } else {
#pragma unroll
            for (int k = 0; k < CPT; k += 4) {
                const float4 t = *(const float4 *)(p + 4 * k);
                x[k] = t.x; x[k + 1] = t.y; x[k + 2] = t.z; x[k + 3] = t.w;
            }
        }
    }
};
template <int CPT> struct Cols<ADASCALE_BF16, CPT> {
    static __device__ __forceinline__ void widen(unsigned u, float *x)
    {
        x[0] = __uint_as_float(u << 16);
        x[1] = __uint_as_float(u & 0xffff0000u);
    }
    static __device__ __forceinline__ void load(const char *p, float *x)
    {
        if constexpr (CPT == 2) {
            widen(*(const unsigned *)p, x);
        } else if constexpr (CPT == 4) {
            const uint2 t = *(const uint2 *)p;
            widen(t.x, x); widen(t.y, x + 2);
        } else {
            const uint4 t = *(const uint4 *)p;
            widen(t.x, x); widen(t.y, x + 2); widen(t.z, x + 4); widen(t.w, x + 6);
        }
    }
};

// The mean gradient is read again by the update kernel right after the reduce kernel ends and
// overwritten by the next iteration: stored with the evict-last L2 priority it survives the
// stream of gradient rows (which are evict-first) and mostly never travels to DRAM and back.
__device__ __forceinline__ u64 l2_keep_policy()
{
    u64 p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ void store_pair_keep(double2 *p, double x, double y, u64 policy)
{
    asm volatile("st.global.L2::cache_hint.v2.f64 [%0], {%1, %2}, %3;" ::"l"(p), "d"(x), "d"(y), "l"(policy) : "memory");
}

template <int CPT>
__device__ __forceinline__ void store_cols_keep(float *g, const float *m, u64 policy)
{
    if constexpr (CPT == 2) {
        asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1, %2}, %3;" ::"l"(g), "f"(m[0]), "f"(m[1]), "l"(policy)
                     : "memory");
    } else {
#pragma unroll
        for (int k = 0; k < CPT; k += 4)
            asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(g + k), "f"(m[k]),
                         "f"(m[k + 1]), "f"(m[k + 2]), "f"(m[k + 3]), "l"(policy)
                         : "memory");
    }
}

template <int CPT>
__device__ __forceinline__ void store_cols(float *g, const float *m)
{
    if constexpr (CPT == 1) {
        g[0] = m[0];
    } else if constexpr (CPT == 2) {
        *(float2 *)g = make_float2(m[0], m[1]);
    } else {
#pragma unroll
        for (int k = 0; k < CPT; k += 4) *(float4 *)(g + k) = make_float4(m[k], m[k + 1], m[k + 2], m[k + 3]);
    }
}


// ---------------------------------------------------------------------------------------
// Reduce kernel.
//
// Per column the S values are shifted by a value c taken from the data:  d_i = g_i - c.
// With s1 = sum d_i and s2 = sum d_i^2 the mean is c + s1/S and the summed squared
// deviation is s2 - s1^2/S.  Because c is (close to) a sample, the subtraction loses a
// factor of order S at worst, not the |mean|^2/sigma^2 that the raw formula of App. B.3
// loses; identical rows give exactly zero; and each row is consumed as it is read.
//   - c is the median of the first three rows (row 0 when S < 3): one outlier among them
//     cannot become the shift, which keeps |s1|, and with it the rounding error of the
//     mean, small under heavy-tailed noise.
//   - s1 is summed in blocks of 8 rows (a fresh partial per block, then one add), so the
//     long chain of roundings happens on small partial sums.
//   - per-column results enter fp64 accumulators; warp shuffles, a block tree and a
//     fixed-order second stage do the rest in fp64.
//
// A producer warp streams tiles into shared memory with bulk asynchronous copies (one copy
// per row, completion counted on an mbarrier); eight consumer warps read them back.  Memory
// latency is covered by the stages in flight rather than by registers, and the consumers
// issue no global loads or address arithmetic.  A work item is (tile, row chunk):
// kThreads * CPT columns of up to max_rows_per_stage rows.  Row chunks let any S through: the
// per-column sums carry over from one chunk of rows to the next and close after the last.
// ---------------------------------------------------------------------------------------
//
// FUSED (lagged estimate only): eta_t is known when the kernel starts, so the same pass also
// reads w and v, applies the update of Eq. 2 and writes them back; the mean gradient lives in
// registers only and the update kernel is not launched: P * (S * b_g + 16) bytes per iteration
// instead of P * (S * b_g + 24), one launch instead of two.
template <int DT, int CPT, bool FUSED>
__global__ void __launch_bounds__(kStagedThreads, kReduceBlocksPerSM) k_reduce(const __grid_constant__ ReduceArgs a)
{
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) u64 full_bar[kStages], empty_bar[kStages];
    __shared__ StageInfo stage_info[kStages];           // what the producer put into each stage
    // Per-thread sums of the tiles in flight, handed from the consumer warps to the producer warp
    // (which has the time to add them up in fp64; a shuffle tree in every consumer warp and tile,
    // and any fence or atomic per tile, measured 5-40 % slower).  A warp releases a stage before it
    // hands over the tile's sums, so its fastest sibling can be handing over the tile kStages
    // further on while it still owes its own: kStages + 1 slots.
    __shared__ float2 tile_part[kSlots][kThreads];
    __shared__ __align__(8) u64 part_bar[kSlots];       // completes when all consumer warps have handed over
    __shared__ double sa[kStagedWarps], sb[kStagedWarps];
    __shared__ bool is_last;
    __shared__ int abort_flag;
    __shared__ float eta_shared;

    constexpr int E = Elem<DT>::kBytes;
    constexpr int kTile = kThreads * CPT;  // columns per tile
    constexpr int kRowBytes = kTile * E;   // one row of a stage
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool producer = warp == kStagedWarps - 1;
    const int S = a.S, T = a.T;
    const int rps = S < max_rows_per_stage(DT) ? S : max_rows_per_stage(DT);  // rows per stage
    const int n_chunks = (S + rps - 1) / rps;
    const unsigned stage_bytes = (unsigned)rps * kRowBytes;
    const long long n_tiles = a.n_tiles;
    const unsigned nst = a.stages;  // stages in use: 2 with the static assignment, 3 with runs (measured)
    // When the next kernel may start.  One-pass mode: the successor is another reduce launch, whose
    // producer warps want to start early, so every thread triggers it as soon as its own wait has
    // returned.  Two-kernel mode: the successor is the update kernel, and a block of it that lands
    // on an SM where a reduce block still runs keeps that SM's split of shared memory and L1
    // (hardly any L1) for its whole life, which costs the update kernel up to a quarter of its
    // speed; so the dependents are released only when every other SM is already idle: by the
    // exit of the last block, or, where a last block stays behind to add up the pairs, by that
    // block before it does so.
    auto trigger_early = [] {
        if constexpr (FUSED) griddep_launch();
    };

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], kWarps);
        }
        for (int i = 0; i < kSlots; ++i) mbar_init(&part_bar[i], kWarps);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    double accD = 0.0, accN = 0.0;  // scalar-path tiles, and the staged tiles of the static assignment
    unsigned item = 0;  // running count of staged work items, identical in every thread
    bool timed_out = false;

    if (producer) {
        u64 policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        const u64 keep_pairs = l2_keep_policy();  // the run pairs are read once more, right after this kernel
        int last_use[kStages];
#pragma unroll
        for (int i = 0; i < kStages; ++i) last_use[i] = -1;
        // How tiles reach the blocks.  Small jobs (a.run_tiles == 0): statically, tile t belongs to
        // block t mod grid.  Large jobs: in runs of a.run_tiles consecutive tiles; a block's first
        // run is run blockIdx.x and every further one comes from a counter, so the blocks of the
        // grid always work on one narrow, advancing window of the gradient matrix whatever the
        // relative speed of the SMs (this keeps DRAM pages hot: 3-6 % on the largest jobs against
        // the static assignment; nothing on small ones, where the extra pairs to add up at the end
        // would cost more).  The counter is written by the previous reduce launch, which may still
        // be running when this block starts (see the ordering rule), so it is touched only after
        // the wait: a block that streams rows early requests its first tile, waits, and only then
        // asks for further runs.  Run indices are fetched two runs ahead, the descriptor one tile
        // ahead and this lane's row pointer (row = lane when S <= 32) one tile ahead, so no table
        // miss delays a copy.
        const long long G = gridDim.x;
        const long long R = a.run_tiles;       // 0: static assignment
        // The last runs of a launch are single tiles: what the blocks differ by when the counter runs
        // dry is then one tile, not one run (10-20 us of idle SMs at the end of a large job).
        const long long A = a.long_runs, AR = A * R;
        const long long n_runs = R > 0 ? A + (n_tiles - AR) : 0;
        auto run_first = [&](long long r) -> long long { return r < A ? r * R : AR + (r - A); };
        auto run_of = [&](long long tile) -> long long { return tile < AR ? tile / R : A + (tile - AR); };
        auto run_ends = [&](long long tile) -> bool { return tile >= AR || (tile + 1) % R == 0; };
        // Before its wait this warp only reads tables that the host wrote (descriptors, row pointers:
        // their uploads are full stream dependencies), so the first tile's addresses are ready when
        // the wait returns.  The rows are the caller's data: unless the caller has vouched that
        // they were complete before this launch could start, the kernel before this one in the
        // stream may be the one that writes them and may have triggered its dependents early, so
        // the wait comes before the first copy.
        bool late_fetch = R > 0;
        bool waited = false;  // griddepcontrol.wait has returned in this warp
        // The next two runs of this block, known to all lanes, and a third that lane 0 has asked the
        // counter for but not yet passed on: the answer is only looked at when the next run is
        // taken, a whole run later, so the warp never waits for the atomic's round trip.
        long long rq0 = n_runs, rq1 = n_runs, rq2_lane0 = n_runs;
        auto ask_run = [&]() {   // lane 0 asks the counter; nobody waits
            if (lane == 0) rq2_lane0 = G + (long long)atomicAdd(a.tile_counter, 1ull);
        };
        auto take_asked = [&]() -> long long { return __shfl_sync(0xffffffffu, rq2_lane0, 0); };
        // the tile after `tile` in this block's sequence (n_tiles when there is none); consumes a
        // prefetched run index at the end of a run
        auto next_tile = [&](long long tile) -> long long {
            if (tile >= n_tiles) return n_tiles;
            if (R == 0) return tile + G < n_tiles ? tile + G : n_tiles;
            if (!run_ends(tile)) return tile + 1;
            const long long r = rq0;
            rq0 = rq1;
            if (late_fetch || r >= n_runs) {
                rq1 = n_runs;
            } else {
                rq1 = take_asked();
                if (rq1 < n_runs) ask_run();
            }
            return r < n_runs ? run_first(r) : n_tiles;
        };
        TileDesc d0, d1 = {}, d2 = {};
        const char *rowptr = nullptr, *rowptr_n = nullptr;
        float *pw = nullptr, *pv = nullptr, *pw_n = nullptr, *pv_n = nullptr;  // fused mode, lane 0 only
        unsigned pfl = 0, pfl_n = 0;
        long long t = R > 0 ? ((long long)blockIdx.x < n_runs ? run_first(blockIdx.x) : n_tiles)
                            : ((long long)blockIdx.x < n_tiles ? (long long)blockIdx.x : n_tiles);
        long long t1 = next_tile(t);
        if (t < n_tiles) d1 = a.tiles[t];
        if (t1 < n_tiles) d2 = a.tiles[t1];
        if (t < n_tiles && lane < S) rowptr_n = (const char *)a.gptr[(size_t)lane * T + d1.tensor];
        if constexpr (FUSED) {
            if (t < n_tiles && lane == 0) {
                pw_n = (float *)a.wv[d1.tensor];
                pv_n = (float *)a.wv[T + d1.tensor];
                pfl_n = a.wflags[d1.tensor];
            }
        }
        // Sums of the staged tiles, in a fixed order whatever block and warp order they are formed
        // in.  The consumers leave the 256 per-thread pairs of a tile in shared memory; lane l of
        // this warp adds threads l, l+32, ... of every tile of a run, in order, into its own fp64
        // pair; a shuffle tree adds the lanes at the end of the run and the result goes to
        // run_partials[run] with a plain store.  Whoever adds those pairs up (k_sum, or the block that
        // finishes last) does so in a fixed order, so nothing depends on which block processed which
        // run.  (Static assignment: none of this; the consumer threads keep their own fp64 pairs.)
        unsigned q = 0;                 // tiles this block has staged
        long long qt0 = 0, qt1 = 0, qt2 = 0, qt3 = 0;  // their indices, by slot (kSlots = 4)
        double runD = 0.0, runN = 0.0;  // this lane's share of the run being delivered
        auto deliver = [&](unsigned seq) -> bool {
            const int slot = seq % kSlots;
            if (!mbar_wait(&part_bar[slot], (seq / kSlots) & 1u, a.spin_limit)) return false;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float2 e = tile_part[slot][w * 32 + lane];
                runD += (double)e.x;
                runN += (double)e.y;
            }
            if (R > 0) {
                const long long tile = slot == 0 ? qt0 : (slot == 1 ? qt1 : (slot == 2 ? qt2 : qt3));
                if (run_ends(tile)) {
                    const double D = warp_sum(runD), N = warp_sum(runN);
                    if (lane == 0) store_pair_keep(&a.run_partials[run_of(tile)], D, N, keep_pairs);
                    runD = runN = 0.0;
                }
            }
            return true;
        };
        while (t < n_tiles && !timed_out) {
            {
                const int slot = q % kSlots;
                if (slot == 0) qt0 = t; else if (slot == 1) qt1 = t; else if (slot == 2) qt2 = t; else qt3 = t;
            }
            ++q;
            d0 = d1;
            rowptr = rowptr_n;
            pw = pw_n; pv = pv_n; pfl = pfl_n;
            d1 = d2;
            const long long t2 = next_tile(t1);
            if (t2 < n_tiles) d2 = a.tiles[t2];
            if (t1 < n_tiles && d1.tensor != d0.tensor) {
                if (lane < S) rowptr_n = (const char *)a.gptr[(size_t)lane * T + d1.tensor];
                if constexpr (FUSED) {
                    if (lane == 0) {
                        pw_n = (float *)a.wv[d1.tensor];
                        pv_n = (float *)a.wv[T + d1.tensor];
                        pfl_n = a.wflags[d1.tensor];
                    }
                }
            }
            const int k = d0.tensor;
            const long long c0 = d0.first;
            const int tc = d0.len;
            for (int ch = 0; ch < n_chunks; ++ch, ++item) {
                const int st = item % nst;
                const unsigned use = item / nst;
                if (!waited && (!a.early_rows || item >= nst)) {
                    // the rows may not be read yet (default), or a stage is about to be reused, which
                    // needs the consumers, and they start only after the previous kernel: from here on
                    // this warp's bounded waits must not count that kernel's run time
                    griddep_wait();
                    trigger_early();
                    waited = true;
                }
                if (!mbar_wait(&empty_bar[st], (use & 1u) ^ 1u, a.spin_limit)) { timed_out = true; break; }
                const int r0 = ch * rps;
                const int rows = S - r0 < rps ? S - r0 : rps;
                if (lane == 0) {
                    StageInfo &si = stage_info[st];
                    si.first = d0.first;
                    si.goff = d0.goff;
                    si.len = tc;
                    if constexpr (FUSED) { si.w = pw; si.v = pv; si.wflag = pfl; }
                    mbar_expect_tx(&full_bar[st], (unsigned)rows * tc * E);  // releases the writes above
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < kStages; ++i)
                    if (i == st) last_use[i] = (int)use;
                unsigned char *dst = stage_mem + (size_t)st * stage_bytes;
                if (r0 + rps <= 32) {
                    // rows r0 .. r0+rows-1 live in lanes r0 .. : each lane copies its own row
                    const int r = lane - r0;
                    if (r >= 0 && r < rows)
                        bulk_load(dst + (size_t)r * kRowBytes, rowptr + (size_t)c0 * E, (unsigned)tc * E, &full_bar[st], policy);
                } else {
                    for (int r = lane; r < rows; r += 32) {
                        const char *src = (const char *)a.gptr[(size_t)(r0 + r) * T + k] + (size_t)c0 * E;
                        bulk_load(dst + (size_t)r * kRowBytes, src, (unsigned)tc * E, &full_bar[st], policy);
                    }
                }
            }
            // With this tile staged, the sums of the tile kStages before it leave: its slot is the one
            // the next tile's sums will use.
            if (R > 0 && !timed_out && q >= (unsigned)kSlots && !deliver(q - kSlots)) timed_out = true;
            long long t_next = t1, t1_next = t2;
            if (late_fetch) {  // the first tile's rows are on their way: now the counter may be used
                late_fetch = false;
                if (!waited) {
                    griddep_wait();
                    trigger_early();
                    waited = true;
                }
                ask_run();
                rq0 = take_asked();
                ask_run();
                rq1 = take_asked();
                ask_run();
                // the sequence was built without the counter: rebuild what follows this tile
                t_next = next_tile(t);
                t1_next = next_tile(t_next);
                if (t_next < n_tiles) {
                    d1 = a.tiles[t_next];
                    if (lane < S) rowptr_n = (const char *)a.gptr[(size_t)lane * T + d1.tensor];
                    if constexpr (FUSED) {
                        if (lane == 0) {
                            pw_n = (float *)a.wv[d1.tensor];
                            pv_n = (float *)a.wv[T + d1.tensor];
                            pfl_n = a.wflags[d1.tensor];
                        }
                    }
                }
                if (t1_next < n_tiles) d2 = a.tiles[t1_next];
            }
            t = t_next;
            t1 = t1_next;
        }
        if (!timed_out) {  // an end mark in the next stage tells the consumers that no tile follows
            const int st = item % nst;
            const unsigned use = item / nst;
            if (mbar_wait(&empty_bar[st], (use & 1u) ^ 1u, a.spin_limit)) {
                if (lane == 0) {
                    stage_info[st].len = -1;
                    mbar_arrive(&full_bar[st]);
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < kStages; ++i)
                    if (i == st) last_use[i] = (int)use;  // the end mark is this stage's last phase
            } else {
                timed_out = true;
            }
        }
        // the sums of the last tiles; with the static assignment, the block's one pair
        for (unsigned seq = q >= (unsigned)kSlots ? q - kSlots + 1 : 0u; R > 0 && seq < q && !timed_out; ++seq)
            if (!deliver(seq)) timed_out = true;
        // The answer to the last question put to the counter must have arrived before this block
        // leaves: the counter is reset once all blocks have (by k_sum, or by the block that takes the
        // last exit ticket), and an increment still on its way would land after the reset.  (Looking
        // at the value makes the warp wait.)
        if (R > 0 && take_asked() < 0) timed_out = true;
        if (timed_out) atomicExch(&abort_flag, 1);
        // Every copy this warp has issued must have landed before the block may leave (its shared
        // memory is handed to the next block): wait for the last phase of each stage, with the long
        // fixed bound whatever the handshake limit is.  In a normal run the consumers are waiting
        // for the same phases, so this costs nothing.
#pragma unroll
        for (int i = 0; i < kStages; ++i)
            if (last_use[i] >= 0 && !mbar_wait(&full_bar[i], (unsigned)last_use[i] & 1u, kSpinLimit))
                atomicExch(&abort_flag, 1);
        if (!waited) {  // a block without a staged tile: every thread passes its wait and triggers
            griddep_wait();
            trigger_early();
        }
    } else {
        // Nothing may be written before the previous kernel in the stream (the update that still
        // reads the old mean gradient and the old eta) has finished.  Only then is the next
        // kernel allowed to start (see the ordering rule above).
        griddep_wait();
        trigger_early();
        // The first half of the scalar part needs only the state this iteration starts from: one
        // thread of block 0 works it out here, while the block's first rows are still on their way,
        // and leaves it for whoever runs the second half: the last block of this launch, or every
        // block of the next kernel (which must not read the state itself: its block 0 overwrites
        // the state while other blocks may still be starting).
        float eta = 0.f;
        if constexpr (FUSED) {
            // one-pass form: eta_t of the lagged estimate is the product of two of its values
            if (tid == 0) {
                const ScalarPrep prep = scalar_prepare(raw_state(a.st), a.sc, a.sched);
                eta_shared = (float)(prep.r_prior * prep.lr);
                if (blockIdx.x == 0) *a.prepared = prep;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");  // consumers only
            eta = eta_shared;
        } else {
            if (blockIdx.x == 0 && tid == 0) *a.prepared = scalar_prepare(raw_state(a.st), a.sc, a.sched);
        }
        constexpr int NP = CPT / 2;
        const u64 keep = l2_keep_policy();
        f2 c[NP], s1[NP], s2[NP], p1[NP];  // per-column state as packed pairs
        const unsigned lane_base = smem_u32(stage_mem) + (unsigned)tid * CPT * E;
        unsigned tseq = 0;  // tiles this block has consumed
        while (!timed_out) {
            // the tile that the producer has put into the next stage, or its end mark
            StageInfo si;
            {
                const int st = item % nst;
                if (!mbar_wait(&full_bar[st], (item / nst) & 1u, a.spin_limit)) { timed_out = true; break; }
                si = stage_info[st];
            }
            if (si.len < 0) break;
            const int tc = si.len;
            const bool active = tid * CPT < tc;
            float wr[CPT], vr[CPT];  // fused mode: this thread's parameters and momentum, requested
            float *wt = nullptr, *vt = nullptr;  // before the rows are consumed so they arrive meanwhile
            bool vec_wv = false;
            if constexpr (FUSED) {
                wt = si.w + si.first + tid * CPT;
                vt = si.v + si.first + tid * CPT;
                vec_wv = (si.wflag & 1u) != 0;
                if (active) {
                    if (vec_wv) {
                        Cols<ADASCALE_F32, CPT>::load((const char *)wt, wr);
                        Cols<ADASCALE_F32, CPT>::load((const char *)vt, vr);
                    } else {
#pragma unroll
                        for (int j = 0; j < CPT; ++j) { wr[j] = wt[j]; vr[j] = vt[j]; }
                    }
                }
            }
            bool tile_complete = false;
            float dacc = 0.f, nacc = 0.f;
            for (int ch = 0; ch < n_chunks; ++ch, ++item) {
                const int st = item % nst;
                const unsigned use = item / nst;
                if (!mbar_wait(&full_bar[st], use & 1u, a.spin_limit)) { timed_out = true; break; }
                const int r0 = ch * rps;
                const int rows = S - r0 < rps ? S - r0 : rps;
                unsigned addr = lane_base + (unsigned)st * stage_bytes;
                if (active) {
                    int r = 0;
                    if (ch == 0) {
#pragma unroll
                        for (int j = 0; j < NP; ++j) s1[j] = s2[j] = 0ull;  // +0.0f, +0.0f
                        if (S >= 3) {  // shift = median of the first three rows
                            typename Held<DT>::type x0[NP], x1[NP], x2[NP];
                            if constexpr (DT == ADASCALE_BF16) {  // taken on the raw words, widened once
                                load_words<CPT, 0>(addr, x0);
                                load_words<CPT, kRowBytes>(addr, x1);
                                load_words<CPT, 2 * kRowBytes>(addr, x2);
#pragma unroll
                                for (int j = 0; j < NP; ++j) c[j] = widen2(median3_bf16x2(x0[j], x1[j], x2[j]));
                            } else {
                                PairLoad<DT, CPT>::template load<0>(addr, x0);
                                PairLoad<DT, CPT>::template load<kRowBytes>(addr, x1);
                                PairLoad<DT, CPT>::template load<2 * kRowBytes>(addr, x2);
#pragma unroll
                                for (int j = 0; j < NP; ++j) {
                                    float a0, a1, b0, b1, e0, e1;
                                    unpack2(x0[j], a0, a1);
                                    unpack2(x1[j], b0, b1);
                                    unpack2(x2[j], e0, e1);
                                    const float m0 = fmaxf(fminf(a0, b0), fminf(fmaxf(a0, b0), e0));
                                    const float m1 = fmaxf(fminf(a1, b1), fminf(fmaxf(a1, b1), e1));
                                    c[j] = pack2(m0, m1);
                                }
                            }
                            if (rows >= 8) {  // first block of 8: the three rows are still in registers
#pragma unroll
                                for (int j = 0; j < NP; ++j) p1[j] = 0ull;
                                consume_held<DT, CPT>(x0, c, p1, s2);
                                consume_held<DT, CPT>(x1, c, p1, s2);
                                consume_held<DT, CPT>(x2, c, p1, s2);
                                consume_row<DT, CPT, 3 * kRowBytes>(addr, c, p1, s2);
                                consume_row<DT, CPT, 4 * kRowBytes>(addr, c, p1, s2);
                                consume_row<DT, CPT, 5 * kRowBytes>(addr, c, p1, s2);
                                consume_row<DT, CPT, 6 * kRowBytes>(addr, c, p1, s2);
                                consume_row<DT, CPT, 7 * kRowBytes>(addr, c, p1, s2);
#pragma unroll
                                for (int j = 0; j < NP; ++j) s1[j] = add2(s1[j], p1[j]);
                                addr += 8 * kRowBytes;
                                r = 8;
                            }
                        } else {
                            PairLoad<DT, CPT>::template load<0>(addr, c);
                        }
                    }
                    for (; r + 8 <= rows; r += 8) {  // s1 in blocks of 8 rows
#pragma unroll
                        for (int j = 0; j < NP; ++j) p1[j] = 0ull;
                        consume_row<DT, CPT, 0 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 1 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 2 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 3 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 4 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 5 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 6 * kRowBytes>(addr, c, p1, s2);
                        consume_row<DT, CPT, 7 * kRowBytes>(addr, c, p1, s2);
#pragma unroll
                        for (int j = 0; j < NP; ++j) s1[j] = add2(s1[j], p1[j]);
                        addr += 8 * kRowBytes;
                    }
                    if (r < rows) {
#pragma unroll
                        for (int j = 0; j < NP; ++j) p1[j] = 0ull;
                        for (; r < rows; ++r) {
                            consume_row<DT, CPT, 0>(addr, c, p1, s2);
                            addr += kRowBytes;
                        }
#pragma unroll
                        for (int j = 0; j < NP; ++j) s1[j] = add2(s1[j], p1[j]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);  // this warp is done with the stage
                if (ch == n_chunks - 1) tile_complete = true;
                if (active && ch == n_chunks - 1) {
                    float m[CPT];
#pragma unroll
                    for (int j = 0; j < NP; ++j) {
                        float cc[2], ss1[2], ss2[2];
                        unpack2(c[j], cc[0], cc[1]);
                        unpack2(s1[j], ss1[0], ss1[1]);
                        unpack2(s2[j], ss2[0], ss2[1]);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            // quotient s1/S: reciprocal multiply plus one residual correction (1/S is not
                            // exact unless S is a power of two, and a biased 1/S would bias every column alike)
                            float q = ss1[h] * a.invS;
                            const float res = fmaf(-q, a.fS, ss1[h]);
                            q = fmaf(res, a.invS, q);
                            m[2 * j + h] = cc[h] + q;
                            dacc += fmaf(-q, ss1[h], ss2[h]);
                            nacc = fmaf(m[2 * j + h], m[2 * j + h], nacc);
                        }
                    }
                    if constexpr (FUSED) {
#pragma unroll
                        for (int j = 0; j < CPT; ++j) {
                            vr[j] = fmaf(a.rho, vr[j], fmaf(a.lambda, wr[j], m[j]));
                            wr[j] = fmaf(-eta, vr[j], wr[j]);
                        }
                        if (vec_wv) {
                            store_cols<CPT>(vt, vr);
                            store_cols<CPT>(wt, wr);
                        } else {
#pragma unroll
                            for (int j = 0; j < CPT; ++j) { vt[j] = vr[j]; wt[j] = wr[j]; }
                        }
                    } else {
                        store_cols_keep<CPT>(a.gbar + si.goff + tid * CPT, m, keep);
                    }
                }
            }
            if (!tile_complete) break;  // a wait gave up inside the tile
            if (a.run_tiles > 0) {
                // runs from the counter: the thread's two sums over its columns of the tile go to
                // the producer warp, which adds them up per run
                const int slot = tseq % kSlots;
                tile_part[slot][tid] = make_float2(dacc, nacc);
                __syncwarp();
                if (lane == 0) mbar_arrive(&part_bar[slot]);
            } else {
                // static assignment: the block's tiles are fixed, so the thread keeps its own fp64 pair
                // for the whole launch and the block adds its threads up once, below
                accD += (double)dacc;
                accN += (double)nacc;
            }
            ++tseq;
        }
        // ragged tails (< 8 elements) and tensors that are not 16-byte aligned: plain loads
        for (long long t = blockIdx.x; t < a.n_stiles; t += gridDim.x) {
            const TileDesc d = a.stiles[t];
            float *gb = a.gbar + d.goff;
            for (int e = tid; e < d.len; e += kThreads) {
                float dd, nn;
                if constexpr (FUSED) {
                    float m;
                    column_scalar<DT>(a.gptr, T, d.tensor, ((size_t)d.first + e) * E, S, a.fS, &m, dd, nn);
                    float *w = (float *)a.wv[d.tensor] + d.first + e;
                    float *v = (float *)a.wv[T + d.tensor] + d.first + e;
                    const float vn = fmaf(a.rho, *v, fmaf(a.lambda, *w, m));
                    *v = vn;
                    *w = fmaf(-eta, vn, *w);
                } else {
                    column_scalar<DT>(a.gptr, T, d.tensor, ((size_t)d.first + e) * E, S, a.fS, gb + e, dd, nn);
                }
                accD += (double)dd;
                accN += (double)nn;
            }
        }
        if (timed_out) atomicExch(&abort_flag, 1);
    }

    // statically assigned tiles (all scalar-path tiles, the staged ones of small jobs): one pair per block
    block_sum2<kStagedWarps>(accD, accN, sa, sb);
    if (tid == 0) {
        if (abort_flag) atomicOr(&a.st->fault, ADASCALE_STATUS_WAIT_TIMEOUT);
        a.partials[blockIdx.x] = make_double2(accD, accN);
    }
    // Scalar part left to the next kernel (small and mid-size jobs, static assignment): every block
    // of that kernel adds up the pairs itself, so nothing here waits for the last block; the
    // dependents are released when the last block exits, which is when every other SM is idle.
    if (a.leave_open) return;
    if (tid == 0) {
        __threadfence();
        const unsigned tk = atomicAdd(a.ticket, 1u);
        is_last = (tk == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    if constexpr (!FUSED) griddep_launch();

    // Last stage, fixed order: thread j adds the pairs j, j+288, ... of the runs in index order,
    // sixteen loads in flight at a time, then the per-block pairs likewise, then the block tree.
    // (The run pairs were stored with the evict-last priority, so they are still in L2.  Bringing
    // them in through the idle stages with bulk copies was measured too: 14 against 11 us for
    // 30 K pairs, one SM cannot keep more bytes in flight that way than with these loads.)
    __threadfence();
    double d = 0.0, n = 0.0;
    const long long n_pairs = a.run_tiles > 0 ? a.long_runs + (n_tiles - a.long_runs * a.run_tiles) : 0;
    {
        constexpr int U = 16;
        long long i = tid;
        for (; i + (U - 1) * (long long)kStagedThreads < n_pairs; i += U * (long long)kStagedThreads) {
            double2 p[U];
#pragma unroll
            for (int u = 0; u < U; ++u) p[u] = __ldcg(&a.run_partials[i + u * (long long)kStagedThreads]);
#pragma unroll
            for (int u = 0; u < U; ++u) { d += p[u].x; n += p[u].y; }
        }
        for (; i < n_pairs; i += kStagedThreads) {
            const double2 p = __ldcg(&a.run_partials[i]);
            d += p.x;
            n += p.y;
        }
    }
    block_sum2<kStagedWarps>(d, n, sa, sb);  // the run pairs (zero with the static assignment)
    // The per-block pairs in the order in which sum_pairs adds them (the producer warp adds zeros), so
    // that this form and the one that leaves the scalar part to the update kernel agree bit for bit.
    double db = 0.0, nb = 0.0;
    if (tid < kThreads) {
        for (int i = tid; i < (int)gridDim.x; i += kThreads) {
            const double2 p = __ldcg(&a.partials[i]);
            db += p.x;
            nb += p.y;
        }
    }
    block_sum2<kStagedWarps>(db, nb, sa, sb);
    d = db + d;
    n = nb + n;
    if (tid == 0) {
        if (a.sums_out) {  // sharded use: the caller adds the shards' sums, k_scalar continues
            a.sums_out[0] = d;
            a.sums_out[1] = n;
        } else {
            bool skip;
            scalar_finish(a.st, load_prepared(a.prepared), a.sc, d, n, __ldcg(&a.st->fault), skip);
        }
        *a.ticket = 0u;
        *a.tile_counter = 0ull;
    }
}


// Scalar part as a kernel of one thread: used when the two sums are completed outside the
// reduce kernel (each GPU of a column-sharded job reduces its own columns, the sums are added
// across GPUs, then every GPU runs the identical scalar step on the identical numbers).
__global__ void k_scalar(const __grid_constant__ ScalarArgs a)
{
    griddep_wait();
    griddep_launch();
    if (threadIdx.x == 0 && blockIdx.x == 0) scalar_step(a.st, a.sc, a.sched, a.sums[0], a.sums[1]);
}

// ---------------------------------------------------------------------------------------
// Update kernel (Eq. 2 with momentum).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void update4(float4 &ww, float4 &vv, const float4 &gg, float rho, float lambda, float eta)
{
    vv.x = fmaf(rho, vv.x, fmaf(lambda, ww.x, gg.x));
    vv.y = fmaf(rho, vv.y, fmaf(lambda, ww.y, gg.y));
    vv.z = fmaf(rho, vv.z, fmaf(lambda, ww.z, gg.z));
    vv.w = fmaf(rho, vv.w, fmaf(lambda, ww.w, gg.w));
    ww.x = fmaf(-eta, vv.x, ww.x);
    ww.y = fmaf(-eta, vv.y, ww.y);
    ww.z = fmaf(-eta, vv.z, ww.z);
    ww.w = fmaf(-eta, vv.w, ww.w);
}

__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Adds the pairs p[0..n) in a fixed order with a block of kThreads threads; the sums are valid in thread 0.
__device__ __forceinline__ void sum_pairs(const double2 *p, int n, double &d, double &nn, double *sa, double *sb)
{
    d = 0.0;
    nn = 0.0;
    for (int i = threadIdx.x; i < n; i += kThreads) {
        const double2 e = __ldcg(&p[i]);
        d += e.x;
        nn += e.y;
    }
    block_sum2<kWarps>(d, nn, sa, sb);
}

// A block's first tile is tile blockIdx.x; every further tile comes from a counter, so at any
// moment the blocks of the grid work on one narrow, advancing window of the three arrays
// whatever the relative speed of the SMs (a narrow window keeps DRAM pages and the read/write
// batches of the memory controller efficient), and no SM idles at the end.  The counter value is fetched one tile ahead and the
// descriptor of the next tile while the current one is processed.  A tile is kUpdateTile =
// 1024 * C elements: C 128-bit accesses per array and thread, all requested before the first
// is used.  The counter needs no reset: every block asks once more than it gets tiles (its last
// answer is the one that tells it to stop), so a launch asks exactly n_tiles times, and the
// counter is an atomicInc that wraps to zero after n_tiles increments.
//
// DEFER: the reduce launch before this one stopped at one pair of sums per block, and every block
// here completes the iteration's scalar part by itself: the same pairs, added in the same order,
// give every block the same eta_t, and block 0 records the new state.  The first half of the
// scalar part (schedule, averaging weight: most of its time) was done by the reduce launch while
// it waited for its first rows, and is read from where it left it (not from the state, which
// block 0 may already have overwritten when a block starts late).  The second half runs while
// the block's first tile is on its way from memory into L2.  What the reduce kernel would spend after its last block has
// finished - an exit ticket, one block adding up the pairs, one thread doing the scalar part,
// about 5 us on the critical path of every iteration - is gone.
template <bool DEFER>
__global__ void __launch_bounds__(kThreads, kUpdateBlocksPerSM) k_update(const __grid_constant__ UpdateArgs a)
{
    constexpr int C = kUpdateVecs;
    __shared__ long long s_next[2];
    __shared__ double sa[kWarps], sb[kWarps];
    __shared__ float s_eta;
    __shared__ int s_skip;
    __shared__ ScalarPrep s_prep;
    const int tid = threadIdx.x, T = a.T;
    const long long n_tiles = a.n_tiles, G = gridDim.x;
    long long c = blockIdx.x;
    TileDesc d = {}, dn = {};
    // Before the wait: only tables that the host wrote (descriptor, the tensor's pointers and flags).
    float *wq = nullptr, *vq = nullptr;
    unsigned fl = 0;
    if (c < n_tiles) {
        d = a.tiles[c];
        wq = (float *)a.wv[d.tensor];
        vq = (float *)a.wv[T + d.tensor];
        fl = a.wflags[d.tensor];
    }
    griddep_wait();
    griddep_launch();
    float eta = 0.f;
    if constexpr (!DEFER) {
        // a skipped iteration (non-finite sums, or a bounded wait that gave up) changes nothing; every
        // block sees the same state, so either all of them ask the counter or none does
        const bool skip = (a.st->status & ADASCALE_STATUS_NONFINITE) || a.st->fault;
        if (skip) return;
        eta = (float)a.st->eta;
    }
    // the counter belongs to the update launches; it is touched only after the wait, so that even
    // two update launches in a row cannot meet on it
    const unsigned wrap = (unsigned)(n_tiles - 1);
    unsigned asked = 0;  // thread 0: the counter's answer, looked at as late as possible
    if (tid == 0) asked = atomicInc(a.next_tile, wrap);
    if constexpr (DEFER) {
        // The block's first tile is asked into L2 (no registers held), and the scalar part is
        // completed while it travels.
        unsigned fault = 0;
        if (tid == 0) {  // requested before the pairs, used after them
            s_prep = load_prepared(a.prepared);
            fault = __ldcg(&a.st->fault);
        }
        if (c < n_tiles) {
            const int e = tid * 4 * C;  // this thread's first element of the tile
            if (e < d.len) {
                prefetch_l2(a.gbar + d.goff + e);
                prefetch_l2(wq + d.first + e);
                prefetch_l2(vq + d.first + e);
            }
        }
        double D, N;
        sum_pairs(a.partials, a.n_partials, D, N, sa, sb);
        if (tid == 0) {
            bool skip;
            s_eta = (float)scalar_finish(blockIdx.x == 0 ? a.st : nullptr, s_prep, a.sc, D, N, fault, skip);
            s_skip = skip ? 1 : 0;
            s_next[0] = G + (long long)asked;
        }
        __syncthreads();
        eta = s_eta;
        if (s_skip) {
            // nothing is applied, but the counter must still see every request of this launch
            if (tid == 0)
                for (long long x = s_next[0]; x < n_tiles;) x = G + (long long)atomicInc(a.next_tile, wrap);
            return;
        }
    } else {
        if (tid == 0) s_next[0] = G + (long long)asked;
        __syncthreads();
    }
    int buf = 0;
    while (c < n_tiles) {
        const long long nc = s_next[buf];
        if (tid == 0 && nc < n_tiles) s_next[buf ^ 1] = G + (long long)atomicInc(a.next_tile, wrap);
        if (nc < n_tiles) dn = a.tiles[nc];
        float *w = wq + d.first;
        float *v = vq + d.first;
        const float *g = a.gbar + d.goff;
        const bool vec = (fl & 1u) != 0;
        const int len = d.len;
        if (vec && len == 1024 * C) {
            float4 gg[C], ww[C], vv[C];
#pragma unroll
            for (int j = 0; j < C; ++j) {
                gg[j] = ((const float4 *)g)[tid + j * kThreads];
                ww[j] = ((const float4 *)w)[tid + j * kThreads];
                vv[j] = ((const float4 *)v)[tid + j * kThreads];
            }
#pragma unroll
            for (int j = 0; j < C; ++j) {
                update4(ww[j], vv[j], gg[j], a.rho, a.lambda, eta);
                ((float4 *)v)[tid + j * kThreads] = vv[j];
                ((float4 *)w)[tid + j * kThreads] = ww[j];
            }
        } else {
            int done = 0;
            if (vec) {
                const int nv = len >> 2;
                for (int i = tid; i < nv; i += kThreads) {
                    const float4 g4 = ((const float4 *)g)[i];
                    float4 w4 = ((const float4 *)w)[i];
                    float4 v4 = ((const float4 *)v)[i];
                    update4(w4, v4, g4, a.rho, a.lambda, eta);
                    ((float4 *)v)[i] = v4;
                    ((float4 *)w)[i] = w4;
                }
                done = nv << 2;
            }
            for (int e = done + tid; e < len; e += kThreads) {
                const float vn = fmaf(a.rho, v[e], fmaf(a.lambda, w[e], g[e]));
                v[e] = vn;
                w[e] = fmaf(-eta, vn, w[e]);
            }
        }
        if (nc < n_tiles && dn.tensor != d.tensor) {  // the next tile's tensor, requested before the barrier
            wq = (float *)a.wv[dn.tensor];
            vq = (float *)a.wv[T + dn.tensor];
            fl = a.wflags[dn.tensor];
        }
        __syncthreads();
        c = nc;
        buf ^= 1;
        d = dn;
    }
}

// Large jobs leave tens of thousands of run pairs.  One block (the reduce kernel's last) needs
// 10-17 us to add them up, with every other SM idle; a few dozen blocks need one round of loads.
// Block b adds the pairs of slice b, thread j the pairs j, j + 256, ... of the slice, then the
// block tree: a fixed order, whatever ran where.  The pairs of this launch join the per-block
// pairs of the reduce launch, and the update kernel (or k_finish) adds up both.
__global__ void __launch_bounds__(kThreads) k_sum(const __grid_constant__ SumArgs a)
{
    __shared__ double sa[kWarps], sb[kWarps];
    griddep_wait();
    griddep_launch();
    const long long per = (a.n_pairs + gridDim.x - 1) / gridDim.x;
    const long long first = (long long)blockIdx.x * per;
    const long long end = first + per < a.n_pairs ? first + per : a.n_pairs;
    double d = 0.0, n = 0.0;
    for (long long i = first + threadIdx.x; i < end; i += kThreads) {
        const double2 e = __ldcg(&a.run_partials[i]);
        d += e.x;
        n += e.y;
    }
    block_sum2<kWarps>(d, n, sa, sb);
    if (threadIdx.x == 0) {
        a.out[blockIdx.x] = make_double2(d, n);
        if (blockIdx.x == 0) *a.tile_counter = 0ull;
    }
}

// The scalar part on its own, one block: when a reduce launch left it open and no update follows
// (the caller asks for the statistics, or reduces again).  Same sums in the same order, same two
// halves as in the update kernel, so the state is the same whichever of the two completes it.
__global__ void __launch_bounds__(kThreads) k_finish(const __grid_constant__ FinishArgs a)
{
    __shared__ double sa[kWarps], sb[kWarps];
    griddep_wait();
    griddep_launch();
    double D, N;
    sum_pairs(a.partials, a.n_partials, D, N, sa, sb);
    if (threadIdx.x == 0) {
        const ScalarPrep prep = load_prepared(a.prepared);
        bool skip;
        scalar_finish(a.st, prep, a.sc, D, N, __ldcg(&a.st->fault), skip);
    }
}

// ---- bandwidth probes -------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_probe_read(const uint4 *a, long long n, unsigned *sink)
{
    unsigned acc = 0;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kThreads) {
        const uint4 q = ld_stream16(a + i);
        acc ^= q.x ^ q.y ^ q.z ^ q.w;
    }
    if (acc == 0x9e3779b9u) *sink = acc;  // keeps the loads alive, practically never taken
}
__global__ void __launch_bounds__(kThreads) k_probe_copy(const uint4 *a, uint4 *b, long long n)
{
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kThreads)
        b[i] = ld_stream16(a + i);
}
__global__ void __launch_bounds__(kThreads) k_probe_rmw(float4 *a, const float4 *b, long long n)
{
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kThreads) {
        float4 x = a[i];
        const float4 y = b[i];
        x.x += y.x;
        x.y += y.y;
        x.z += y.z;
        x.w += y.w;
        a[i] = x;
    }
}

}  // namespace
