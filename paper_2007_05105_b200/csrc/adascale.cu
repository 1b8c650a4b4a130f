// AdaScale SGD gain-ratio step for sm_100a: kernels and the C-ABI host glue.
//
// Two kernels make up one iteration (paper: Sec. 3.2, App. B.3, Eq. 2-3):
//   reduce  - streams the S x P gradient matrix once through shared memory (bulk asynchronous
//             copies completed on mbarriers, a producer warp and eight consumer warps), writes
//             the mean gradient and one pair (sum of squared deviations, squared norm of the
//             mean) per block; the block that finishes last adds the pairs in index order and
//             runs the scalar part (estimates, clamps, moving averages, r_t, eta_t, tau_{t+1}).
//   update  - v <- rho v + (gbar + lambda w), w <- w - eta_t v, reading eta_t from the device.
// Three trivial streaming kernels calibrate the bandwidth ceiling.
// The path is bound by HBM bandwidth; there is no contraction, hence no tensor-core work.
//
// Work distribution: every tensor is cut into tiles; tile t belongs to block t mod gridDim.
// All blocks therefore advance through each gradient row as one front, which keeps DRAM
// pages hot, and the split does not depend on how the hardware schedules blocks, so the
// fixed-order sums are reproducible from run to run.
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
constexpr int kStages = 3;                // shared-memory stages per block
constexpr int kMaxRowsPerStage = 16;      // rows of one stage; larger S goes through in row chunks
constexpr int kStageBytes = 32 * 1024;    // upper bound of one stage
constexpr int kReduceBlocksPerSM = 2;
constexpr int kUpdateBlocksPerSM = 8;
constexpr int kScalarTile = 2048;         // elements per tile on the unaligned / ragged-tail path
constexpr int kUpdateTile = 1024;         // elements per tile of the update kernel: one 128-bit access per thread
constexpr int kGbarAlign = 64;            // every tensor's mean gradient starts on a 256-byte boundary
constexpr int kRing = 4;                  // pinned staging slots for pointer-table uploads
constexpr int kMaxS = 4096;
constexpr unsigned kSpinLimit = 1u << 22; // bounded waits: give up, flag, leave

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
// where the tile's mean gradient lives in the library's workspace.  Tile t belongs to block
// t mod gridDim.  The descriptors hold no pointers, so they change only with the tiling.
struct __align__(16) TileDesc {
    long long first;
    long long goff;
    int tensor;
    int len;
    int pad[2];
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
    double2 *partials;
    unsigned *ticket;
    DevState *st;
    int S, T;
    float invS, fS;
    ScalarCfg sc;
    Sched sched;
};

struct UpdateArgs {
    const u64 *wv;            // [2 * T]: parameters then momentum
    const unsigned *wflags;   // [T] bit0: both pointers 16-byte aligned
    const TileDesc *tiles;    // tiles of kUpdateTile elements
    long long n_tiles;
    const float *gbar;
    const DevState *st;
    int T;
    float rho, lambda;
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
        int passed = 0;
        for (int i = 0; i < s.n; ++i) passed += (t > s.w[i]) ? 1 : 0;
        return s.eta0 * pow(s.decay, (double)passed);
    }
    return s.eta0;
}

__device__ __forceinline__ double ema(double prev, double sample, double theta, long long n)
{
    // plain mean of the first samples until the exponential weight takes over (App. B.3)
    double warm = 1.0 - 1.0 / (double)n;
    double th = theta < warm ? theta : warm;
    return th * prev + (1.0 - th) * sample;
}

// Scalar part of the iteration: one thread, fp64, no host involvement.
__device__ void scalar_step(DevState *st, const ScalarCfg &c, const Sched &sched, double D, double N)
{
    st->D = D;
    st->N = N;
    if (!isfinite(D) || !isfinite(N)) {  // skip the iteration, leave every average and tau alone
        st->status = ADASCALE_STATUS_NONFINITE;
        st->skipped += 1;
        st->eta = 0.0;
        return;
    }
    st->status = 0;
    const double S = (double)c.S;
    const double tau = st->tau;
    const double t_arg = (c.flags & ADASCALE_FLAG_CONT_TAU) ? tau : floor(tau);
    double r;
    if (c.S == 1) {  // App. A.2: unit gain at scale one
        st->sigma2_raw = 0.0;
        st->mu2_raw = N;
        r = 1.0;
    } else {
        double a, b, r_prior;
        const bool ratio = (c.flags & ADASCALE_FLAG_RATIO) != 0;
        if (ratio) {
            // Sec. 3.4: (1/S) sum_i ||g_i||^2 = D/S + N  and ||gbar||^2
            a = D / S + N;
            b = N;
            st->sigma2_raw = a;
            st->mu2_raw = b;
            r_prior = st->n > 0 ? (st->avg_a + c.eps) / (st->avg_b + c.eps) : 1.0;
        } else {
            // App. B.3: sigma^2 = D/(S-1) equals 1/(S-1) sum||g_i||^2 - S/(S-1)||gbar||^2
            double sigma2 = D / (S - 1.0);
            double mu2 = N - sigma2 / S;
            st->sigma2_raw = sigma2;
            st->mu2_raw = mu2;
            a = sigma2 > c.eps ? sigma2 : c.eps;
            b = mu2 > 0.0 ? mu2 : 0.0;
            r_prior = st->n > 0 ? (st->avg_a + st->avg_b) / (st->avg_a / S + st->avg_b) : 1.0;
        }
        const long long n = st->n + 1;
        const double na = ema(st->avg_a, a, c.theta, n);
        const double nb = ema(st->avg_b, b, c.theta, n);
        st->n = n;
        st->avg_a = na;
        st->avg_b = nb;
        if (c.flags & ADASCALE_FLAG_LAGGED)
            r = r_prior;
        else
            r = ratio ? (na + c.eps) / (nb + c.eps) : (na + nb) / (na / S + nb);  // Eq. 3
    }
    const double lr = lr_eval(sched, t_arg);
    st->r = r;
    st->lr = lr;
    st->eta = r * lr;     // Sec. 3.2
    st->tau = tau + r;
    st->t += 1;
}

// Persistent grid: every block walks its own segments and keeps two fp64 accumulators per
// thread for the whole launch, so there is one block reduction and one partial pair per block.
// Lagged estimate (App. B.3: r_t from the averages of prior iterations only, r_0 = 1): the
// learning rate of the coming iteration is known before its gradients are read.  Same
// expressions as in scalar_step, so both give the identical value.
__device__ double lagged_eta(const DevState *st, const ScalarCfg &c, const Sched &sched)
{
    const double S = (double)c.S;
    double r = 1.0;
    if (c.S > 1 && st->n > 0)
        r = (c.flags & ADASCALE_FLAG_RATIO) ? (st->avg_a + c.eps) / (st->avg_b + c.eps)
                                            : (st->avg_a + st->avg_b) / (st->avg_a / S + st->avg_b);
    const double tau = st->tau;
    const double t_arg = (c.flags & ADASCALE_FLAG_CONT_TAU) ? tau : floor(tau);
    return r * lr_eval(sched, t_arg);
}

// Programmatic dependent launch: a kernel lets its successor in the stream be scheduled
// early, and waits for its predecessor (completion and visibility of its writes) only where
// it first depends on it.  Both are no-ops for a launch without the attribute.
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
// Returns false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(u64 *bar, unsigned parity)
{
    const unsigned addr = smem_u32(bar);
    for (unsigned spin = 0; spin < kSpinLimit; ++spin) {
        unsigned done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done)
                     : "r"(addr), "r"(parity)
                     : "memory");
        if (done) return true;
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

// One staged row into the running sums: d = x - c, p1 += d, s2 += d * d.
template <int DT, int CPT, int OFF>
__device__ __forceinline__ void consume_row(unsigned addr, const f2 *c, f2 *p1, f2 *s2)
{
    f2 x[CPT / 2];
    PairLoad<DT, CPT>::template load<OFF>(addr, x);
#pragma unroll
    for (int j = 0; j < CPT / 2; ++j) {
        const f2 d = sub2(x[j], c[j]);
        p1[j] = add2(p1[j], d);
        s2[j] = fma2(d, d, s2[j]);
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
// kThreads * CPT columns of up to kMaxRowsPerStage rows.  Row chunks let any S through: the
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
    const int rps = S < kMaxRowsPerStage ? S : kMaxRowsPerStage;  // rows per stage
    const int n_chunks = (S + rps - 1) / rps;
    const unsigned stage_bytes = (unsigned)rps * kRowBytes;
    const long long n_tiles = a.n_tiles;

    griddep_launch();
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], kWarps);
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    double accD = 0.0, accN = 0.0;
    unsigned item = 0;  // running count of staged work items, identical in every thread
    bool timed_out = false;

    if (producer) {
        u64 policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        int last_use[kStages];
#pragma unroll
        for (int i = 0; i < kStages; ++i) last_use[i] = -1;
        // Round-robin tiles make every block visit most tensors, so table misses must stay off
        // the copy queue: the descriptor is fetched two tiles ahead and this lane's row pointer
        // (row = lane when S <= 32) one tile ahead.
        const long long G = gridDim.x;
        TileDesc d0, d1 = {}, d2 = {};
        const char *rowptr = nullptr, *rowptr_n = nullptr;
        if ((long long)blockIdx.x < n_tiles) d1 = a.tiles[blockIdx.x];
        if ((long long)blockIdx.x + G < n_tiles) d2 = a.tiles[blockIdx.x + G];
        if ((long long)blockIdx.x < n_tiles && lane < S) rowptr_n = (const char *)a.gptr[(size_t)lane * T + d1.tensor];
        for (long long t = blockIdx.x; t < n_tiles && !timed_out; t += G) {
            d0 = d1;
            rowptr = rowptr_n;
            d1 = d2;
            if (t + 2 * G < n_tiles) d2 = a.tiles[t + 2 * G];
            if (t + G < n_tiles && d1.tensor != d0.tensor && lane < S)
                rowptr_n = (const char *)a.gptr[(size_t)lane * T + d1.tensor];
            const int k = d0.tensor;
            const long long c0 = d0.first;
            const int tc = d0.len;
            for (int ch = 0; ch < n_chunks; ++ch, ++item) {
                const int st = item % kStages;
                const unsigned use = item / kStages;
                if (!mbar_wait(&empty_bar[st], (use & 1u) ^ 1u)) { timed_out = true; break; }
                const int r0 = ch * rps;
                const int rows = S - r0 < rps ? S - r0 : rps;
                if (lane == 0) mbar_expect_tx(&full_bar[st], (unsigned)rows * tc * E);
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
        }
        if (timed_out) atomicExch(&abort_flag, 1);
        if (timed_out || *(volatile int *)&abort_flag) {
            // leaving early: copies already issued must land before this block's shared memory is reused
#pragma unroll
            for (int i = 0; i < kStages; ++i)
                if (last_use[i] >= 0) mbar_wait(&full_bar[i], (unsigned)last_use[i] & 1u);
        }
    } else {
        // The producer above may already stream gradient rows while the previous kernel in the
        // stream (the update that still reads the old mean gradient) drains; nothing may be
        // written before it has finished.
        griddep_wait();
        float eta = 0.f;
        if constexpr (FUSED) {
            if (tid == 0) eta_shared = (float)lagged_eta(a.st, a.sc, a.sched);
            asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");  // consumers only
            eta = eta_shared;
        }
        constexpr int NP = CPT / 2;
        const u64 keep = l2_keep_policy();
        f2 c[NP], s1[NP], s2[NP], p1[NP];  // per-column state as packed pairs
        const long long G = gridDim.x;
        TileDesc d0, d1 = {};  // descriptor one tile ahead, as above
        if ((long long)blockIdx.x < n_tiles) d1 = a.tiles[blockIdx.x];
        // fused mode: the tile's parameter and momentum pointers, fetched one tile ahead as well
        float *wp = nullptr, *vp = nullptr, *wp_n = nullptr, *vp_n = nullptr;
        unsigned fl = 0, fl_n = 0;
        if constexpr (FUSED) {
            if ((long long)blockIdx.x < n_tiles) {
                wp_n = (float *)a.wv[d1.tensor];
                vp_n = (float *)a.wv[T + d1.tensor];
                fl_n = a.wflags[d1.tensor];
            }
        }
        const unsigned lane_base = smem_u32(stage_mem) + (unsigned)tid * CPT * E;
        for (long long t = blockIdx.x; t < n_tiles && !timed_out; t += G) {
            d0 = d1;
            if (t + G < n_tiles) d1 = a.tiles[t + G];
            const int tc = d0.len;
            const bool active = tid * CPT < tc;
            float wr[CPT], vr[CPT];  // fused mode: this thread's parameters and momentum, requested
            float *wt = nullptr, *vt = nullptr;  // before the rows are consumed so they arrive meanwhile
            bool vec_wv = false;
            if constexpr (FUSED) {
                wp = wp_n; vp = vp_n; fl = fl_n;
                if (t + G < n_tiles && d1.tensor != d0.tensor) {
                    wp_n = (float *)a.wv[d1.tensor];
                    vp_n = (float *)a.wv[T + d1.tensor];
                    fl_n = a.wflags[d1.tensor];
                }
                wt = wp + d0.first + tid * CPT;
                vt = vp + d0.first + tid * CPT;
                vec_wv = (fl & 1u) != 0;
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
            for (int ch = 0; ch < n_chunks; ++ch, ++item) {
                const int st = item % kStages;
                const unsigned use = item / kStages;
                if (!mbar_wait(&full_bar[st], use & 1u)) { timed_out = true; break; }
                const int r0 = ch * rps;
                const int rows = S - r0 < rps ? S - r0 : rps;
                unsigned addr = lane_base + (unsigned)st * stage_bytes;
                if (active) {
                    if (ch == 0) {
                        if (S >= 3) {  // shift = median of the first three rows
                            f2 x0[NP], x1[NP], x2[NP];
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
                        } else {
                            PairLoad<DT, CPT>::template load<0>(addr, c);
                        }
#pragma unroll
                        for (int j = 0; j < NP; ++j) s1[j] = s2[j] = 0ull;  // +0.0f, +0.0f
                    }
                    int r = 0;
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
                if (active && ch == n_chunks - 1) {
                    float m[CPT];
                    float dacc = 0.f, nacc = 0.f;
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
                        store_cols_keep<CPT>(a.gbar + d0.goff + tid * CPT, m, keep);
                    }
                    accD += (double)dacc;
                    accN += (double)nacc;
                }
            }
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

    block_sum2<kStagedWarps>(accD, accN, sa, sb);
    if (tid == 0) {
        if (abort_flag) atomicOr(&a.st->fault, ADASCALE_STATUS_WAIT_TIMEOUT);
        a.partials[blockIdx.x] = make_double2(accD, accN);
        __threadfence();
        const unsigned tk = atomicAdd(a.ticket, 1u);
        is_last = (tk == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;

    // Second stage, fixed order: thread j adds partials j, j+288, ... in index order, then the
    // same block tree.  The result depends on the tiling only, not on how blocks were scheduled.
    __threadfence();
    double d = 0.0, n = 0.0;
    for (int i = tid; i < (int)gridDim.x; i += kStagedThreads) {
        const double2 p = __ldcg(&a.partials[i]);
        d += p.x;
        n += p.y;
    }
    block_sum2<kStagedWarps>(d, n, sa, sb);
    if (tid == 0) {
        scalar_step(a.st, a.sc, a.sched, d, n);
        *a.ticket = 0u;
    }
}

// ---------------------------------------------------------------------------------------
// Update kernel (Eq. 2 with momentum): tiles of kUpdateTile elements, one 128-bit access per
// array and thread, tiles dealt round-robin like in the reduce kernel.
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

__global__ void __launch_bounds__(kThreads, kUpdateBlocksPerSM) k_update(const __grid_constant__ UpdateArgs a)
{
    griddep_launch();
    const int tid = threadIdx.x, T = a.T;
    const long long n_tiles = a.n_tiles, G = gridDim.x;
    // descriptor two tiles ahead, the tensor's pointers one tile ahead (see the reduce kernel)
    TileDesc d0, d1 = {}, d2 = {};
    float *wp = nullptr, *vp = nullptr, *wp_n = nullptr, *vp_n = nullptr;
    unsigned fl = 0, fl_n = 0;
    if ((long long)blockIdx.x < n_tiles) {
        d1 = a.tiles[blockIdx.x];
        wp_n = (float *)a.wv[d1.tensor];
        vp_n = (float *)a.wv[T + d1.tensor];
        fl_n = a.wflags[d1.tensor];
    }
    if ((long long)blockIdx.x + G < n_tiles) d2 = a.tiles[blockIdx.x + G];
    // w and v of the first tile do not depend on the reduce kernel: they are requested while it
    // still drains; eta_t and the mean gradient are read only after the wait
    float4 w_first = make_float4(0.f, 0.f, 0.f, 0.f), v_first = w_first;
    const bool first_fast = (long long)blockIdx.x < n_tiles && (fl_n & 1u) && d1.len == kUpdateTile;
    if (first_fast) {
        w_first = ((const float4 *)(wp_n + d1.first))[tid];
        v_first = ((const float4 *)(vp_n + d1.first))[tid];
    }
    griddep_wait();
    if (a.st->status & ADASCALE_STATUS_NONFINITE) return;
    const float eta = (float)a.st->eta;
    for (long long t = blockIdx.x; t < n_tiles; t += G) {
        d0 = d1; wp = wp_n; vp = vp_n; fl = fl_n;
        d1 = d2;
        if (t + 2 * G < n_tiles) d2 = a.tiles[t + 2 * G];
        if (t + G < n_tiles && d1.tensor != d0.tensor) {
            wp_n = (float *)a.wv[d1.tensor];
            vp_n = (float *)a.wv[T + d1.tensor];
            fl_n = a.wflags[d1.tensor];
        }
        const long long first = d0.first;
        const int len = d0.len;
        float *w = wp + first, *v = vp + first;
        const float *g = a.gbar + d0.goff;
        const bool vec = (fl & 1u) != 0;
        if (vec && len == kUpdateTile) {
            const bool have = first_fast && t == (long long)blockIdx.x;
            const float4 gg = ((const float4 *)g)[tid];
            float4 ww = have ? w_first : ((const float4 *)w)[tid];
            float4 vv = have ? v_first : ((const float4 *)v)[tid];
            update4(ww, vv, gg, a.rho, a.lambda, eta);
            ((float4 *)v)[tid] = vv;
            ((float4 *)w)[tid] = ww;
        } else {
            int done = 0;
            if (vec) {
                const int nv = len >> 2;
                if (tid < nv) {
                    const float4 gg = ((const float4 *)g)[tid];
                    float4 ww = ((const float4 *)w)[tid];
                    float4 vv = ((const float4 *)v)[tid];
                    update4(ww, vv, gg, a.rho, a.lambda, eta);
                    ((float4 *)v)[tid] = vv;
                    ((float4 *)w)[tid] = ww;
                }
                done = nv << 2;
            }
            for (int e = done + tid; e < len; e += kThreads) {
                const float vn = fmaf(a.rho, v[e], fmaf(a.lambda, w[e], g[e]));
                v[e] = vn;
                w[e] = fmaf(-eta, vn, w[e]);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Allocation-free variant of the reduce kernel for one tensor: the same shifted sums, the
// same fp64 partials and fixed-order second stage, but rows are read with plain 128-bit loads
// and everything the kernel needs besides its inputs and outputs (row-pointer table, ticket,
// per-block partials) lives in one file-scope device array instead of memory from cudaMalloc.
// ---------------------------------------------------------------------------------------
constexpr int kStaticMaxRows = ADASCALE_STATIC_MAX_ROWS;
constexpr int kStaticMaxBlocks = 1024;
constexpr size_t kStaticPtrBytes = 256;     // 32 row pointers
constexpr size_t kStaticTicketOff = 256;    // one counter, padded to 256 bytes
constexpr size_t kStaticPartialOff = 512;   // kStaticMaxBlocks pairs of doubles
constexpr size_t kStaticScratchBytes = kStaticPartialOff + kStaticMaxBlocks * sizeof(double2);

// Shared by every call on this device and kept until the process exits (about 17 KB).
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticArgs {
    unsigned char *scratch;  // device address of g_static_scratch, resolved on the host
    float *gbar;
    double *sums;            // [0] = sum_i ||g_i - gbar||^2, [1] = ||gbar||^2
    long long n;
    int S;
    float invS, fS;
};

template <int DT>
__global__ void __launch_bounds__(kThreads) k_grad_stats_static(const __grid_constant__ StaticArgs a)
{
    __shared__ double sa[kWarps], sb[kWarps];
    __shared__ bool is_last;
    constexpr int E = Elem<DT>::kBytes;
    constexpr int V = 8;  // columns per thread and step
    const u64 *rows = reinterpret_cast<const u64 *>(a.scratch);
    unsigned *ticket = reinterpret_cast<unsigned *>(a.scratch + kStaticTicketOff);
    double2 *partials = reinterpret_cast<double2 *>(a.scratch + kStaticPartialOff);
    const int tid = threadIdx.x, S = a.S;
    const long long nv = a.n / V;
    double accD = 0.0, accN = 0.0;

    for (long long v = (long long)blockIdx.x * kThreads + tid; v < nv; v += (long long)gridDim.x * kThreads) {
        const size_t boff = (size_t)v * V * E;
        float c[V], s1[V], s2[V], p1[V], x[V];
        if (S >= 3) {  // shift = median of the first three rows
            float x1[V], x2[V];
            Cols<DT, V>::load((const char *)rows[0] + boff, x);
            Cols<DT, V>::load((const char *)rows[1] + boff, x1);
            Cols<DT, V>::load((const char *)rows[2] + boff, x2);
#pragma unroll
            for (int j = 0; j < V; ++j) {
                const float lo = fminf(x[j], x1[j]), hi = fmaxf(x[j], x1[j]);
                c[j] = fmaxf(lo, fminf(hi, x2[j]));
            }
        } else {
            Cols<DT, V>::load((const char *)rows[0] + boff, c);
        }
#pragma unroll
        for (int j = 0; j < V; ++j) s1[j] = s2[j] = 0.f;
        for (int r = 0; r < S; r += 8) {  // s1 in blocks of 8 rows
#pragma unroll
            for (int j = 0; j < V; ++j) p1[j] = 0.f;
            for (int rr = r; rr < S && rr < r + 8; ++rr) {
                Cols<DT, V>::load((const char *)rows[rr] + boff, x);
                accumulate_row<V>(x, c, p1, s2);
            }
#pragma unroll
            for (int j = 0; j < V; ++j) s1[j] += p1[j];
        }
        float m[V];
        float dacc = 0.f, nacc = 0.f;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            float q = s1[j] * a.invS;
            const float res = fmaf(-q, a.fS, s1[j]);
            q = fmaf(res, a.invS, q);
            m[j] = c[j] + q;
            dacc += fmaf(-q, s1[j], s2[j]);
            nacc = fmaf(m[j], m[j], nacc);
        }
        store_cols<V>(a.gbar + v * V, m);
        accD += (double)dacc;
        accN += (double)nacc;
    }
    if (blockIdx.x == 0) {  // ragged tail, fewer than 8 elements
        for (long long e = nv * V + tid; e < a.n; e += kThreads) {
            float d, nn;
            column_scalar<DT>(rows, 1, 0, (size_t)e * E, S, a.fS, a.gbar + e, d, nn);
            accD += (double)d;
            accN += (double)nn;
        }
    }

    block_sum2<kWarps>(accD, accN, sa, sb);
    if (tid == 0) {
        partials[blockIdx.x] = make_double2(accD, accN);
        __threadfence();
        const unsigned tk = atomicAdd(ticket, 1u);
        is_last = (tk == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double d = 0.0, n = 0.0;
    for (int i = tid; i < (int)gridDim.x; i += kThreads) {
        const double2 p = __ldcg(&partials[i]);
        d += p.x;
        n += p.y;
    }
    block_sum2<kWarps>(d, n, sa, sb);
    if (tid == 0) {
        a.sums[0] = d;
        a.sums[1] = n;
        *ticket = 0u;
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

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------

// A table of pointers (plus per-tensor flags and tile prefixes) mirrored on the host and
// uploaded only when it changes, through a small ring of pinned slots so that an upload
// still in flight is never overwritten.
struct PtrTable {
    std::vector<u64> mirror;   // last uploaded contents, 8-byte words
    u64 *dev = nullptr;
    u64 *pinned[kRing] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t ev[kRing] = {nullptr, nullptr, nullptr, nullptr};
    bool used[kRing] = {false, false, false, false};
    int next = 0;
    size_t words = 0;
    bool valid = false;
};

struct StateBlob {  // ADASCALE_STATE_BYTES
    unsigned magic, version;
    int S;
    unsigned flags;
    double tau, avg_a, avg_b;
    long long n, t, skipped;
    double r, eta, lr;
    double pad[5];
};
static_assert(sizeof(StateBlob) == ADASCALE_STATE_BYTES, "state blob size");
constexpr unsigned kMagic = 0x41645363u;  // "AdSc"

}  // namespace

struct adascale_ctx {
    int device = 0, sms = 0;
    int S = 1, max_S = 1, T = 0, dtype = 0;
    double rho = 0, lambda = 0, eps = 1e-6, theta_cfg = -1;
    unsigned flags = 0;
    std::vector<long long> numel;
    std::vector<long long> goff;
    long long P = 0, gbar_elems = 0;
    TileDesc *d_rtiles = nullptr;   // reduce kernel: staged tiles, then scalar tiles
    TileDesc *d_utiles = nullptr;   // update kernel
    long long rtiles_cap = 0, n_utiles = 0;
    std::vector<const void *> last_grads;      // the caller's pointer arrays as of the last upload
    std::vector<void *> last_w, last_v;
    std::vector<unsigned char> tiled_aligned;  // alignment flags and tile width the device descriptors were built for
    int tiled_cpt = 0;
    float *d_gbar = nullptr;
    double2 *d_partials = nullptr;
    unsigned *d_ticket = nullptr;
    DevState *d_state = nullptr;
    PtrTable tg, tw;
    long long n_tiles = 0, n_stiles = 0;  // of the descriptors on the device
    DevState *h_snap = nullptr;  // pinned
    cudaEvent_t ev_snap = nullptr;
    bool snap_inflight = false;
    DevState latest{};
    cudaStream_t last_stream = nullptr;
    bool reduced = false;
    long long launches = 0;
    void *d_stage = nullptr;     // host-gradient staging (adascale_step_host)
    std::vector<const void *> stage_ptrs;
    std::string err;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

adascale_status cuda_fail(adascale_ctx *c, cudaError_t e, const char *what)
{
    if (c) {
        c->err = what;
        c->err += ": ";
        c->err += cudaGetErrorString(e);
    }
    cudaGetLastError();  // a non-sticky error must not leak into the caller's next CUDA call
    return ADASCALE_ERR_CUDA;
}

#define CU(call)                                                    \
    do {                                                            \
        cudaError_t e_ = (call);                                    \
        if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call);    \
    } while (0)

double resolve_theta(const adascale_ctx *c)
{
    if (c->theta_cfg >= 0.0) return c->theta_cfg;
    const double th = 1.0 - (double)c->S / 1000.0;  // Sec. 3.4: theta = max{1 - S/1000, 0}
    return th > 0.0 ? th : 0.0;
}

// ---- tiling of the reduce kernel ---------------------------------------------------------

int rows_per_stage(int S) { return S < kMaxRowsPerStage ? S : kMaxRowsPerStage; }

long long staged_tiles(const long long *numel, const unsigned char *aligned, int T, int tile_cols)
{
    long long n = 0;
    for (int k = 0; k < T; ++k)
        if (!aligned || aligned[k]) n += ((numel[k] & ~7LL) + tile_cols - 1) / tile_cols;
    return n;
}

// Columns per consumer thread.  A thread reads 8, 16 or 32 bytes of each row; the widest
// access that keeps one stage (rows x 256 threads x bytes) within kStageBytes is used, and
// small jobs step down so that every block still gets a few tiles.
int choose_cpt(int dtype, int S, const long long *numel, const unsigned char *aligned, int T, int n_blocks)
{
    const int esz = dtype == ADASCALE_BF16 ? 2 : 4;
    int bpt = dtype == ADASCALE_BF16 ? 16 : 32;
    while (bpt > 8 && rows_per_stage(S) * kThreads * bpt > kStageBytes) bpt >>= 1;
    while (bpt > 8 && staged_tiles(numel, aligned, T, kThreads * bpt / esz) < 4LL * n_blocks) bpt >>= 1;
    return bpt / esz;
}

void build_prefixes(const long long *numel, const unsigned char *aligned, int T, int tile_cols,
                    long long *tprefix, long long *sprefix)
{
    long long nt = 0, ns = 0;
    for (int k = 0; k < T; ++k) {
        tprefix[k] = nt;
        sprefix[k] = ns;
        const long long n = numel[k];
        if (!aligned || aligned[k]) {
            nt += ((n & ~7LL) + tile_cols - 1) / tile_cols;
            ns += (n & 7LL) ? 1 : 0;
        } else {
            ns += (n + kScalarTile - 1) / kScalarTile;
        }
    }
    tprefix[T] = nt;
    sprefix[T] = ns;
}

// Descriptors of the reduce kernel's tiles: all staged tiles in tensor order, then all
// scalar-path tiles.
void build_reduce_tiles(const long long *numel, const long long *goff, const unsigned char *aligned, int T,
                        int tile_cols, std::vector<TileDesc> &out, long long &n_staged)
{
    out.clear();
    auto emit = [&](int k, long long first, long long len) {
        TileDesc d = {};
        d.first = first;
        d.goff = goff[k] + first;
        d.tensor = k;
        d.len = (int)len;
        out.push_back(d);
    };
    for (int k = 0; k < T; ++k) {
        if (aligned && !aligned[k]) continue;
        const long long cols = numel[k] & ~7LL;
        for (long long c0 = 0; c0 < cols; c0 += tile_cols) emit(k, c0, cols - c0 < tile_cols ? cols - c0 : tile_cols);
    }
    n_staged = (long long)out.size();
    for (int k = 0; k < T; ++k) {
        const long long n = numel[k];
        const long long start = (!aligned || aligned[k]) ? (n & ~7LL) : 0;
        for (long long f = start; f < n; f += kScalarTile) emit(k, f, n - f < kScalarTile ? n - f : kScalarTile);
    }
}

// ---- pointer tables ----------------------------------------------------------------------

adascale_status table_alloc(adascale_ctx *ctx, PtrTable &t, size_t words)
{
    t.words = words;
    t.mirror.assign(words, 0);
    CU(cudaMalloc(&t.dev, words * sizeof(u64)));
    for (int i = 0; i < kRing; ++i) {
        CU(cudaMallocHost(&t.pinned[i], words * sizeof(u64)));
        CU(cudaEventCreateWithFlags(&t.ev[i], cudaEventDisableTiming));
    }
    return ADASCALE_OK;
}

void table_free(PtrTable &t)
{
    if (t.dev) cudaFree(t.dev);
    for (int i = 0; i < kRing; ++i) {
        if (t.pinned[i]) cudaFreeHost(t.pinned[i]);
        if (t.ev[i]) cudaEventDestroy(t.ev[i]);
    }
    t = PtrTable();
}

// Uploads `fresh` (t.words entries) if it differs from what the device already holds.
adascale_status table_sync(adascale_ctx *ctx, PtrTable &t, const std::vector<u64> &fresh, cudaStream_t s)
{
    if (t.valid && std::memcmp(fresh.data(), t.mirror.data(), t.words * sizeof(u64)) == 0) return ADASCALE_OK;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU(cudaStreamIsCapturing(s, &cap));
    if (cap != cudaStreamCaptureStatusNone) {
        ctx->err = "pointer table changed inside a stream capture";
        return ADASCALE_ERR_STATE;
    }
    const int slot = t.next;
    t.next = (t.next + 1) % kRing;
    if (t.used[slot]) CU(cudaEventSynchronize(t.ev[slot]));
    std::memcpy(t.pinned[slot], fresh.data(), t.words * sizeof(u64));
    CU(cudaMemcpyAsync(t.dev, t.pinned[slot], t.words * sizeof(u64), cudaMemcpyHostToDevice, s));
    CU(cudaEventRecord(t.ev[slot], s));
    t.used[slot] = true;
    t.mirror = fresh;
    t.valid = true;
    return ADASCALE_OK;
}

// ---- launches ----------------------------------------------------------------------------

// Launch that may overlap its prologue with the tail of the previous kernel in the stream.
template <typename Args>
cudaError_t launch_overlapped(void (*kernel)(Args), int n_blocks, int threads, size_t smem, cudaStream_t s,
                              const Args &a)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_blocks);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

template <int DT, int CPT, bool FUSED>
cudaError_t launch_reduce_one(int n_blocks, const ReduceArgs &a, size_t smem, cudaStream_t s)
{
    static bool configured[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(k_reduce<DT, CPT, FUSED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kStages * kStageBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    return launch_overlapped(k_reduce<DT, CPT, FUSED>, n_blocks, kStagedThreads, smem, s, a);
}

template <bool FUSED>
cudaError_t launch_reduce_mode(int dtype, int cpt, int n_blocks, const ReduceArgs &a, size_t smem, cudaStream_t s)
{
    if (dtype == ADASCALE_BF16)
        return cpt == 4 ? launch_reduce_one<ADASCALE_BF16, 4, FUSED>(n_blocks, a, smem, s)
                        : launch_reduce_one<ADASCALE_BF16, 8, FUSED>(n_blocks, a, smem, s);
    switch (cpt) {
    case 2: return launch_reduce_one<ADASCALE_F32, 2, FUSED>(n_blocks, a, smem, s);
    case 4: return launch_reduce_one<ADASCALE_F32, 4, FUSED>(n_blocks, a, smem, s);
    default: return launch_reduce_one<ADASCALE_F32, 8, FUSED>(n_blocks, a, smem, s);
    }
}

cudaError_t launch_reduce(bool fused, int dtype, int cpt, int n_blocks, const ReduceArgs &a, size_t smem,
                          cudaStream_t s)
{
    return fused ? launch_reduce_mode<true>(dtype, cpt, n_blocks, a, smem, s)
                 : launch_reduce_mode<false>(dtype, cpt, n_blocks, a, smem, s);
}

bool valid_sched(const adascale_lr_schedule *s)
{
    if (!s) return false;
    if (s->kind < ADASCALE_LR_CONST || s->kind > ADASCALE_LR_STEP) return false;
    if (!(s->eta0 > 0.0)) return false;
    if (s->kind != ADASCALE_LR_CONST && !(s->decay > 0.0)) return false;
    if (s->kind == ADASCALE_LR_EXP && !(s->t_s1 > 0.0)) return false;
    if (s->kind == ADASCALE_LR_STEP && (s->n_milestones < 0 || s->n_milestones > ADASCALE_MAX_MILESTONES)) return false;
    return true;
}

// Layout of the reduce table in 8-byte words: [max_S * T row pointers]
adascale_status do_reduce(adascale_ctx *ctx, const void *const *grads, const adascale_lr_schedule *sched,
                          cudaStream_t s, bool fused)
{
    const int S = ctx->S, T = ctx->T;
    const size_t esz = ctx->dtype == ADASCALE_BF16 ? 2 : 4;
    const int max_blocks = ctx->sms * kReduceBlocksPerSM;
    const size_t n_ptrs = (size_t)S * T;
    // The usual case, the same pointers as in the previous call: nothing to validate, build or upload.
    const bool unchanged = ctx->tg.valid && ctx->tiled_cpt != 0 && ctx->last_grads.size() == n_ptrs &&
                           std::memcmp(ctx->last_grads.data(), grads, n_ptrs * sizeof(void *)) == 0;
    int cpt = ctx->tiled_cpt;
    if (!unchanged) {
    std::vector<u64> fresh(ctx->tg.words, 0);
    std::vector<unsigned char> aligned((size_t)T, 1);
    for (int k = 0; k < T; ++k) {
        for (int i = 0; i < S; ++i) {
            const u64 p = (u64)(uintptr_t)grads[(size_t)i * T + k];
            if (ctx->numel[k] > 0) {
                if (p == 0) return ADASCALE_ERR_INVALID_ARG;
                if (p % esz) return ADASCALE_ERR_ALIGNMENT;
                if (p % 16) aligned[k] = 0;
            }
            fresh[(size_t)i * T + k] = p;
        }
    }
    cpt = choose_cpt(ctx->dtype, S, ctx->numel.data(), aligned.data(), T, max_blocks);
    if (cpt != ctx->tiled_cpt || aligned != ctx->tiled_aligned) {
        // the tiling follows the tile width (a function of S) and the alignment of the pointers
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        CU(cudaStreamIsCapturing(s, &cap));
        if (cap != cudaStreamCaptureStatusNone) {
            ctx->err = "tiling changed inside a stream capture";
            return ADASCALE_ERR_STATE;
        }
        std::vector<TileDesc> tiles;
        long long n_staged = 0;
        build_reduce_tiles(ctx->numel.data(), ctx->goff.data(), aligned.data(), T, kThreads * cpt, tiles, n_staged);
        if ((long long)tiles.size() > ctx->rtiles_cap) return ADASCALE_ERR_TOO_LARGE;  // cannot happen: sized for the worst case
        if (!tiles.empty()) {
            // pageable source: the runtime stages it before the call returns
            CU(cudaMemcpyAsync(ctx->d_rtiles, tiles.data(), tiles.size() * sizeof(TileDesc), cudaMemcpyHostToDevice, s));
            CU(cudaStreamSynchronize(s));
        }
        ctx->n_tiles = n_staged;
        ctx->n_stiles = (long long)tiles.size() - n_staged;
        ctx->tiled_cpt = cpt;
        ctx->tiled_aligned = aligned;
    }
    adascale_status st = table_sync(ctx, ctx->tg, fresh, s);
    if (st != ADASCALE_OK) return st;
    ctx->last_grads.assign(grads, grads + n_ptrs);
    }
    const long long n_tiles = ctx->n_tiles, n_stiles = ctx->n_stiles;
    if (n_tiles + n_stiles == 0) return ADASCALE_OK;  // nothing but empty tensors

    ReduceArgs a;
    a.gptr = ctx->tg.dev;
    a.tiles = ctx->d_rtiles;
    a.stiles = ctx->d_rtiles + n_tiles;
    a.n_tiles = n_tiles;
    a.n_stiles = n_stiles;
    a.gbar = ctx->d_gbar;
    a.wv = ctx->tw.dev;  // read by the fused kernel only; sync_update_table has run before
    a.wflags = reinterpret_cast<const unsigned *>(ctx->tw.dev + (size_t)2 * T);
    a.rho = (float)ctx->rho;
    a.lambda = (float)ctx->lambda;
    a.partials = ctx->d_partials;
    a.ticket = ctx->d_ticket;
    a.st = ctx->d_state;
    a.S = S;
    a.T = T;
    a.fS = (float)S;
    a.invS = 1.0f / (float)S;
    a.sc.eps = ctx->eps;
    a.sc.theta = resolve_theta(ctx);
    a.sc.flags = ctx->flags;
    a.sc.S = S;
    a.sched.kind = sched->kind;
    a.sched.n = sched->kind == ADASCALE_LR_STEP ? sched->n_milestones : 0;
    a.sched.eta0 = sched->eta0;
    a.sched.decay = sched->decay;
    a.sched.t_s1 = sched->t_s1;
    for (int i = 0; i < ADASCALE_MAX_MILESTONES; ++i) a.sched.w[i] = sched->milestones[i];

    long long nb = n_tiles + n_stiles;
    if (nb > max_blocks) nb = max_blocks;
    const size_t smem = (size_t)kStages * rows_per_stage(S) * kThreads * cpt * esz;
    cudaError_t e = launch_reduce(fused, ctx->dtype, cpt, (int)nb, a, smem, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the reduce kernel");
    ctx->launches += 1;
    ctx->reduced = true;
    ctx->last_stream = s;
    return ADASCALE_OK;
}

// Layout of the update table in 8-byte words: [T parameters][T momentum][ceil(T/2) flags]
adascale_status sync_update_table(adascale_ctx *ctx, void *const *params, void *const *momentum, cudaStream_t s)
{
    const int T = ctx->T;
    if (ctx->tw.valid && ctx->last_w.size() == (size_t)T &&
        std::memcmp(ctx->last_w.data(), params, (size_t)T * sizeof(void *)) == 0 &&
        std::memcmp(ctx->last_v.data(), momentum, (size_t)T * sizeof(void *)) == 0)
        return ADASCALE_OK;  // same pointers as in the previous call
    std::vector<u64> fresh(ctx->tw.words, 0);
    unsigned *flags = reinterpret_cast<unsigned *>(fresh.data() + (size_t)2 * T);
    for (int k = 0; k < T; ++k) {
        const u64 pw = (u64)(uintptr_t)params[k], pv = (u64)(uintptr_t)momentum[k];
        if (ctx->numel[k] > 0) {
            if (!pw || !pv) return ADASCALE_ERR_INVALID_ARG;
            if ((pw % 4) || (pv % 4)) return ADASCALE_ERR_ALIGNMENT;
        }
        fresh[k] = pw;
        fresh[(size_t)T + k] = pv;
        flags[k] = ((pw % 16) == 0 && (pv % 16) == 0) ? 1u : 0u;
    }
    adascale_status st = table_sync(ctx, ctx->tw, fresh, s);
    if (st != ADASCALE_OK) return st;
    ctx->last_w.assign(params, params + T);
    ctx->last_v.assign(momentum, momentum + T);
    return ADASCALE_OK;
}

adascale_status do_update(adascale_ctx *ctx, void *const *params, void *const *momentum, cudaStream_t s)
{
    const int T = ctx->T;
    adascale_status st = sync_update_table(ctx, params, momentum, s);
    if (st != ADASCALE_OK) return st;
    const long long n_tiles = ctx->n_utiles;
    if (n_tiles == 0) return ADASCALE_OK;

    UpdateArgs a;
    a.wv = ctx->tw.dev;
    a.wflags = reinterpret_cast<const unsigned *>(ctx->tw.dev + (size_t)2 * T);
    a.tiles = ctx->d_utiles;
    a.n_tiles = n_tiles;
    a.gbar = ctx->d_gbar;
    a.st = ctx->d_state;
    a.T = T;
    a.rho = (float)ctx->rho;
    a.lambda = (float)ctx->lambda;
    long long nb = n_tiles;
    if (nb > (long long)ctx->sms * kUpdateBlocksPerSM) nb = (long long)ctx->sms * kUpdateBlocksPerSM;
    cudaError_t e = launch_overlapped(k_update, (int)nb, kThreads, 0, s, a);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the update kernel");
    ctx->launches += 1;
    ctx->last_stream = s;
    return ADASCALE_OK;
}

void fill_stats(const DevState &d, adascale_stats *o)
{
    std::memset(o, 0, sizeof *o);
    o->r = d.r;
    o->tau = d.tau;
    o->eta = d.eta;
    o->lr = d.lr;
    o->sigma2_raw = d.sigma2_raw;
    o->mu2_raw = d.mu2_raw;
    o->sigma2_avg = d.avg_a;
    o->mu2_avg = d.avg_b;
    o->gbar_sqnorm = d.N;
    o->dev_sqsum = d.D;
    o->t = d.t;
    o->n_samples = d.n;
    o->skipped = d.skipped;
    o->status_bits = d.status | d.fault;
}

}  // namespace

extern "C" {

const char *adascale_strerror(adascale_status s)
{
    switch (s) {
    case ADASCALE_OK: return "ok";
    case ADASCALE_ERR_INVALID_ARG: return "invalid argument";
    case ADASCALE_ERR_ALIGNMENT: return "pointer not aligned to its element size";
    case ADASCALE_ERR_CUDA: return "CUDA runtime error";
    case ADASCALE_ERR_STATE: return "call not allowed in the current state";
    case ADASCALE_ERR_TOO_LARGE: return "size beyond the documented maximum";
    }
    return "unknown status";
}

const char *adascale_last_error(const adascale_ctx *ctx) { return ctx ? ctx->err.c_str() : ""; }

int64_t adascale_launch_count(const adascale_ctx *ctx) { return ctx ? ctx->launches : 0; }

adascale_status adascale_tiling(const int64_t *numel, int32_t n_tensors, int32_t grad_dtype, int32_t S,
                                const uint8_t *aligned, int32_t n_blocks, int64_t *tprefix, int64_t *sprefix,
                                int32_t *tile_cols, int32_t *rows)
{
    if (!numel || n_tensors < 1 || S < 1 || n_blocks < 1 || !tprefix || !sprefix || !tile_cols || !rows)
        return ADASCALE_ERR_INVALID_ARG;
    if (grad_dtype != ADASCALE_F32 && grad_dtype != ADASCALE_BF16) return ADASCALE_ERR_INVALID_ARG;
    std::vector<long long> n(numel, numel + n_tensors);
    for (long long x : n)
        if (x < 0) return ADASCALE_ERR_INVALID_ARG;
    const int cpt = choose_cpt(grad_dtype, S, n.data(), aligned, n_tensors, n_blocks);
    std::vector<long long> tp((size_t)n_tensors + 1), sp((size_t)n_tensors + 1);
    build_prefixes(n.data(), aligned, n_tensors, kThreads * cpt, tp.data(), sp.data());
    for (int k = 0; k <= n_tensors; ++k) {
        tprefix[k] = tp[(size_t)k];
        sprefix[k] = sp[(size_t)k];
    }
    *tile_cols = kThreads * cpt;
    *rows = rows_per_stage(S);
    return ADASCALE_OK;
}

adascale_status adascale_init(const adascale_config *cfg, adascale_ctx **out)
{
    if (!cfg || !out) return ADASCALE_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->S < 1 || cfg->n_tensors < 1 || !cfg->numel) return ADASCALE_ERR_INVALID_ARG;
    const int max_S = cfg->max_S > 0 ? cfg->max_S : cfg->S;
    if (max_S < cfg->S) return ADASCALE_ERR_INVALID_ARG;
    if (max_S > kMaxS) return ADASCALE_ERR_TOO_LARGE;
    if (cfg->grad_dtype != ADASCALE_F32 && cfg->grad_dtype != ADASCALE_BF16) return ADASCALE_ERR_INVALID_ARG;
    if (!(cfg->theta < 1.0) || !(cfg->eps >= 0.0) || cfg->device < 0) return ADASCALE_ERR_INVALID_ARG;
    if (!std::isfinite(cfg->momentum) || !std::isfinite(cfg->weight_decay)) return ADASCALE_ERR_INVALID_ARG;
    if (cfg->flags & ~(ADASCALE_FLAG_LAGGED | ADASCALE_FLAG_CONT_TAU | ADASCALE_FLAG_RATIO | ADASCALE_FLAG_FUSED))
        return ADASCALE_ERR_INVALID_ARG;
    if ((cfg->flags & ADASCALE_FLAG_FUSED) && !(cfg->flags & ADASCALE_FLAG_LAGGED))
        return ADASCALE_ERR_INVALID_ARG;  // the one-pass form needs eta_t before the gradients are read
    for (int k = 0; k < cfg->n_tensors; ++k)
        if (cfg->numel[k] < 0) return ADASCALE_ERR_INVALID_ARG;

    adascale_ctx *ctx = new (std::nothrow) adascale_ctx();
    if (!ctx) return ADASCALE_ERR_INVALID_ARG;
    ctx->device = cfg->device;
    ctx->S = cfg->S;
    ctx->max_S = max_S;
    ctx->T = cfg->n_tensors;
    ctx->dtype = cfg->grad_dtype;
    ctx->rho = cfg->momentum;
    ctx->lambda = cfg->weight_decay;
    ctx->eps = cfg->eps;
    ctx->theta_cfg = cfg->theta;
    ctx->flags = cfg->flags;
    ctx->numel.assign(cfg->numel, cfg->numel + cfg->n_tensors);

    long long g = 0;
    std::vector<TileDesc> utiles;
    long long rcap = 0;  // worst case of the reduce tiling: everything unaligned, or the narrowest staged tile
    for (int k = 0; k < ctx->T; ++k) {
        const long long n = ctx->numel[k];
        ctx->goff.push_back(g);
        ctx->P += n;
        for (long long f = 0; f < n; f += kUpdateTile) {
            TileDesc d = {};
            d.first = f;
            d.goff = g + f;
            d.tensor = k;
            d.len = (int)(n - f < kUpdateTile ? n - f : kUpdateTile);
            utiles.push_back(d);
        }
        const long long narrow = kThreads * 8 / 4;  // 8 bytes per thread and row of fp32
        rcap += (n + narrow - 1) / narrow + 1;
        g += (n + kGbarAlign - 1) / kGbarAlign * kGbarAlign;
    }
    ctx->gbar_elems = g;
    ctx->n_utiles = (long long)utiles.size();
    ctx->rtiles_cap = rcap;

    DeviceGuard guard(ctx->device);
    auto body = [&]() -> adascale_status {
        if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
        CU(cudaDeviceGetAttribute(&ctx->sms, cudaDevAttrMultiProcessorCount, ctx->device));
        const size_t T = (size_t)ctx->T;
        CU(cudaMalloc(&ctx->d_rtiles, (size_t)(rcap > 0 ? rcap : 1) * sizeof(TileDesc)));
        CU(cudaMalloc(&ctx->d_utiles, (utiles.empty() ? 1 : utiles.size()) * sizeof(TileDesc)));
        if (!utiles.empty())
            CU(cudaMemcpy(ctx->d_utiles, utiles.data(), utiles.size() * sizeof(TileDesc), cudaMemcpyHostToDevice));
        const size_t gbar_alloc = (g > 0 && !(ctx->flags & ADASCALE_FLAG_FUSED)) ? (size_t)g : 1;
        CU(cudaMalloc(&ctx->d_gbar, gbar_alloc * sizeof(float)));
        CU(cudaMemset(ctx->d_gbar, 0, gbar_alloc * sizeof(float)));
        CU(cudaMalloc(&ctx->d_partials, (size_t)(ctx->sms * kReduceBlocksPerSM + 1) * sizeof(double2)));
        CU(cudaMalloc(&ctx->d_ticket, sizeof(unsigned)));
        CU(cudaMemset(ctx->d_ticket, 0, sizeof(unsigned)));
        CU(cudaMalloc(&ctx->d_state, sizeof(DevState)));
        CU(cudaMemset(ctx->d_state, 0, sizeof(DevState)));
        adascale_status s1 = table_alloc(ctx, ctx->tg, (size_t)ctx->max_S * T);
        if (s1 != ADASCALE_OK) return s1;
        s1 = table_alloc(ctx, ctx->tw, 2 * T + (T + 1) / 2);
        if (s1 != ADASCALE_OK) return s1;
        CU(cudaMallocHost(&ctx->h_snap, sizeof(DevState)));
        std::memset(ctx->h_snap, 0, sizeof(DevState));
        CU(cudaEventCreateWithFlags(&ctx->ev_snap, cudaEventDisableTiming));
        return ADASCALE_OK;
    };
    const adascale_status rc = body();
    if (rc != ADASCALE_OK) {
        adascale_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return ADASCALE_OK;
}

adascale_status adascale_destroy(adascale_ctx *ctx)
{
    if (!ctx) return ADASCALE_OK;
    DeviceGuard guard(ctx->device);
    if (guard.ok) {
        cudaDeviceSynchronize();
        cudaFree(ctx->d_rtiles);
        cudaFree(ctx->d_utiles);
        cudaFree(ctx->d_gbar);
        cudaFree(ctx->d_partials);
        cudaFree(ctx->d_ticket);
        cudaFree(ctx->d_state);
        cudaFree(ctx->d_stage);
        table_free(ctx->tg);
        table_free(ctx->tw);
        if (ctx->h_snap) cudaFreeHost(ctx->h_snap);
        if (ctx->ev_snap) cudaEventDestroy(ctx->ev_snap);
        cudaGetLastError();
    }
    delete ctx;
    return ADASCALE_OK;
}

adascale_status adascale_reduce(adascale_ctx *ctx, const void *const *grads, const adascale_lr_schedule *sched,
                                void *cuda_stream)
{
    if (!ctx || !grads || !valid_sched(sched)) return ADASCALE_ERR_INVALID_ARG;
    if (ctx->flags & ADASCALE_FLAG_FUSED) return ADASCALE_ERR_STATE;  // one pass: only adascale_step exists
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    return do_reduce(ctx, grads, sched, (cudaStream_t)cuda_stream, false);
}

adascale_status adascale_update(adascale_ctx *ctx, void *const *params, void *const *momentum, void *cuda_stream)
{
    if (!ctx || !params || !momentum) return ADASCALE_ERR_INVALID_ARG;
    if (!ctx->reduced || (ctx->flags & ADASCALE_FLAG_FUSED)) return ADASCALE_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    return do_update(ctx, params, momentum, (cudaStream_t)cuda_stream);
}

adascale_status adascale_step(adascale_ctx *ctx, const void *const *grads, void *const *params,
                              void *const *momentum, const adascale_lr_schedule *sched, void *cuda_stream)
{
    if (!ctx || !grads || !params || !momentum || !valid_sched(sched)) return ADASCALE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    // validate the update's pointers before anything is enqueued
    for (int k = 0; k < ctx->T; ++k) {
        if (ctx->numel[k] > 0) {
            if (!params[k] || !momentum[k]) return ADASCALE_ERR_INVALID_ARG;
            if (((uintptr_t)params[k] % 4) || ((uintptr_t)momentum[k] % 4)) return ADASCALE_ERR_ALIGNMENT;
        }
    }
    if (ctx->flags & ADASCALE_FLAG_FUSED) {
        adascale_status sf = sync_update_table(ctx, params, momentum, (cudaStream_t)cuda_stream);
        if (sf != ADASCALE_OK) return sf;
        return do_reduce(ctx, grads, sched, (cudaStream_t)cuda_stream, true);
    }
    adascale_status st = do_reduce(ctx, grads, sched, (cudaStream_t)cuda_stream, false);
    if (st != ADASCALE_OK) return st;
    return do_update(ctx, params, momentum, (cudaStream_t)cuda_stream);
}

adascale_status adascale_get_gain_tau(adascale_ctx *ctx, adascale_stats *out, int blocking)
{
    if (!ctx || !out) return ADASCALE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    cudaStream_t s = ctx->last_stream;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU(cudaStreamIsCapturing(s, &cap));
    if (cap != cudaStreamCaptureStatusNone) return ADASCALE_ERR_STATE;
    if (ctx->snap_inflight) {
        if (blocking) {
            CU(cudaEventSynchronize(ctx->ev_snap));
            ctx->latest = *ctx->h_snap;
            ctx->snap_inflight = false;
        } else {
            cudaError_t q = cudaEventQuery(ctx->ev_snap);
            if (q == cudaSuccess) {
                ctx->latest = *ctx->h_snap;
                ctx->snap_inflight = false;
            } else if (q != cudaErrorNotReady) {
                return cuda_fail(ctx, q, "cudaEventQuery");
            }
        }
    }
    if (!ctx->snap_inflight) {
        CU(cudaMemcpyAsync(ctx->h_snap, ctx->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, s));
        CU(cudaEventRecord(ctx->ev_snap, s));
        ctx->snap_inflight = true;
        if (blocking) {
            CU(cudaEventSynchronize(ctx->ev_snap));
            ctx->latest = *ctx->h_snap;
            ctx->snap_inflight = false;
        }
    }
    fill_stats(ctx->latest, out);
    return ADASCALE_OK;
}

adascale_status adascale_mean_grad(adascale_ctx *ctx, const void **gbar)
{
    if (!ctx || !gbar) return ADASCALE_ERR_INVALID_ARG;
    if (ctx->flags & ADASCALE_FLAG_FUSED) return ADASCALE_ERR_STATE;  // the mean gradient is never stored
    for (int k = 0; k < ctx->T; ++k) gbar[k] = ctx->d_gbar + ctx->goff[k];
    return ADASCALE_OK;
}

adascale_status adascale_set_scale(adascale_ctx *ctx, int32_t S)
{
    if (!ctx || S < 1) return ADASCALE_ERR_INVALID_ARG;
    if (S > ctx->max_S) return ADASCALE_ERR_TOO_LARGE;
    if (S != ctx->S) {
        ctx->S = S;
        ctx->tg.valid = false;
    }
    return ADASCALE_OK;
}

adascale_status adascale_get_state(adascale_ctx *ctx, void *buf)
{
    if (!ctx || !buf) return ADASCALE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    DevState d;
    CU(cudaStreamSynchronize(ctx->last_stream));
    CU(cudaMemcpy(&d, ctx->d_state, sizeof d, cudaMemcpyDeviceToHost));
    StateBlob b;
    std::memset(&b, 0, sizeof b);
    b.magic = kMagic;
    b.version = 1;
    b.S = ctx->S;
    b.flags = ctx->flags;
    b.tau = d.tau;
    b.avg_a = d.avg_a;
    b.avg_b = d.avg_b;
    b.n = d.n;
    b.t = d.t;
    b.skipped = d.skipped;
    b.r = d.r;
    b.eta = d.eta;
    b.lr = d.lr;
    std::memcpy(buf, &b, sizeof b);
    return ADASCALE_OK;
}

adascale_status adascale_set_state(adascale_ctx *ctx, const void *buf)
{
    if (!ctx || !buf) return ADASCALE_ERR_INVALID_ARG;
    StateBlob b;
    std::memcpy(&b, buf, sizeof b);
    if (b.magic != kMagic || b.version != 1) return ADASCALE_ERR_INVALID_ARG;
    if (b.S < 1 || b.S > ctx->max_S) return ADASCALE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    DevState d;
    std::memset(&d, 0, sizeof d);
    d.tau = b.tau;
    d.avg_a = b.avg_a;
    d.avg_b = b.avg_b;
    d.n = b.n;
    d.t = b.t;
    d.skipped = b.skipped;
    d.r = b.r;
    d.eta = b.eta;
    d.lr = b.lr;
    CU(cudaStreamSynchronize(ctx->last_stream));
    CU(cudaMemcpy(ctx->d_state, &d, sizeof d, cudaMemcpyHostToDevice));
    if (b.S != ctx->S) {
        ctx->S = b.S;
        ctx->tg.valid = false;
    }
    ctx->reduced = false;
    return ADASCALE_OK;
}

adascale_status adascale_step_host(adascale_ctx *ctx, const void *const *grads, void *const *params,
                                   void *const *momentum, const adascale_lr_schedule *sched,
                                   adascale_stats *out, void *cuda_stream)
{
    if (!ctx || !grads || !params || !momentum || !valid_sched(sched)) return ADASCALE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t esz = ctx->dtype == ADASCALE_BF16 ? 2 : 4;
    const int S = ctx->S, T = ctx->T;
    if (!ctx->d_stage) {
        CU(cudaMalloc(&ctx->d_stage, (size_t)ctx->max_S * (size_t)(ctx->gbar_elems > 0 ? ctx->gbar_elems : 1) * esz));
    }
    ctx->stage_ptrs.assign((size_t)S * T, nullptr);
    for (int i = 0; i < S; ++i)
        for (int k = 0; k < T; ++k)
            if (ctx->numel[k] > 0 && !grads[(size_t)i * T + k]) return ADASCALE_ERR_INVALID_ARG;
    for (int i = 0; i < S; ++i) {
        char *row = (char *)ctx->d_stage + (size_t)i * ctx->gbar_elems * esz;
        // tensors that continue each other in host memory and in the staging row travel as one copy
        const char *run_src = nullptr;
        char *run_dst = nullptr;
        size_t run_bytes = 0;
        for (int k = 0; k < T; ++k) {
            const char *src = (const char *)grads[(size_t)i * T + k];
            char *dst = row + (size_t)ctx->goff[k] * esz;
            ctx->stage_ptrs[(size_t)i * T + k] = dst;
            const size_t bytes = (size_t)ctx->numel[k] * esz;
            if (bytes == 0) continue;
            if (run_bytes && src == run_src + run_bytes && dst == run_dst + run_bytes) {
                run_bytes += bytes;
                continue;
            }
            if (run_bytes) CU(cudaMemcpyAsync(run_dst, run_src, run_bytes, cudaMemcpyHostToDevice, s));
            run_src = src;
            run_dst = dst;
            run_bytes = bytes;
        }
        if (run_bytes) CU(cudaMemcpyAsync(run_dst, run_src, run_bytes, cudaMemcpyHostToDevice, s));
    }
    adascale_status st = adascale_step(ctx, ctx->stage_ptrs.data(), params, momentum, sched, cuda_stream);
    if (st != ADASCALE_OK) return st;
    adascale_stats tmp;
    st = adascale_get_gain_tau(ctx, out ? out : &tmp, 1);
    if (st != ADASCALE_OK) return st;
    CU(cudaStreamSynchronize(s));
    return ADASCALE_OK;
}

adascale_status adascale_stream_probe(int32_t kind, void *a, void *b, int64_t n_bytes, void *cuda_stream)
{
    adascale_ctx *ctx = nullptr;
    if (!a || n_bytes < 16 || (n_bytes % 16) || ((uintptr_t)a % 16)) return ADASCALE_ERR_INVALID_ARG;
    if (kind < 0 || kind > 2) return ADASCALE_ERR_INVALID_ARG;
    if (kind != 0 && (!b || ((uintptr_t)b % 16))) return ADASCALE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const long long n = n_bytes / 16;
    int dev = 0, sms = 0;
    CU(cudaGetDevice(&dev));
    CU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    long long blocks = (n + kThreads - 1) / kThreads;
    const long long cap = (long long)sms * 32;
    if (blocks > cap) blocks = cap;
    if (kind == 0) {
        if (!b) return ADASCALE_ERR_INVALID_ARG;  // 4-byte sink that keeps the loads alive
        k_probe_read<<<(unsigned)blocks, kThreads, 0, s>>>((const uint4 *)a, n, (unsigned *)b);
    } else if (kind == 1) {
        k_probe_copy<<<(unsigned)blocks, kThreads, 0, s>>>((const uint4 *)a, (uint4 *)b, n);
    } else {
        k_probe_rmw<<<(unsigned)blocks, kThreads, 0, s>>>((float4 *)a, (const float4 *)b, n);
    }
    CU(cudaGetLastError());
    return ADASCALE_OK;
}

adascale_status adascale_grad_stats_static(const void *const *rows, int32_t S, int32_t grad_dtype, int64_t n,
                                           void *gbar, void *sums, void *cuda_stream)
{
    adascale_ctx *ctx = nullptr;  // for the CU macro: there is no context here
    if (!rows || !gbar || !sums || S < 1 || n < 1) return ADASCALE_ERR_INVALID_ARG;
    if (grad_dtype != ADASCALE_F32 && grad_dtype != ADASCALE_BF16) return ADASCALE_ERR_INVALID_ARG;
    if (S > kStaticMaxRows || n > ADASCALE_STATIC_MAX_NUMEL) return ADASCALE_ERR_TOO_LARGE;
    for (int i = 0; i < S; ++i) {
        if (!rows[i]) return ADASCALE_ERR_INVALID_ARG;
        if ((uintptr_t)rows[i] % 16) return ADASCALE_ERR_ALIGNMENT;
    }
    if (((uintptr_t)gbar % 16) || ((uintptr_t)sums % 8)) return ADASCALE_ERR_ALIGNMENT;
    cudaStream_t s = (cudaStream_t)cuda_stream;

    // Set-up, once per device and with that device current: in host code the array's name is
    // only a handle, the address a kernel can use comes from cudaGetSymbolAddress.
    static std::mutex mu;
    static unsigned char *scratch_of[64] = {nullptr};
    static int sms_of[64] = {0};
    int dev = 0;
    CU(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ADASCALE_ERR_INVALID_ARG;
    unsigned char *scratch = nullptr;
    int sms = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!scratch_of[dev]) {
            void *p = nullptr;
            CU(cudaGetSymbolAddress(&p, g_static_scratch));
            CU(cudaDeviceGetAttribute(&sms_of[dev], cudaDevAttrMultiProcessorCount, dev));
            scratch_of[dev] = static_cast<unsigned char *>(p);
        }
        scratch = scratch_of[dev];
        sms = sms_of[dev];
    }

    // the row pointers go into the scratch array; the ticket must start at zero whatever the
    // previous call left behind
    u64 table[kStaticMaxRows] = {0};
    for (int i = 0; i < S; ++i) table[i] = (u64)(uintptr_t)rows[i];
    CU(cudaMemcpyAsync(scratch, table, kStaticPtrBytes, cudaMemcpyHostToDevice, s));  // pageable: staged before return
    CU(cudaMemsetAsync(scratch + kStaticTicketOff, 0, sizeof(unsigned), s));

    StaticArgs a;
    a.scratch = scratch;
    a.gbar = static_cast<float *>(gbar);
    a.sums = static_cast<double *>(sums);
    a.n = n;
    a.S = S;
    a.fS = (float)S;
    a.invS = 1.0f / (float)S;
    long long blocks = (n / 8 + kThreads - 1) / kThreads;
    const long long cap = (long long)sms * 8 < kStaticMaxBlocks ? (long long)sms * 8 : kStaticMaxBlocks;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (grad_dtype == ADASCALE_BF16)
        k_grad_stats_static<ADASCALE_BF16><<<(unsigned)blocks, kThreads, 0, s>>>(a);
    else
        k_grad_stats_static<ADASCALE_F32><<<(unsigned)blocks, kThreads, 0, s>>>(a);
    CU(cudaGetLastError());
    return ADASCALE_OK;
}

}  // extern "C"
