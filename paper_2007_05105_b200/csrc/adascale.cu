// AdaScale SGD gain-ratio step for sm_100a: C-ABI host glue around the kernels of
// adascale_kernels.cuh, plus the one kernel whose scratch memory is a static device array
// (kept in this file together with the host code that looks up its address).
#include "adascale_kernels.cuh"

namespace {

// ---------------------------------------------------------------------------------------
// Allocation-free variant of the reduce kernel for one tensor: the same shifted sums, the
// same fp64 partials and fixed-order second stage, but rows are read with plain 128-bit loads
// and the scratch the kernel needs besides its inputs and outputs (ticket, per-block
// partials) lives in one file-scope device array instead of memory from cudaMalloc.  The row
// pointers travel by value in the kernel's parameters, so the call copies nothing from host
// memory.
// ---------------------------------------------------------------------------------------
constexpr int kStaticMaxRows = ADASCALE_STATIC_MAX_ROWS;
constexpr int kStaticMaxBlocks = 1024;
constexpr size_t kStaticTicketOff = 0;      // one counter, padded to 256 bytes
constexpr size_t kStaticPartialOff = 256;   // kStaticMaxBlocks pairs of doubles
constexpr size_t kStaticScratchBytes = kStaticPartialOff + kStaticMaxBlocks * sizeof(double2);

// Shared by every call on this device and kept until the process exits (about 16 KB).
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticArgs {
    u64 rows[kStaticMaxRows];  // device addresses of the S rows
    unsigned char *scratch;    // device address of g_static_scratch, resolved on the host
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
    const u64 *rows = a.rows;
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
    double2 *d_partials = nullptr;        // per block (scalar-path tiles)
    double2 *d_run_partials = nullptr;    // per run of staged tiles, or per block
    unsigned *d_ticket = nullptr;
    DevState *d_state = nullptr;
    // A reduce launch of a small or mid-size job leaves the scalar part of its iteration to the
    // kernel that follows: normally the update, else a one-block kernel enqueued as soon as
    // anything else needs the state.
    bool scalar_open = false;
    int open_pairs = 0;
    ScalarCfg open_sc;
    PtrTable tg, tw;
    long long n_tiles = 0, n_stiles = 0;  // of the descriptors on the device
    DevState *h_snap = nullptr;  // pinned
    cudaEvent_t ev_snap = nullptr;
    bool snap_inflight = false;
    DevState latest{};
    cudaStream_t last_stream = nullptr;
    bool reduced = false;
    unsigned wait_spins = kSpinLimit;  // bound of the reduce kernel's handshake waits
    int forced_runs = -1;              // >= 0: tiles per run (0 = static assignment) whatever the job's size
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

int rows_per_stage(int dtype, int S) { return S < max_rows_per_stage(dtype) ? S : max_rows_per_stage(dtype); }

long long staged_tiles(const long long *numel, const unsigned char *aligned, int T, int tile_cols)
{
    long long n = 0;
    for (int k = 0; k < T; ++k)
        if (!aligned || aligned[k]) n += ((numel[k] & ~7LL) + tile_cols - 1) / tile_cols;
    return n;
}

// Columns per consumer thread.  A thread reads 8, 16 or 32 bytes of each row; the widest
// access that keeps one stage (rows x 256 threads x bytes) within kStageBytes is used, and
// small jobs step down so that every block still gets two tiles (more, narrower tiles cost
// more barrier round trips than they gain in balance: 1M parameters, S = 4: 7.9 against 10.2 us).
int choose_cpt(int dtype, int S, const long long *numel, const unsigned char *aligned, int T, int n_blocks)
{
    const int esz = dtype == ADASCALE_BF16 ? 2 : 4;
    int bpt = dtype == ADASCALE_BF16 ? 16 : 32;
    while (bpt > 8 && rows_per_stage(dtype, S) * kThreads * bpt > kStageBytes) bpt >>= 1;
    while (bpt > 8 && staged_tiles(numel, aligned, T, kThreads * bpt / esz) < 2LL * n_blocks) bpt >>= 1;
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

void fill_scalar_args(const adascale_ctx *ctx, const adascale_lr_schedule *sched, ScalarCfg &sc, Sched &out)
{
    sc.eps = ctx->eps;
    sc.theta = resolve_theta(ctx);
    sc.flags = ctx->flags;
    sc.S = ctx->S;
    out.kind = sched->kind;
    out.n = sched->kind == ADASCALE_LR_STEP ? sched->n_milestones : 0;
    out.eta0 = sched->eta0;
    out.decay = sched->decay;
    out.t_s1 = sched->t_s1;
    for (int i = 0; i < ADASCALE_MAX_MILESTONES; ++i) out.w[i] = sched->milestones[i];
}

// Validates the caller's gradient pointers, rebuilds the tiling if the tile width or a tensor's
// alignment changed, and uploads the pointer table ([max_S * T] row pointers).  Skipped entirely
// when the pointers are those of the previous call.
adascale_status sync_reduce_table(adascale_ctx *ctx, const void *const *grads, cudaStream_t s)
{
    const int S = ctx->S, T = ctx->T;
    const size_t esz = ctx->dtype == ADASCALE_BF16 ? 2 : 4;
    const size_t n_ptrs = (size_t)S * T;
    if (ctx->tg.valid && ctx->tiled_cpt != 0 && ctx->last_grads.size() == n_ptrs &&
        std::memcmp(ctx->last_grads.data(), grads, n_ptrs * sizeof(void *)) == 0)
        return ADASCALE_OK;

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
    const int cpt = choose_cpt(ctx->dtype, S, ctx->numel.data(), aligned.data(), T, ctx->sms * kReduceBlocksPerSM);
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
        if ((long long)tiles.size() > ctx->rtiles_cap) return ADASCALE_ERR_TOO_LARGE;  // sized for the worst case
        if (!tiles.empty()) {
            CU(cudaMemcpyAsync(ctx->d_rtiles, tiles.data(), tiles.size() * sizeof(TileDesc), cudaMemcpyHostToDevice, s));
            CU(cudaStreamSynchronize(s));  // `tiles` goes out of scope
        }
        ctx->n_tiles = n_staged;
        ctx->n_stiles = (long long)tiles.size() - n_staged;
        ctx->tiled_cpt = cpt;
        ctx->tiled_aligned = aligned;
    }
    adascale_status st = table_sync(ctx, ctx->tg, fresh, s);
    if (st != ADASCALE_OK) return st;
    ctx->last_grads.assign(grads, grads + n_ptrs);
    return ADASCALE_OK;
}

// Staged tiles handed out together by the reduce kernel; 0 = static assignment (tile t to block
// t mod grid).  Handing tiles out from a counter pays on large jobs only (it keeps all blocks on
// one narrow window of the matrix); runs keep the number of pairs to add up afterwards small.
long long run_tiles_for(long long n_tiles, int S)
{
    // tiles of a single row chunk (S <= 8) are too short for the producer warp's extra work per tile:
    // 6 % slower from the counter than statically at 50-100M parameters
    if (n_tiles < kDynamicMinTiles || S <= max_rows_per_stage(0)) return 0;
    return n_tiles >= 4 * kDynamicMinTiles ? 4 : 2;
}

// Completes an iteration whose scalar part a reduce launch has left open and that no update launch took over.
adascale_status finish_open_scalar(adascale_ctx *ctx, cudaStream_t s)
{
    if (!ctx->scalar_open) return ADASCALE_OK;
    FinishArgs a;
    a.st = ctx->d_state;
    a.partials = ctx->d_partials;
    a.n_partials = ctx->open_pairs;
    a.prepared = reinterpret_cast<const ScalarPrep *>(ctx->d_ticket + 128);
    a.sc = ctx->open_sc;
    cudaError_t e = launch_overlapped(k_finish, 1, kThreads, 0, s, a);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the scalar kernel");
    ctx->launches += 1;
    ctx->scalar_open = false;
    ctx->last_stream = s;
    return ADASCALE_OK;
}

adascale_status do_reduce(adascale_ctx *ctx, const void *const *grads, const adascale_lr_schedule *sched,
                          cudaStream_t s, bool fused, double *sums_out = nullptr)
{
    const int S = ctx->S, T = ctx->T;
    if (ctx->scalar_open) {  // two reduce launches in a row: the first one's iteration is completed first
        adascale_status so = finish_open_scalar(ctx, s);
        if (so != ADASCALE_OK) return so;
    }
    const size_t esz = ctx->dtype == ADASCALE_BF16 ? 2 : 4;
    const int max_blocks = ctx->sms * kReduceBlocksPerSM;
    adascale_status st = sync_reduce_table(ctx, grads, s);
    if (st != ADASCALE_OK) return st;
    const int cpt = ctx->tiled_cpt;
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
    a.run_partials = ctx->d_run_partials;
    a.run_tiles = ctx->forced_runs >= 0 ? ctx->forced_runs : run_tiles_for(n_tiles, S);
    // Two stages in flight per block are enough and measured 2-5 % faster than three when tiles are
    // assigned statically; with runs from a counter three were 2 % faster.
    a.stages = a.run_tiles > 0 ? (unsigned)kStages : 2u;
    // Runs of run_tiles tiles, except at the end of the launch: the tiles of the last runs (two per
    // block, but no more than half of all) are handed out one by one, so that the blocks finish
    // within a tile of each other.
    a.long_runs = 0;
    if (a.run_tiles > 0) {
        const long long n_full = n_tiles / a.run_tiles;
        long long singles = 2LL * max_blocks;
        if (singles > n_full / 2) singles = n_full / 2;
        a.long_runs = n_full - singles;
    }
    const long long n_run_pairs = a.run_tiles > 0 ? a.long_runs + (n_tiles - a.long_runs * a.run_tiles) : 0;
    a.ticket = ctx->d_ticket;
    a.tile_counter = reinterpret_cast<u64 *>(ctx->d_ticket + 192);
    a.st = ctx->d_state;
    a.sums_out = sums_out;
    // Sums not wanted by the caller: the reduce kernel stops at its pairs of sums.  Two-kernel form,
    // static assignment: one pair per block, which every block of the update kernel adds up itself.
    // Runs from the counter: a small kernel first brings the run pairs down to a few dozen; in the
    // one-pass form, where no update kernel follows, the one-block scalar kernel comes right after
    // it (with the static assignment the one-pass form keeps its last block: the next launch's
    // blocks are then already waiting on the SMs when the scalar part ends).
    const bool leave_open = !sums_out && (!fused || a.run_tiles > 0);
    a.prepared = reinterpret_cast<ScalarPrep *>(ctx->d_ticket + 128);
    a.leave_open = leave_open ? 1u : 0u;
    a.spin_limit = ctx->wait_spins;
    a.early_rows = (ctx->flags & ADASCALE_FLAG_GRADS_READY) ? 1u : 0u;
    a.S = S;
    a.T = T;
    a.fS = (float)S;
    a.invS = 1.0f / (float)S;
    fill_scalar_args(ctx, sched, a.sc, a.sched);

    long long nb = n_tiles + n_stiles;
    if (nb > max_blocks) nb = max_blocks;
    const size_t smem = (size_t)a.stages * rows_per_stage(ctx->dtype, S) * kThreads * cpt * esz;
    cudaError_t e = launch_reduce(fused, ctx->dtype, cpt, (int)nb, a, smem, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the reduce kernel");
    ctx->launches += 1;
    ctx->reduced = true;
    ctx->last_stream = s;
    if (leave_open) {
        ctx->scalar_open = true;
        ctx->open_pairs = (int)nb;
        ctx->open_sc = a.sc;
        if (a.run_tiles > 0) {
            SumArgs sa;
            sa.run_partials = ctx->d_run_partials;
            sa.n_pairs = n_run_pairs;
            sa.out = ctx->d_partials + nb;
            sa.tile_counter = a.tile_counter;
            long long sb = (sa.n_pairs + kThreads - 1) / kThreads;
            if (sb > kSumBlocks) sb = kSumBlocks;
            if (sb < 1) sb = 1;
            e = launch_overlapped(k_sum, (int)sb, kThreads, 0, s, sa);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the pair-sum kernel");
            ctx->launches += 1;
            ctx->open_pairs = (int)(nb + sb);
        }
        if (fused) return finish_open_scalar(ctx, s);
    }
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
    a.next_tile = ctx->d_ticket + 64;
    a.T = T;
    a.rho = (float)ctx->rho;
    a.lambda = (float)ctx->lambda;
    a.partials = ctx->d_partials;
    a.n_partials = ctx->open_pairs;
    a.prepared = reinterpret_cast<const ScalarPrep *>(ctx->d_ticket + 128);
    a.sc = ctx->open_sc;
    long long nb = n_tiles;
    if (nb > (long long)ctx->sms * kUpdateBlocksPerSM) nb = (long long)ctx->sms * kUpdateBlocksPerSM;
    cudaError_t e = ctx->scalar_open ? launch_overlapped(k_update<true>, (int)nb, kThreads, 0, s, a)
                                     : launch_overlapped(k_update<false>, (int)nb, kThreads, 0, s, a);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the update kernel");
    ctx->scalar_open = false;
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
    *rows = rows_per_stage(grad_dtype, S);
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
    if (cfg->flags & ~(ADASCALE_FLAG_LAGGED | ADASCALE_FLAG_CONT_TAU | ADASCALE_FLAG_RATIO | ADASCALE_FLAG_FUSED |
                       ADASCALE_FLAG_GRADS_READY))
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
    if (ctx->n_utiles > 0xffffffffLL) {  // the update kernel's tile counter is 32 bits wide
        delete ctx;
        return ADASCALE_ERR_TOO_LARGE;
    }
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
        CU(cudaMalloc(&ctx->d_partials, (size_t)(ctx->sms * kReduceBlocksPerSM + kSumBlocks + 1) * sizeof(double2)));
        CU(cudaMalloc(&ctx->d_run_partials,
                      (size_t)(rcap + ctx->sms * kReduceBlocksPerSM + 1) * sizeof(double2)));
        // counters and scratch, 256 bytes apart: exit ticket, update tiles, prepared scalar part, runs
        CU(cudaMalloc(&ctx->d_ticket, 4 * 256));
        CU(cudaMemset(ctx->d_ticket, 0, 4 * 256));
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
        cudaFree(ctx->d_run_partials);
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

adascale_status adascale_reduce_sums(adascale_ctx *ctx, const void *const *grads, void *sums, void *cuda_stream)
{
    if (!ctx || !grads || !sums) return ADASCALE_ERR_INVALID_ARG;
    if ((uintptr_t)sums % 8) return ADASCALE_ERR_ALIGNMENT;
    if (ctx->flags & ADASCALE_FLAG_FUSED) return ADASCALE_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (ctx->P == 0) {  // no kernel runs for a shard without elements: its sums are zero
        CU(cudaMemsetAsync(sums, 0, 2 * sizeof(double), s));
        ctx->last_stream = s;
        return ADASCALE_OK;
    }
    adascale_lr_schedule unused = {};
    unused.kind = ADASCALE_LR_CONST;
    unused.eta0 = 1.0;
    return do_reduce(ctx, grads, &unused, s, false, static_cast<double *>(sums));
}

adascale_status adascale_apply_sums(adascale_ctx *ctx, const void *sums, const adascale_lr_schedule *sched,
                                    void *const *params, void *const *momentum, void *cuda_stream)
{
    if (!ctx || !sums || !params || !momentum || !valid_sched(sched)) return ADASCALE_ERR_INVALID_ARG;
    if ((uintptr_t)sums % 8) return ADASCALE_ERR_ALIGNMENT;
    if (ctx->flags & ADASCALE_FLAG_FUSED) return ADASCALE_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    adascale_status st = sync_update_table(ctx, params, momentum, s);  // before anything is enqueued
    if (st != ADASCALE_OK) return st;
    st = finish_open_scalar(ctx, s);
    if (st != ADASCALE_OK) return st;
    ScalarArgs a;
    a.st = ctx->d_state;
    a.sums = static_cast<const double *>(sums);
    fill_scalar_args(ctx, sched, a.sc, a.sched);
    cudaError_t e = launch_overlapped(k_scalar, 1, 32, 0, s, a);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch of the scalar kernel");
    ctx->launches += 1;
    ctx->reduced = true;
    ctx->last_stream = s;
    return do_update(ctx, params, momentum, s);
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
    {
        adascale_status so = finish_open_scalar(ctx, s);  // a reduce launch with no update after it
        if (so != ADASCALE_OK) return so;
    }
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

adascale_status adascale_set_wait_limit(adascale_ctx *ctx, uint32_t polls)
{
    if (!ctx) return ADASCALE_ERR_INVALID_ARG;
    ctx->wait_spins = polls;
    return ADASCALE_OK;
}

adascale_status adascale_set_tile_runs(adascale_ctx *ctx, int32_t run_tiles)
{
    if (!ctx || run_tiles < -1 || run_tiles > 64) return ADASCALE_ERR_INVALID_ARG;
    ctx->forced_runs = run_tiles;
    return ADASCALE_OK;
}

adascale_status adascale_get_state(adascale_ctx *ctx, void *buf)
{
    if (!ctx || !buf) return ADASCALE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    DevState d;
    {
        adascale_status so = finish_open_scalar(ctx, ctx->last_stream);
        if (so != ADASCALE_OK) return so;
    }
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
    ctx->scalar_open = false;  // the state is replaced as a whole: an iteration left open is dropped with it
    CU(cudaStreamSynchronize(ctx->last_stream));
    CU(cudaMemcpy(ctx->d_state, &d, sizeof d, cudaMemcpyHostToDevice));
    // a launch that gave up on a wait may have left its work counters half way
    CU(cudaMemset(ctx->d_ticket, 0, 4 * 256));
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

    // the ticket must start at zero whatever the previous call left behind
    CU(cudaMemsetAsync(scratch + kStaticTicketOff, 0, sizeof(unsigned), s));

    StaticArgs a;
    for (int i = 0; i < kStaticMaxRows; ++i) a.rows[i] = i < S ? (u64)(uintptr_t)rows[i] : 0;
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
