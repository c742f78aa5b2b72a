// C interface of the CD-Adam library (see include/cdadam.h): context, state buffers and the
// per-step launch sequence.  No arithmetic of the method lives here.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/cdadam.h"
#include "kernels.h"
#include "topk.h"

using namespace cdadam;

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

#define CU_TRY(expr)                                                                       \
    do {                                                                                   \
        cudaError_t e_ = (expr);                                                           \
        if (e_ != cudaSuccess)                                                             \
            return fail(e_ == cudaErrorMemoryAllocation ? CDADAM_ERR_ALLOC : CDADAM_ERR_CUDA, \
                        "%s: %s", #expr, cudaGetErrorString(e_));                          \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) {
            cudaSetDevice(dev);
            switched = true;
        }
    }
    ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

// Tile sizes, multiples of kSub.  Larger tiles amortise the per-block reduction, make the
// streams longer and (from 4 sub-tiles on) enable the worker pass's prefetch ring; but every
// tile that contains a segment boundary takes the scalar path, and a row needs enough tiles
// to fill the machine.  The scalar path of the server pass loops over the n workers per
// coordinate and is the costlier one, so the server side (server pass, update pass) gets its
// own, more cautious, tile size: `slack` bounds 1 / (share of coordinates in cut tiles).
int choose_tile(int64_t d, int q, bool server_side)
{
    const int64_t slack = server_side ? 50 : 16;
    int tile = kSub;
    if (d >= ((int64_t)1 << 23) && (int64_t)(q - 1) * (2 * kSub) * slack <= d && !server_side) tile = 2 * kSub;
    if (d >= ((int64_t)1 << 24) && (int64_t)(q - 1) * (2 * kSub) * slack <= d) tile = 2 * kSub;
    if (d >= ((int64_t)1 << 25) && (int64_t)(q - 1) * (4 * kSub) * slack <= d) tile = 4 * kSub;
    // The worker pass with its prefetch ring gains from long tiles (a block's ring starts empty
    // and its partial sum costs a block reduction): on 8 x 110 M coordinates 16384 -> 1.60 ms,
    // 20480 -> 1.56, 32768 -> 1.57, 65536 -> 1.61 per pass under a power cap, the step 2.62 ->
    // 2.54 ms; 4 x 1.5 G: 11.3 -> 10.6 ms per pass.  The server pass is best at 16384.
    if (!server_side && d >= ((int64_t)1 << 26) && (int64_t)(q - 1) * (8 * kSub) * slack <= d) tile = 8 * kSub;
    return tile;
}

// Host tables + their device copies.
struct TableSet {
    Tables tb{};
    std::vector<int64_t> off;
    void *dev = nullptr;        // one allocation holding off, pbase, tile_first, tile_last

    int build(int64_t d, int q, const int64_t *offsets, int tile, cudaStream_t st, bool async)
    {
        release(st, async);
        off.assign(offsets, offsets + q + 1);
        const int64_t ntiles = (d + tile - 1) / tile;
        std::vector<int32_t> first(ntiles), last(ntiles);
        std::vector<int64_t> pbase(ntiles);
        int r = 0;
        int64_t np = 0;
        for (int64_t T = 0; T < ntiles; ++T) {
            const int64_t lo = T * tile, hi = std::min<int64_t>(d, lo + tile) - 1;
            while (off[r + 1] <= lo) ++r;
            first[T] = r;
            int e = r;
            while (off[e + 1] <= hi) ++e;
            last[T] = e;
            pbase[T] = np;
            np += e - r + 1;
        }
        std::vector<int32_t> order;
        order.reserve(ntiles);
        for (int pass = 0; pass < 2; ++pass)          // slow tiles first, then the rest in order
            for (int64_t T = 0; T < ntiles; ++T) {
                const bool slow = first[T] != last[T] || (T + 1) * (int64_t)tile > d;
                if (slow == (pass == 0)) order.push_back((int32_t)T);
            }
        const size_t b_off = (size_t)(q + 1) * 8, b_pb = (size_t)ntiles * 8, b_t = (size_t)ntiles * 4;
        const size_t total = b_off + b_pb + 3 * b_t;
        cudaError_t e = async ? cudaMallocAsync(&dev, total, st) : cudaMalloc(&dev, total);
        if (e != cudaSuccess) { dev = nullptr; return fail(CDADAM_ERR_ALLOC, "table allocation: %s", cudaGetErrorString(e)); }
        char *p = (char *)dev;
        // pageable sources: the runtime stages them before these calls return
        CU_TRY(cudaMemcpyAsync(p, off.data(), b_off, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(p + b_off, pbase.data(), b_pb, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(p + b_off + b_pb, first.data(), b_t, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(p + b_off + b_pb + b_t, last.data(), b_t, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(p + b_off + b_pb + 2 * b_t, order.data(), b_t, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaStreamSynchronize(st));
        tb.d = d; tb.q = q; tb.tile = tile; tb.ntiles = ntiles; tb.nparts = np;
        tb.off = (const int64_t *)p;
        tb.pbase = (const int64_t *)(p + b_off);
        tb.tile_first = (const int32_t *)(p + b_off + b_pb);
        tb.tile_last = (const int32_t *)(p + b_off + b_pb + b_t);
        tb.order = (const int32_t *)(p + b_off + b_pb + 2 * b_t);
        return CDADAM_OK;
    }
    void release(cudaStream_t st, bool async)
    {
        if (dev) { if (async) cudaFreeAsync(dev, st); else cudaFree(dev); }
        dev = nullptr;
    }
};

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

constexpr int64_t kFuseMaxBlocks = 4 * 148;   // one wave of 256-thread blocks at 4 per SM

struct cdadam_ctx {
    int64_t d = 0, k = 0, wp = 0, steps = 0;
    int n = 0, comp = 0, device = 0;
    // Distributed deployment: this context holds the workers [first, first + nloc) of the n.
    // An ordinary context holds all of them (first = 0, nloc = n).  The worker state and the
    // worker pass's scratch have nloc rows; the message buffers (wbits, wscale) have n rows.
    int first = 0, nloc = 0;
    int phase = 0;          // split step: 0 = between iterations, 1 = worker stage queued, 2 = server stage queued
    // Coordinate-sharded iteration: this context owns the coordinates [range_lo, range_lo + d)
    // of all n workers' vectors and of the server's, in a problem of dimension range_dim, as
    // range number range_rank of range_count.  Segments are those of the whole problem cut to
    // the range: local segment r is segment rs_gidx[r] of q_all, of whole length rs_glen[r].
    bool is_range = false;
    int64_t range_lo = 0, range_dim = 0;
    int range_rank = 0, range_count = 1, q_all = 1;
    dd *rs_w = nullptr, *rs_s = nullptr;      // l1 sums of all ranges: range_count x n x q_all, range_count x q_all
    int32_t *rs_gidx = nullptr;               // q_loc (device)
    int64_t *rs_glen = nullptr;               // q_loc (device)
    std::vector<int64_t> range_off_all;       // the whole problem's q_all + 1 segment offsets
    int64_t range_k = 0;                      // top-k: entries kept in the WHOLE vector
    uint32_t *rx_w = nullptr, *rx_s = nullptr;   // top-k exchange buffers: range_count x (n | 1) x 2048 words
    int tile_override = 0;  // 0 = choose from d and q
    int mode = CDADAM_MARKOV;
    Hyper hp{};
    float wd = 0.0f;             // decoupled weight decay lambda
    float base_lr = 0.0f, gamma = 1.0f;          // step-size milestones
    std::vector<int64_t> milestones;
    TableSet ts;            // worker pass
    TableSet ts_s;          // server pass and update pass
    float *ghat_w = nullptr, *ghat_s = nullptr, *gtil = nullptr;
    float *m = nullptr, *v = nullptr, *vhat = nullptr, *x = nullptr;
    // scaled sign
    uint32_t *wbits = nullptr, *sbits = nullptr;
    float *wscale[2] = {nullptr, nullptr}, *sscale = nullptr, *zero_scale = nullptr;
    dd *wpart = nullptr, *spart = nullptr;
    unsigned int *wdone = nullptr, *sdone = nullptr;   // tickets of the in-kernel scale finish
    int wsplit = 1, ssplit = 1;  // blocks that share a segment in the separate scale kernel
    dd *wsums = nullptr, *ssums = nullptr;
    bool fuse_finish = false;    // scales finished inside the worker / server pass
    int *error_flag = nullptr;   // device word set by a kernel whose bounded wait ran out
    int wait_limit = -1;         // polls before such a wait gives up (< 0: the kernels' default)
    bool void_state = false;     // a wait ran out (seen by cdadam_device_status): no further iterations
    int cur = 0;            // wscale[cur] holds the scales of the last worker payloads
    bool pending = false;   // the last worker payloads are not yet added to ghat_w
    bool sets_given = false;   // rand-k: coordinate sets have been supplied
    // top-k
    TopkWorkspace *tk_w = nullptr, *tk_s = nullptr;
    // a top-k context that holds a part of the workers: the messages of all n workers
    // (n x k coordinates and values); tk_w then selects into the rows of its own workers
    uint32_t *pay_idx = nullptr;
    float *pay_val = nullptr;
    // top-k per segment: a selection workspace per segment (rows strided by d); tk_w / tk_s
    // then hold only the concatenated payloads
    std::vector<int64_t> seg_off, seg_k, seg_at;
    std::vector<TopkWorkspace *> seg_w, seg_s;
    // host-gradient staging
    float *stage = nullptr;
    // Replay of a step as a CUDA graph where launches matter: scaled sign with grids of one
    // wave, and top-k (some thirty launches, most of them short).  A graph is recorded for a
    // gradient buffer seen twice; the key holds every launch argument that changes between
    // steps.
    struct StepGraph {
        const void *grads = nullptr;
        bool bf16 = false, pending = false;
        int cur = 0, hits = 0;
        uint64_t stamp = 0;
        cudaGraphExec_t exec = nullptr;
    };
    StepGraph graphs[4];
    uint64_t graph_clock = 0;
    cudaStream_t cap_stream = nullptr;
    bool graphs_ok = true;       // cleared for good when recording fails once, or when graphs go
                                 // stale too often (a step size that changes every step)
    int graph_drops = 0;
    std::vector<cudaGraphExec_t> retired;   // stale graphs, possibly still running: freed with the context
    // optional per-kernel timing: events[step][0..nslots] recorded around every stage
    bool prof_on = false;
    std::vector<cudaEvent_t> prof_ev;   // groups of (nslots + 1) events, one group per step
    std::vector<cudaEvent_t> prof_pool;
};

namespace {

template <typename T>
int dev_zalloc(T **p, size_t count)
{
    *p = nullptr;
    const size_t bytes = (count ? count : 1) * sizeof(T);
    cudaError_t e = cudaMalloc((void **)p, bytes);
    if (e != cudaSuccess) return fail(CDADAM_ERR_ALLOC, "cudaMalloc(%zu bytes): %s", bytes, cudaGetErrorString(e));
    CU_TRY(cudaMemset(*p, 0, bytes));
    return CDADAM_OK;
}

// Blocks of the separate scale kernel that share one segment: one per 4096 tiles, up to 32.
int finalize_split(const TableSet &ts)
{
    int64_t most = 1;
    for (size_t r = 0; r + 1 < ts.off.size(); ++r)
        most = std::max(most, (ts.off[r + 1] - 1) / ts.tb.tile - ts.off[r] / ts.tb.tile + 1);
    return (int)std::min<int64_t>(32, (most + 4095) / 4096);
}

int alloc_sign_buffers(cdadam_ctx *c)
{
    const int q = c->ts.tb.q;
    cudaFree(c->wscale[0]); cudaFree(c->wscale[1]); cudaFree(c->sscale); cudaFree(c->zero_scale);
    cudaFree(c->wpart); cudaFree(c->spart); cudaFree(c->wdone); cudaFree(c->sdone);
    cudaFree(c->wsums); cudaFree(c->ssums);
    c->wsums = c->ssums = nullptr;
    int rc;
    if ((rc = dev_zalloc(&c->wscale[0], (size_t)c->n * q))) return rc;
    if ((rc = dev_zalloc(&c->wscale[1], (size_t)c->n * q))) return rc;
    if ((rc = dev_zalloc(&c->zero_scale, (size_t)c->n * q))) return rc;
    if ((rc = dev_zalloc(&c->sscale, (size_t)q))) return rc;
    if ((rc = dev_zalloc(&c->wpart, (size_t)c->nloc * c->ts.tb.nparts))) return rc;
    if ((rc = dev_zalloc(&c->spart, (size_t)c->ts_s.tb.nparts))) return rc;
    if ((rc = dev_zalloc(&c->wdone, (size_t)c->nloc * q))) return rc;
    if ((rc = dev_zalloc(&c->sdone, (size_t)q))) return rc;
    // Finishing the scales inside the passes saves two launches but lengthens every block by
    // a fence and an atomic round trip: measured 12 % faster when all blocks of a pass are
    // resident at once (d = 65,536, n = 4) and 4 to 13 % slower on grids of many waves.
    c->fuse_finish = (int64_t)c->nloc * c->ts.tb.ntiles <= kFuseMaxBlocks && c->ts_s.tb.ntiles <= kFuseMaxBlocks;
    // a segment of more than 4096 tiles is shared by several blocks of the scale kernel
    c->wsplit = finalize_split(c->ts);
    c->ssplit = finalize_split(c->ts_s);
    if (c->wsplit > 1 && (rc = dev_zalloc(&c->wsums, (size_t)c->nloc * q * c->wsplit))) return rc;
    if (c->ssplit > 1 && (rc = dev_zalloc(&c->ssums, (size_t)q * c->ssplit))) return rc;
    return CDADAM_OK;
}

// Segments of the whole problem cut to the context's coordinate range: local offsets (from 0
// to d), and for every local segment its number and length in the whole problem.
void cut_segments(const cdadam_ctx *c, int q_all, const int64_t *off_all, std::vector<int64_t> &off_loc,
                  std::vector<int32_t> &gidx, std::vector<int64_t> &glen)
{
    const int64_t lo = c->range_lo, hi = c->range_lo + c->d;
    off_loc.assign(1, 0);
    gidx.clear(); glen.clear();
    for (int r = 0; r < q_all; ++r) {
        const int64_t a = std::max(off_all[r], lo), b = std::min(off_all[r + 1], hi);
        if (a >= b) continue;
        off_loc.push_back(b - lo);
        gidx.push_back(r);
        glen.push_back(off_all[r + 1] - off_all[r]);
    }
}

// Buffers of the coordinate-sharded iteration for the current segments (tables already built).
int alloc_range_buffers(cdadam_ctx *c, int q_all, const std::vector<int32_t> &gidx, const std::vector<int64_t> &glen)
{
    cudaFree(c->rs_w); cudaFree(c->rs_s); cudaFree(c->rs_gidx); cudaFree(c->rs_glen);
    c->rs_w = c->rs_s = nullptr; c->rs_gidx = nullptr; c->rs_glen = nullptr;
    c->q_all = q_all;
    int rc;
    if ((rc = dev_zalloc(&c->rs_w, (size_t)c->range_count * c->n * q_all))) return rc;
    if ((rc = dev_zalloc(&c->rs_s, (size_t)c->range_count * q_all))) return rc;
    if ((rc = dev_zalloc(&c->rs_gidx, gidx.size()))) return rc;
    if ((rc = dev_zalloc(&c->rs_glen, glen.size()))) return rc;
    CU_TRY(cudaMemcpy(c->rs_gidx, gidx.data(), gidx.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    CU_TRY(cudaMemcpy(c->rs_glen, glen.data(), glen.size() * sizeof(int64_t), cudaMemcpyHostToDevice));
    c->fuse_finish = false;      // a scale needs the other ranges' sums: never finished inside a pass
    return CDADAM_OK;
}

float *state_ptr(cdadam_ctx *c, int name)
{
    switch (name) {
    case CDADAM_STATE_GHAT_W: return c->ghat_w;
    case CDADAM_STATE_GHAT_S: return c->ghat_s;
    case CDADAM_STATE_GTIL: return c->gtil;
    case CDADAM_STATE_M: return c->m;
    case CDADAM_STATE_V: return c->v;
    case CDADAM_STATE_VHAT: return c->vhat;
    case CDADAM_STATE_X: return c->x;
    }
    return nullptr;
}

int prof_slots(const cdadam_ctx *c)
{
    return c->comp == CDADAM_SIGN ? (c->fuse_finish && c->mode != CDADAM_NAIVE ? 3 : 5) : (c->comp == CDADAM_TOPK || c->comp == CDADAM_RANDK) ? 4 : 1;
}

// Record the boundary event after a stage (or before the first one) when timing is on.
void prof_mark(cdadam_ctx *c, cudaStream_t st)
{
    if (!c->prof_on) return;
    cudaEvent_t e;
    if (!c->prof_pool.empty()) { e = c->prof_pool.back(); c->prof_pool.pop_back(); }
    else if (cudaEventCreate(&e) != cudaSuccess) return;
    cudaEventRecord(e, st);
    c->prof_ev.push_back(e);
}

void drop_graphs(cdadam_ctx *c);

// The step size and everything derived from it (launch arguments, hence recorded graphs).
void apply_lr(cdadam_ctx *c, float lr)
{
    const float lrwd = lr * c->wd;
    if (lr == c->hp.lr && lrwd == c->hp.lrwd && (c->wd != 0.0f) == (c->hp.decay != 0)) return;
    drop_graphs(c);
    c->hp.lr = lr;
    c->hp.lrwd = lrwd;
    c->hp.decay = c->wd != 0.0f;
}

constexpr int kMaxGraphDrops = 4;

// A recorded graph whose launch arguments are stale.  It may still be running, so it is only
// set aside; a context that keeps invalidating its graphs stops recording them.
void retire_graph(cdadam_ctx *c, cdadam_ctx::StepGraph &g)
{
    if (g.exec) {
        c->retired.push_back(g.exec);
        if (++c->graph_drops > kMaxGraphDrops * 4) c->graphs_ok = false;
    }
    g = cdadam_ctx::StepGraph{};
}

void drop_graphs(cdadam_ctx *c)
{
    for (auto &g : c->graphs) retire_graph(c, g);
}

// The stages of one scaled-sign step, queued on st; none changes host state.  `new_scale`
// is the n x q array that receives (workers) or holds (server) the scales of this iteration's
// worker messages.  The worker stage covers the context's own workers: rows
// [first, first + nloc) of the message buffers.
void enqueue_sign_workers(cdadam_ctx *c, const void *grads_in, bool bf16, bool vec, float *new_scale, cudaStream_t st)
{
    const Tables &tb = c->ts.tb;
    const bool naive = c->mode == CDADAM_NAIVE;
    const bool fuse = c->fuse_finish && !naive;
    const int64_t so = (int64_t)c->first * tb.q;
    const float *old_scale = (c->pending ? c->wscale[c->cur] : c->zero_scale) + so;
    uint32_t *bits = c->wbits + (int64_t)c->first * c->wp;
    if (c->nloc > 0) {
        if (naive)      // the payload is C(g) itself: no worker state is read or written
            launch_pack_sign(static_cast<const float *>(grads_in), bits, c->wpart, tb, c->nloc, c->wp, vec, st);
        else
            launch_worker_sign(grads_in, bf16, c->ghat_w, bits, old_scale, c->wpart, tb, c->nloc, c->wp, vec,
                               c->mode == CDADAM_EF, c->error_flag, fuse ? new_scale + so : nullptr, c->wdone, st,
                               c->wait_limit);
    }
    prof_mark(c, st);
    if (!fuse) {
        if (c->nloc > 0) launch_finalize_scales(c->wpart, new_scale + so, tb, c->nloc, st, c->wsplit, c->wsums, c->wdone);
        prof_mark(c, st);
    }
}

void enqueue_sign_server(cdadam_ctx *c, const float *new_scale, cudaStream_t st)
{
    const Tables &tbs = c->ts_s.tb;
    const bool fuse = c->fuse_finish && c->mode != CDADAM_NAIVE;
    launch_server_sign(c->wbits, new_scale, c->ghat_s, c->gtil, c->sbits, c->spart, tbs, c->n, c->wp, c->d % 4 == 0, c->mode,
                       fuse ? c->sscale : nullptr, c->sdone, st);
    prof_mark(c, st);
    if (!fuse) {
        launch_finalize_scales(c->spart, c->sscale, tbs, 1, st, c->ssplit, c->ssums, c->sdone);
        prof_mark(c, st);
    }
}

void enqueue_sign_update(cdadam_ctx *c, cudaStream_t st)
{
    launch_update_sign(c->sbits, c->sscale, c->ghat_s, c->gtil, c->m, c->v, c->vhat, c->x, c->ts_s.tb, c->hp, c->d % 4 == 0,
                       c->mode, st);
    prof_mark(c, st);
}

// The three to five launches of one scaled-sign step, queued on st.  Changes no host state.
void enqueue_sign_step(cdadam_ctx *c, const void *grads_in, bool bf16, bool vec, cudaStream_t st)
{
    float *new_scale = c->wscale[c->cur ^ 1];
    enqueue_sign_workers(c, grads_in, bf16, vec, new_scale, st);
    enqueue_sign_server(c, new_scale, st);
    enqueue_sign_update(c, st);
}

// One iteration of Algorithm 1 with the top-k compressor, queued on st.  No host state changes.
void enqueue_topk_step(cdadam_ctx *c, const void *grads_in, bool, bool vec, cudaStream_t st)
{
    const float *grads = static_cast<const float *>(grads_in);
    const bool svec = c->d % 4 == 0;
    if (!c->seg_w.empty()) {
        // the compressor on every segment on its own; the payloads are concatenated (still
        // listed by increasing coordinate) and the rest of the iteration is as without segments
        const int q = (int)c->seg_w.size();
        for (int r = 0; r < q; ++r) {
            const int64_t lo = c->seg_off[r];
            topk_select(c->seg_w[r], grads + lo, c->ghat_w + lo, true, vec && lo % 4 == 0, st);
            topk_payload_concat(c->tk_w, c->seg_at[r], c->seg_w[r], lo, st);
        }
        prof_mark(c, st);
        topk_aggregate(c->tk_w, c->ghat_s, c->n, st);
        prof_mark(c, st);
        for (int r = 0; r < q; ++r) {
            const int64_t lo = c->seg_off[r];
            topk_select(c->seg_s[r], c->ghat_s + lo, c->gtil + lo, true, svec && lo % 4 == 0, st);
            topk_payload_concat(c->tk_s, c->seg_at[r], c->seg_s[r], lo, st);
        }
        prof_mark(c, st);
        launch_amsgrad(c->gtil, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
        prof_mark(c, st);
        return;
    }
    topk_select(c->tk_w, grads, c->ghat_w, true, vec, st);            // workers: compress, update ghat^(i)
    prof_mark(c, st);
    prof_mark(c, st);                                                  // (the aggregation runs inside the server's dense pass)
    topk_select_aggregated(c->tk_s, c->tk_w, c->ghat_s, c->gtil, c->n, svec, st);   // server: ghat += mean; compress, update gtil
    prof_mark(c, st);
    launch_amsgrad(c->gtil, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
    prof_mark(c, st);
}

// Launch-bound steps: replays the recorded graph of this step on st and returns true, or
// returns false when the step has to be queued launch by launch (first sighting of the
// gradient buffer, timing on, recording unavailable).
typedef void (*enqueue_fn)(cdadam_ctx *, const void *, bool, bool, cudaStream_t);

bool replay_step(cdadam_ctx *c, const void *grads_in, bool bf16, bool vec, cudaStream_t st, enqueue_fn enqueue)
{
    if (!c->graphs_ok || c->prof_on) return false;
    cdadam_ctx::StepGraph *slot = nullptr, *oldest = &c->graphs[0];
    for (auto &g : c->graphs) {
        if (g.hits && g.grads == grads_in && g.bf16 == bf16 && g.pending == c->pending && g.cur == c->cur) slot = &g;
        if (g.stamp < oldest->stamp) oldest = &g;
    }
    if (!slot) {                                               // remember the sighting only
        retire_graph(c, *oldest);
        oldest->grads = grads_in; oldest->bf16 = bf16; oldest->pending = c->pending; oldest->cur = c->cur;
        oldest->hits = 1; oldest->stamp = ++c->graph_clock;
        return false;
    }
    slot->hits += 1;
    slot->stamp = ++c->graph_clock;
    if (!slot->exec) {
        cudaGraph_t graph = nullptr;
        bool ok = c->cap_stream || cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
        if (ok) {
            enqueue(c, grads_in, bf16, vec, c->cap_stream);
            ok = cudaStreamEndCapture(c->cap_stream, &graph) == cudaSuccess && graph;
        }
        ok = ok && cudaGraphInstantiate(&slot->exec, graph, 0) == cudaSuccess;
        if (graph) cudaGraphDestroy(graph);
        if (!ok) {
            cudaGetLastError();
            slot->exec = nullptr;
            c->graphs_ok = false;
            return false;
        }
    }
    if (cudaGraphLaunch(slot->exec, st) != cudaSuccess) {
        cudaGetLastError();
        c->graphs_ok = false;
        return false;
    }
    return true;
}

int check_launch(const char *what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CDADAM_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return CDADAM_OK;
}

}  // namespace

namespace cdadam {
void set_last_error(const char *message) { snprintf(g_err, sizeof g_err, "%s", message); }
}  // namespace cdadam

extern "C" {

const char *cdadam_last_error(void) { return g_err; }

static cdadam_ctx *create_impl(int64_t d, int n, int first, int nloc, int compressor, int64_t k, float beta1,
                               float beta2, float lr, float eps)
{
    if (d < 1 || d >= ((int64_t)1 << 32)) { fail(CDADAM_ERR_ARG, "d must be in [1, 2^32)"); return nullptr; }
    if (n < 1 || n > 65535) { fail(CDADAM_ERR_ARG, "n must be in [1, 65535]"); return nullptr; }
    if (first < 0 || nloc < 0 || first + nloc > n) { fail(CDADAM_ERR_ARG, "the context's workers [first, first + n_local) must lie in [0, n)"); return nullptr; }
    if (nloc != n && compressor != CDADAM_SIGN && compressor != CDADAM_TOPK) { fail(CDADAM_ERR_ARG, "a context that holds a part of the workers needs the scaled-sign or the top-k compressor"); return nullptr; }
    if (compressor < CDADAM_SIGN || compressor > CDADAM_RANDK) { fail(CDADAM_ERR_ARG, "unknown compressor %d", compressor); return nullptr; }
    if ((compressor == CDADAM_TOPK || compressor == CDADAM_RANDK) && (k < 1 || k > d)) { fail(CDADAM_ERR_ARG, "top-k and rand-k need 1 <= k <= d"); return nullptr; }
    cdadam_ctx *c = new (std::nothrow) cdadam_ctx;
    if (!c) { fail(CDADAM_ERR_ALLOC, "out of host memory"); return nullptr; }
    c->d = d; c->n = n; c->first = first; c->nloc = nloc;
    c->comp = compressor; c->k = (compressor == CDADAM_TOPK || compressor == CDADAM_RANDK) ? k : 0;
    c->wp = (d + 31) / 32;
    c->hp.beta1 = beta1; c->hp.beta2 = beta2; c->hp.lr = lr; c->hp.nu = eps;
    c->hp.omb1 = 1.0f - beta1; c->hp.omb2 = 1.0f - beta2;
    if (cudaGetDevice(&c->device) != cudaSuccess) { fail(CDADAM_ERR_CUDA, "no CUDA device"); delete c; return nullptr; }
    int rc = CDADAM_OK;
    const int64_t flat[2] = {0, d};
    do {
        if ((rc = dev_zalloc(&c->ghat_w, (size_t)nloc * d))) break;
        if ((rc = dev_zalloc(&c->ghat_s, (size_t)d))) break;
        if ((rc = dev_zalloc(&c->gtil, (size_t)d))) break;
        if ((rc = dev_zalloc(&c->m, (size_t)d))) break;
        if ((rc = dev_zalloc(&c->v, (size_t)d))) break;
        if ((rc = dev_zalloc(&c->vhat, (size_t)d))) break;
        if ((rc = dev_zalloc(&c->x, (size_t)d))) break;
        if ((rc = dev_zalloc(&c->error_flag, 1))) break;
        if (compressor == CDADAM_SIGN) {
            if ((rc = dev_zalloc(&c->wbits, (size_t)n * c->wp))) break;
            if ((rc = dev_zalloc(&c->sbits, (size_t)c->wp))) break;
            if ((rc = c->ts.build(d, 1, flat, choose_tile(d, 1, false), nullptr, false))) break;
            if ((rc = c->ts_s.build(d, 1, flat, choose_tile(d, 1, true), nullptr, false))) break;
            if ((rc = alloc_sign_buffers(c))) break;
        } else if (compressor == CDADAM_RANDK) {
            if ((rc = topk_workspace_create(&c->tk_w, d, c->k, n, nullptr, nullptr, false))) { fail(rc, "rand-k payload allocation failed"); break; }
            if ((rc = topk_workspace_create(&c->tk_s, d, c->k, 1, nullptr, nullptr, false))) { fail(rc, "rand-k payload allocation failed"); break; }
        } else if (compressor == CDADAM_TOPK && nloc != n) {
            if ((rc = dev_zalloc(&c->pay_idx, (size_t)n * c->k))) break;
            if ((rc = dev_zalloc(&c->pay_val, (size_t)n * c->k))) break;
            if ((rc = topk_workspace_create(&c->tk_w, d, c->k, nloc > 0 ? nloc : 1, c->pay_idx + (int64_t)first * c->k,
                                            c->pay_val + (int64_t)first * c->k))) { fail(rc, "top-k workspace allocation failed"); break; }
            if ((rc = topk_workspace_create(&c->tk_s, d, c->k, 1))) { fail(rc, "top-k workspace allocation failed"); break; }
        } else if (compressor == CDADAM_TOPK) {
            if ((rc = topk_workspace_create(&c->tk_w, d, c->k, n))) { fail(rc, "top-k workspace allocation failed"); break; }
            if ((rc = topk_workspace_create(&c->tk_s, d, c->k, 1))) { fail(rc, "top-k workspace allocation failed"); break; }
        }
    } while (0);
    if (rc != CDADAM_OK || cudaDeviceSynchronize() != cudaSuccess) { cdadam_destroy(c); return nullptr; }
    // the stream on which a step is recorded for replay (not inside cdadam_step)
    if (cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); c->cap_stream = nullptr; }
    topk_workspace_set_error_flag(c->tk_w, c->error_flag);
    topk_workspace_set_error_flag(c->tk_s, c->error_flag);
    // Algorithm 1 with top-k: ghat^(i) += c^(i) at the kept coordinates is left to the next
    // iteration's dense pass (cdadam_get_state applies what is pending)
    if (compressor == CDADAM_TOPK) topk_workspace_set_defer(c->tk_w, true);
    return c;
}

cdadam_ctx *cdadam_create(int64_t d, int n, int compressor, int64_t k, float beta1, float beta2,
                          float lr, float eps)
{
    return create_impl(d, n, 0, n, compressor, k, beta1, beta2, lr, eps);
}

cdadam_ctx *cdadam_create_shard(int64_t d, int n, int first_worker, int n_local, int compressor, int64_t k,
                                float beta1, float beta2, float lr, float eps)
{
    if (compressor != CDADAM_SIGN && compressor != CDADAM_TOPK) {
        fail(CDADAM_ERR_ARG, "the staged iteration takes the scaled-sign or the top-k compressor");
        return nullptr;
    }
    return create_impl(d, n, first_worker, n_local, compressor, k, beta1, beta2, lr, eps);
}

cdadam_ctx *cdadam_create_range(int64_t d, int n, int64_t lo, int64_t hi, int range, int ranges, int compressor,
                                int64_t k, float beta1, float beta2, float lr, float eps)
{
    if (compressor != CDADAM_SIGN && compressor != CDADAM_TOPK) {
        fail(CDADAM_ERR_ARG, "the coordinate-sharded iteration takes the scaled-sign or the top-k compressor");
        return nullptr;
    }
    if (d < 1 || d >= ((int64_t)1 << 32)) { fail(CDADAM_ERR_ARG, "d must be in [1, 2^32)"); return nullptr; }
    if (lo < 0 || hi <= lo || hi > d) { fail(CDADAM_ERR_ARG, "the range [lo, hi) must be non-empty and lie in [0, d)"); return nullptr; }
    if (ranges < 1 || ranges > 4096 || range < 0 || range >= ranges) { fail(CDADAM_ERR_ARG, "range number must be in [0, ranges), ranges in [1, 4096]"); return nullptr; }
    if (compressor == CDADAM_TOPK && (k < 1 || k > d)) { fail(CDADAM_ERR_ARG, "top-k needs 1 <= k <= d"); return nullptr; }
    // a payload row of this range holds at most min(k, hi - lo) entries
    cdadam_ctx *c = create_impl(hi - lo, n, 0, n, compressor, compressor == CDADAM_TOPK ? std::min(k, hi - lo) : 0,
                                beta1, beta2, lr, eps);
    if (!c) return nullptr;
    c->is_range = true;
    c->range_lo = lo; c->range_dim = d; c->range_rank = range; c->range_count = ranges;
    if (compressor == CDADAM_SIGN) {
        const int64_t flat[2] = {0, d};
        if (cdadam_set_segments(c, 1, flat) != CDADAM_OK) { cdadam_destroy(c); return nullptr; }
        return c;
    }
    c->range_k = k;
    topk_workspace_set_defer(c->tk_w, false);          // the staged selection updates ghat^(i) at once
    const size_t per = (size_t)topk_range_exchange_words(c->tk_s);
    if (dev_zalloc(&c->rx_w, (size_t)ranges * n * per) || dev_zalloc(&c->rx_s, (size_t)ranges * per)) {
        cdadam_destroy(c);
        return nullptr;
    }
    return c;
}

void cdadam_destroy(cdadam_ctx *c)
{
    if (!c) return;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    cudaFree(c->ghat_w); cudaFree(c->ghat_s); cudaFree(c->gtil);
    cudaFree(c->m); cudaFree(c->v); cudaFree(c->vhat); cudaFree(c->x);
    cudaFree(c->wbits); cudaFree(c->sbits); cudaFree(c->error_flag);
    cudaFree(c->pay_idx); cudaFree(c->pay_val);
    cudaFree(c->rs_w); cudaFree(c->rs_s); cudaFree(c->rs_gidx); cudaFree(c->rs_glen);
    cudaFree(c->rx_w); cudaFree(c->rx_s);
    cudaFree(c->wscale[0]); cudaFree(c->wscale[1]); cudaFree(c->sscale); cudaFree(c->zero_scale);
    cudaFree(c->wpart); cudaFree(c->spart); cudaFree(c->stage);
    cudaFree(c->wdone); cudaFree(c->sdone); cudaFree(c->wsums); cudaFree(c->ssums);
    topk_workspace_destroy(c->tk_w); topk_workspace_destroy(c->tk_s);
    for (TopkWorkspace *w : c->seg_w) topk_workspace_destroy(w);
    for (TopkWorkspace *w : c->seg_s) topk_workspace_destroy(w);
    drop_graphs(c);
    for (cudaGraphExec_t e : c->retired) cudaGraphExecDestroy(e);
    if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    for (cudaEvent_t e : c->prof_pool) cudaEventDestroy(e);
    c->ts.release(nullptr, false);
    c->ts_s.release(nullptr, false);
    delete c;
}

static int ensure_stage(cdadam_ctx *c)
{
    if (c->stage) return CDADAM_OK;
    const size_t bytes = (size_t)(c->nloc ? c->nloc : 1) * c->d * sizeof(float);
    cudaError_t e = cudaMalloc((void **)&c->stage, bytes);
    if (e != cudaSuccess) { c->stage = nullptr; return fail(CDADAM_ERR_ALLOC, "staging buffer: %s", cudaGetErrorString(e)); }
    return CDADAM_OK;
}

// Launch arguments alternate from step to step (double-buffered scales, the deferred
// payload), so a step recorded into a caller's graph would replay wrongly.
static int refuse_capture(cudaStream_t st)
{
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) cudaGetLastError();
    else if (cs != cudaStreamCaptureStatusNone)
        return fail(CDADAM_ERR_STATE, "cdadam_step: the stream is being captured; a step cannot be part of a caller's graph");
    return CDADAM_OK;
}

// alpha_t = base * gamma^(milestones already passed), by repeated binary32 products
static void step_size_of_this_step(cdadam_ctx *c)
{
    if (c->milestones.empty()) return;
    float lr = c->base_lr;
    for (int64_t after : c->milestones)
        if (after <= c->steps) lr = lr * c->gamma;
    apply_lr(c, lr);
}

static int step_impl(cdadam_ctx *c, const void *grads_in, bool bf16, void *stream)
{
    if (!c || !grads_in) return fail(CDADAM_ERR_ARG, "cdadam_step: NULL argument");
    if (c->nloc != c->n) return fail(CDADAM_ERR_STATE, "cdadam_step: this context holds a part of the workers; use the staged calls");
    if (c->is_range) return fail(CDADAM_ERR_STATE, "cdadam_step: this context holds a part of the coordinates; use the cdadam_range_* calls");
    if (c->phase != 0) return fail(CDADAM_ERR_STATE, "cdadam_step: a staged iteration is under way");
    if (c->void_state) return fail(CDADAM_ERR_STATE, "cdadam_step: a kernel's wait ran out in an earlier iteration; the state is not valid");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    const float *grads = static_cast<const float *>(grads_in);
    if (bf16 && (c->comp != CDADAM_SIGN || c->mode == CDADAM_NAIVE)) {
        // only the scaled-sign worker pass reads bfloat16 directly; the other compressors
        // (and naive compression) get an exact binary32 copy in the context's staging buffer
        int rc = ensure_stage(c);
        if (rc) return rc;
        launch_widen_bf16(c->stage, grads_in, (int64_t)c->n * c->d, st);
        grads = c->stage;
        bf16 = false;
    }
    const bool vec = aligned16(grads) && c->d % (bf16 ? 8 : 4) == 0;
    step_size_of_this_step(c);
    prof_mark(c, st);
    const bool ef = c->mode == CDADAM_EF;
    const bool naive = c->mode == CDADAM_NAIVE;
    const bool svec = c->d % 4 == 0;
    if (c->comp == CDADAM_SIGN) {
        const void *gin = bf16 ? grads_in : grads;
        const bool launch_bound = c->fuse_finish && !naive;
        if (!(launch_bound && replay_step(c, gin, bf16, vec, st, enqueue_sign_step))) enqueue_sign_step(c, gin, bf16, vec, st);
        c->cur ^= 1;
        c->pending = !naive;             // naive compression has no worker state to bring up to date
    } else if (naive && (c->comp == CDADAM_TOPK || c->comp == CDADAM_RANDK)) {
        // Naive compression (Section 4): c^(i) = C(g^(i)), c = C(mean_i c^(i)), AMSGrad on c.
        // ghat_s is all zero between steps: it receives the sparse mean, is compressed, then
        // carries the dense decoded server payload for AMSGrad and is cleared again.
        if (c->comp == CDADAM_RANDK && !c->sets_given)
            return fail(CDADAM_ERR_STATE, "rand-k needs cdadam_set_random_sets before the first step");
        const uint32_t *widx, *sidx;
        const float *wval, *sval;
        topk_payload(c->tk_w, 0, &widx, &wval);
        topk_payload(c->tk_s, 0, &sidx, &sval);
        if (c->comp == CDADAM_TOPK) topk_select(c->tk_w, grads, nullptr, false, vec, st);
        else randk_gather(c->tk_w, grads, nullptr, false, st);
        prof_mark(c, st);
        topk_aggregate(c->tk_w, c->ghat_s, c->n, st);
        prof_mark(c, st);
        if (c->comp == CDADAM_TOPK) topk_select(c->tk_s, c->ghat_s, nullptr, false, svec, st);
        else randk_gather(c->tk_s, c->ghat_s, nullptr, false, st);
        launch_scatter_zero_shared(c->ghat_s, widx, c->k, c->n, st);
        launch_scatter_set(c->ghat_s, sidx, sval, c->k, c->d, 1, st);
        prof_mark(c, st);
        launch_amsgrad(c->ghat_s, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
        launch_scatter_set(c->ghat_s, sidx, nullptr, c->k, c->d, 1, st);
        prof_mark(c, st);
    } else if (c->comp == CDADAM_TOPK && !ef) {
        // some thirty launches, most of them short: replayed from a graph where possible
        if (!replay_step(c, grads, false, vec, st, enqueue_topk_step)) enqueue_topk_step(c, grads, false, vec, st);
    } else if (c->comp == CDADAM_TOPK) {
        // classical error feedback: the delta buffers (ghat_w rows, gtil) first receive the
        // compressor inputs p = g + delta and p = mean + delta, are compressed in place, and
        // keep p - c, which is p outside the kept coordinates and 0 on them.  ghat_s is all
        // zero between steps and carries the dense decoded server payload for AMSGrad.
        const uint32_t *widx, *sidx;
        const float *wval, *sval;
        topk_payload(c->tk_w, 0, &widx, &wval);
        topk_payload(c->tk_s, 0, &sidx, &sval);
        launch_add_into(c->ghat_w, grads, (int64_t)c->n * c->d, vec, st);
        topk_select(c->tk_w, c->ghat_w, nullptr, false, svec, st);
        launch_scatter_set(c->ghat_w, widx, nullptr, c->k, c->d, c->n, st);
        prof_mark(c, st);
        topk_aggregate(c->tk_w, c->gtil, c->n, st);
        prof_mark(c, st);
        topk_select(c->tk_s, c->gtil, nullptr, false, svec, st);
        launch_scatter_set(c->gtil, sidx, nullptr, c->k, c->d, 1, st);
        launch_scatter_set(c->ghat_s, sidx, sval, c->k, c->d, 1, st);
        prof_mark(c, st);
        launch_amsgrad(c->ghat_s, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
        launch_scatter_set(c->ghat_s, sidx, nullptr, c->k, c->d, 1, st);
        prof_mark(c, st);
    } else if (c->comp == CDADAM_RANDK) {
        if (!c->sets_given) return fail(CDADAM_ERR_STATE, "rand-k needs cdadam_set_random_sets before the first step");
        const uint32_t *widx, *sidx;
        const float *wval, *sval;
        topk_payload(c->tk_w, 0, &widx, &wval);
        topk_payload(c->tk_s, 0, &sidx, &sval);
        if (!ef) {
            randk_gather(c->tk_w, grads, c->ghat_w, true, st);                 // workers: compress, update ghat^(i)
            prof_mark(c, st);
            topk_aggregate(c->tk_w, c->ghat_s, c->n, st);                      // server: ghat += mean
            prof_mark(c, st);
            randk_gather(c->tk_s, c->ghat_s, c->gtil, true, st);               // server: compress, update gtil
            prof_mark(c, st);
            launch_amsgrad(c->gtil, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
            prof_mark(c, st);
        } else {                                                               // as top-k above
            launch_add_into(c->ghat_w, grads, (int64_t)c->n * c->d, vec, st);
            randk_gather(c->tk_w, c->ghat_w, nullptr, false, st);
            launch_scatter_set(c->ghat_w, widx, nullptr, c->k, c->d, c->n, st);
            prof_mark(c, st);
            topk_aggregate(c->tk_w, c->gtil, c->n, st);
            prof_mark(c, st);
            randk_gather(c->tk_s, c->gtil, nullptr, false, st);
            launch_scatter_set(c->gtil, sidx, nullptr, c->k, c->d, 1, st);
            launch_scatter_set(c->ghat_s, sidx, sval, c->k, c->d, 1, st);
            prof_mark(c, st);
            launch_amsgrad(c->ghat_s, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
            launch_scatter_set(c->ghat_s, sidx, nullptr, c->k, c->d, 1, st);
            prof_mark(c, st);
        }
    } else {
        launch_step_identity(grads, c->ghat_w, c->ghat_s, c->gtil, c->m, c->v, c->vhat, c->x, c->d, c->n, c->hp, c->mode, st);
        prof_mark(c, st);
    }
    int rc = check_launch("cdadam_step");
    if (rc) return rc;
    c->steps += 1;
    return CDADAM_OK;
}

int cdadam_step(cdadam_ctx *c, const float *grads, void *stream) { return step_impl(c, grads, false, stream); }

// ---- one iteration in its three stages (distributed deployment of Algorithm 1) ---------------

static int staged_ok(cdadam_ctx *c, const char *what)
{
    if (!c) return fail(CDADAM_ERR_ARG, "%s: NULL context", what);
    if (c->comp != CDADAM_SIGN && c->comp != CDADAM_TOPK)
        return fail(CDADAM_ERR_STATE, "%s: the staged calls take the scaled-sign or the top-k compressor", what);
    if (c->comp == CDADAM_TOPK && (c->mode != CDADAM_MARKOV || !c->seg_w.empty()))
        return fail(CDADAM_ERR_STATE, "%s: with top-k the staged calls run Algorithm 1 on the whole vector only", what);
    if (c->prof_on) return fail(CDADAM_ERR_STATE, "%s: per-stage timing covers cdadam_step only", what);
    if (c->is_range) return fail(CDADAM_ERR_STATE, "%s: this context holds a part of the coordinates; use the cdadam_range_* calls", what);
    return CDADAM_OK;
}

int cdadam_step_workers(cdadam_ctx *c, const float *grads, void *stream)
{
    if (int rc = staged_ok(c, "cdadam_step_workers")) return rc;
    if (c->nloc > 0 && !grads) return fail(CDADAM_ERR_ARG, "cdadam_step_workers: NULL gradients");
    if (c->phase != 0) return fail(CDADAM_ERR_STATE, "cdadam_step_workers: the previous iteration has not been completed by cdadam_step_update");
    if (c->void_state) return fail(CDADAM_ERR_STATE, "cdadam_step_workers: a kernel's wait ran out in an earlier iteration; the state is not valid");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    step_size_of_this_step(c);
    const bool vec = aligned16(grads) && c->d % 4 == 0;
    if (c->comp == CDADAM_TOPK) {
        if (c->nloc > 0) topk_select(c->tk_w, grads, c->ghat_w, true, vec, st);   // workers: compress, update ghat^(i)
        if (int rc = check_launch("cdadam_step_workers")) return rc;
        c->phase = 1;
        return CDADAM_OK;
    }
    enqueue_sign_workers(c, grads, false, vec, c->wscale[c->cur ^ 1], st);
    if (int rc = check_launch("cdadam_step_workers")) return rc;
    c->cur ^= 1;                              // wscale[cur] now holds this iteration's scales
    c->pending = c->mode != CDADAM_NAIVE;
    c->phase = 1;
    return CDADAM_OK;
}

int cdadam_step_server(cdadam_ctx *c, void *stream)
{
    if (int rc = staged_ok(c, "cdadam_step_server")) return rc;
    if (c->phase != 1) return fail(CDADAM_ERR_STATE, "cdadam_step_server: call cdadam_step_workers first (once per iteration)");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    if (c->comp == CDADAM_TOPK) {
        // messages gathered from other processes come without the selecting side's per-tile
        // offsets: their entries are found by searching the sorted coordinates
        if (c->pay_idx) topk_aggregate_rows(c->pay_idx, c->pay_val, c->k, c->d, c->n, c->ghat_s, st);
        else topk_aggregate(c->tk_w, c->ghat_s, c->n, st);                       // server: ghat += mean
        topk_select(c->tk_s, c->ghat_s, c->gtil, true, c->d % 4 == 0, st);       // server: compress, update gtil
    } else {
        enqueue_sign_server(c, c->wscale[c->cur], st);
    }
    if (int rc = check_launch("cdadam_step_server")) return rc;
    c->phase = 2;
    return CDADAM_OK;
}

int cdadam_step_update(cdadam_ctx *c, void *stream)
{
    if (int rc = staged_ok(c, "cdadam_step_update")) return rc;
    if (c->phase == 0) return fail(CDADAM_ERR_STATE, "cdadam_step_update: call cdadam_step_workers first");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    if (c->comp == CDADAM_TOPK) {
        // a process that did not run the server stage holds the server's message (k coordinates
        // and values) in the buffers: gtil += c there, as the server did on its own copy
        if (c->phase == 1) {
            const uint32_t *sidx; const float *sval;
            topk_payload(c->tk_s, 0, &sidx, &sval);
            launch_scatter_add(c->gtil, sidx, sval, c->k, c->d, st);
        }
        launch_amsgrad(c->gtil, c->m, c->v, c->vhat, c->x, c->d, c->hp, c->d % 4 == 0, st);
    } else {
        enqueue_sign_update(c, st);
    }
    if (int rc = check_launch("cdadam_step_update")) return rc;
    c->phase = 0;
    c->steps += 1;
    return CDADAM_OK;
}

int cdadam_exchange_buffers(cdadam_ctx *c, uint32_t **worker_bits, float **worker_scales, uint32_t **server_bits,
                            float **server_scales, int64_t *words, int *q)
{
    if (int rc = staged_ok(c, "cdadam_exchange_buffers")) return rc;
    if (c->comp == CDADAM_TOPK) {
        const uint32_t *widx, *sidx;
        const float *wval, *sval;
        topk_payload(c->tk_w, 0, &widx, &wval);
        topk_payload(c->tk_s, 0, &sidx, &sval);
        if (worker_bits) *worker_bits = c->pay_idx ? c->pay_idx : const_cast<uint32_t *>(widx);
        if (worker_scales) *worker_scales = c->pay_val ? c->pay_val : const_cast<float *>(wval);
        if (server_bits) *server_bits = const_cast<uint32_t *>(sidx);
        if (server_scales) *server_scales = const_cast<float *>(sval);
        if (words) *words = c->k;
        if (q) *q = (int)std::min<int64_t>(c->k, 0x7fffffff);
        return CDADAM_OK;
    }
    if (worker_bits) *worker_bits = c->wbits;
    if (worker_scales) *worker_scales = c->wscale[c->cur];
    if (server_bits) *server_bits = c->sbits;
    if (server_scales) *server_scales = c->sscale;
    if (words) *words = c->wp;
    if (q) *q = c->ts.tb.q;
    return CDADAM_OK;
}

// ---- one iteration on a coordinate range (coordinate-sharded deployment) ----------------------

static int range_ok(cdadam_ctx *c, const char *what)
{
    if (!c) return fail(CDADAM_ERR_ARG, "%s: NULL context", what);
    if (!c->is_range) return fail(CDADAM_ERR_STATE, "%s: the context was not made by cdadam_create_range", what);
    if (c->comp != CDADAM_SIGN) return fail(CDADAM_ERR_STATE, "%s: scaled sign only; a top-k range context runs cdadam_range_topk", what);
    if (c->mode == CDADAM_NAIVE) return fail(CDADAM_ERR_STATE, "%s: Algorithm 1 and the error-feedback mode only", what);
    if (c->prof_on) return fail(CDADAM_ERR_STATE, "%s: per-stage timing covers cdadam_step only", what);
    return CDADAM_OK;
}

int cdadam_range_workers(cdadam_ctx *c, const float *grads, void *stream)
{
    if (int rc = range_ok(c, "cdadam_range_workers")) return rc;
    if (!grads) return fail(CDADAM_ERR_ARG, "cdadam_range_workers: NULL gradients");
    if (c->phase != 0) return fail(CDADAM_ERR_STATE, "cdadam_range_workers: the previous iteration has not been completed by cdadam_range_update");
    if (c->void_state) return fail(CDADAM_ERR_STATE, "cdadam_range_workers: a kernel's wait ran out in an earlier iteration; the state is not valid");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    step_size_of_this_step(c);
    const Tables &tb = c->ts.tb;
    const bool vec = aligned16(grads) && c->d % 4 == 0;
    const float *old_scale = c->pending ? c->wscale[c->cur] : c->zero_scale;
    launch_worker_sign(grads, false, c->ghat_w, c->wbits, old_scale, c->wpart, tb, c->n, c->wp, vec, c->mode == CDADAM_EF,
                       c->error_flag, nullptr, c->wdone, st, c->wait_limit);
    launch_range_sums(c->wpart, c->rs_w + (int64_t)c->range_rank * c->n * c->q_all, tb, c->n, c->rs_gidx, c->q_all, st);
    if (int rc = check_launch("cdadam_range_workers")) return rc;
    c->cur ^= 1;                              // wscale[cur] receives this iteration's scales in the server stage
    c->pending = true;
    c->phase = 1;
    return CDADAM_OK;
}

int cdadam_range_server(cdadam_ctx *c, void *stream)
{
    if (int rc = range_ok(c, "cdadam_range_server")) return rc;
    if (c->phase != 1) return fail(CDADAM_ERR_STATE, "cdadam_range_server: call cdadam_range_workers first (once per iteration)");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    const Tables &tbs = c->ts_s.tb;
    launch_range_scales(c->rs_w, c->range_count, c->n, c->q_all, c->rs_gidx, c->rs_glen, c->wscale[c->cur], tbs.q, st);
    launch_server_sign(c->wbits, c->wscale[c->cur], c->ghat_s, c->gtil, c->sbits, c->spart, tbs, c->n, c->wp, c->d % 4 == 0,
                       c->mode, nullptr, c->sdone, st);
    launch_range_sums(c->spart, c->rs_s + (int64_t)c->range_rank * c->q_all, tbs, 1, c->rs_gidx, c->q_all, st);
    if (int rc = check_launch("cdadam_range_server")) return rc;
    c->phase = 2;
    return CDADAM_OK;
}

int cdadam_range_update(cdadam_ctx *c, void *stream)
{
    if (int rc = range_ok(c, "cdadam_range_update")) return rc;
    if (c->phase != 2) return fail(CDADAM_ERR_STATE, "cdadam_range_update: call cdadam_range_server first");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    launch_range_scales(c->rs_s, c->range_count, 1, c->q_all, c->rs_gidx, c->rs_glen, c->sscale, c->ts_s.tb.q, st);
    enqueue_sign_update(c, st);
    if (int rc = check_launch("cdadam_range_update")) return rc;
    c->phase = 0;
    c->steps += 1;
    return CDADAM_OK;
}

int cdadam_range_buffers(cdadam_ctx *c, double **worker_sums, double **server_sums, int64_t *worker_doubles,
                         int64_t *server_doubles, int *q_local, const int32_t **segment_of_local)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_range_buffers: NULL context");
    if (!c->is_range) return fail(CDADAM_ERR_STATE, "cdadam_range_buffers: the context was not made by cdadam_create_range");
    if (worker_sums) *worker_sums = reinterpret_cast<double *>(c->rs_w);
    if (server_sums) *server_sums = reinterpret_cast<double *>(c->rs_s);
    if (worker_doubles) *worker_doubles = 2 * (int64_t)c->n * c->q_all;
    if (server_doubles) *server_doubles = 2 * (int64_t)c->q_all;
    if (q_local) *q_local = c->ts.tb.q;
    if (segment_of_local) *segment_of_local = c->rs_gidx;
    return CDADAM_OK;
}

int cdadam_range_topk(cdadam_ctx *c, int stage, const float *grads, void *stream)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_range_topk: NULL context");
    if (!c->is_range || c->comp != CDADAM_TOPK) return fail(CDADAM_ERR_STATE, "cdadam_range_topk: the context was not made by cdadam_create_range with CDADAM_TOPK");
    if (c->mode != CDADAM_MARKOV) return fail(CDADAM_ERR_STATE, "cdadam_range_topk: Algorithm 1 only");
    if (stage < 0 || stage > 9) return fail(CDADAM_ERR_ARG, "cdadam_range_topk: stages are 0..9");
    if (stage != c->phase) return fail(CDADAM_ERR_STATE, "cdadam_range_topk: stage %d is next", c->phase);
    if (stage <= 4 && !grads) return fail(CDADAM_ERR_ARG, "cdadam_range_topk: the worker stages 0..4 take the gradients");
    if (c->prof_on) return fail(CDADAM_ERR_STATE, "cdadam_range_topk: per-stage timing covers cdadam_step only");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = refuse_capture(st)) return rc;
    if (stage == 0) step_size_of_this_step(c);
    const bool svec = c->d % 4 == 0;
    if (stage <= 4) {                                  // workers: c^(i) = C(g^(i) - ghat^(i)); ghat^(i) += c^(i)
        topk_range_stage(c->tk_w, stage, grads, c->ghat_w, aligned16(grads) && svec, c->range_k, c->rx_w,
                         c->range_rank, c->range_count, st);
    } else {                                           // server: ghat += mean; c = C(ghat - gtil); gtil += c
        if (stage == 5) {
            const uint32_t *widx; const float *wval;
            topk_payload(c->tk_w, 0, &widx, &wval);
            topk_aggregate_rows(widx, wval, c->k, c->d, c->n, c->ghat_s, st);
        }
        topk_range_stage(c->tk_s, stage - 5, c->ghat_s, c->gtil, svec, c->range_k, c->rx_s, c->range_rank,
                         c->range_count, st);
        if (stage == 9) launch_amsgrad(c->gtil, c->m, c->v, c->vhat, c->x, c->d, c->hp, svec, st);
    }
    if (int rc = check_launch("cdadam_range_topk")) return rc;
    c->phase = stage == 9 ? 0 : stage + 1;
    if (stage == 9) c->steps += 1;
    return CDADAM_OK;
}

int cdadam_range_topk_buffer(cdadam_ctx *c, int stage, uint32_t **buffer, int64_t *words_per_range)
{
    if (!c || !buffer || !words_per_range) return fail(CDADAM_ERR_ARG, "cdadam_range_topk_buffer: NULL argument");
    if (!c->is_range || c->comp != CDADAM_TOPK) return fail(CDADAM_ERR_STATE, "cdadam_range_topk_buffer: the context was not made by cdadam_create_range with CDADAM_TOPK");
    if (stage < 0 || stage > 9) return fail(CDADAM_ERR_ARG, "cdadam_range_topk_buffer: stages are 0..9");
    const int64_t per = topk_range_exchange_words(c->tk_s);
    if (stage == 4 || stage == 9) { *buffer = nullptr; *words_per_range = 0; }      // nothing to exchange after these
    else if (stage < 4) { *buffer = c->rx_w; *words_per_range = (int64_t)c->n * per; }
    else { *buffer = c->rx_s; *words_per_range = per; }
    return CDADAM_OK;
}

int cdadam_step_bf16(cdadam_ctx *c, const void *grads, void *stream) { return step_impl(c, grads, true, stream); }

int cdadam_step_host(cdadam_ctx *c, const float *grads_host, float *x_out_host, void *stream)
{
    if (!c || !grads_host) return fail(CDADAM_ERR_ARG, "cdadam_step_host: NULL argument");
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (c->nloc != c->n || c->is_range) return fail(CDADAM_ERR_STATE, "cdadam_step_host: this context holds a part of the workers or coordinates; use the staged calls");
    const size_t bytes = (size_t)c->n * c->d * sizeof(float);
    int rc0 = ensure_stage(c);
    if (rc0) return rc0;
    CU_TRY(cudaMemcpyAsync(c->stage, grads_host, bytes, cudaMemcpyHostToDevice, st));
    int rc = cdadam_step(c, c->stage, stream);
    if (rc) return rc;
    if (x_out_host)
        CU_TRY(cudaMemcpyAsync(x_out_host, c->x, (size_t)c->d * sizeof(float), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    return CDADAM_OK;
}

const float *cdadam_params(cdadam_ctx *c) { return c ? c->x : nullptr; }

int cdadam_set_params(cdadam_ctx *c, const float *x0, void *stream)
{
    return cdadam_set_state(c, CDADAM_STATE_X, x0, stream);
}

int cdadam_set_topk_segments(cdadam_ctx *c, int q, const int64_t *offsets, const int64_t *k_per_segment)
{
    if (!c || !offsets || !k_per_segment) return fail(CDADAM_ERR_ARG, "cdadam_set_topk_segments: NULL argument");
    if (c->comp != CDADAM_TOPK) return fail(CDADAM_ERR_STATE, "top-k segments apply to the top-k compressor only");
    if (c->is_range) return fail(CDADAM_ERR_STATE, "top-k segments are not available on a coordinate range");
    if (c->mode != CDADAM_MARKOV) return fail(CDADAM_ERR_STATE, "top-k segments are available for Algorithm 1 only");
    if (c->steps != 0 || c->phase != 0) return fail(CDADAM_ERR_STATE, "segments must be set before the first step");
    if (q < 1 || (int64_t)q > c->d) return fail(CDADAM_ERR_ARG, "q must be in [1, d]");
    if (offsets[0] != 0 || offsets[q] != c->d) return fail(CDADAM_ERR_ARG, "offsets must start at 0 and end at d");
    int64_t total = 0;
    for (int r = 0; r < q; ++r) {
        if (offsets[r + 1] <= offsets[r]) return fail(CDADAM_ERR_ARG, "offsets must be strictly increasing (segment %d)", r);
        if (k_per_segment[r] < 1 || k_per_segment[r] > offsets[r + 1] - offsets[r])
            return fail(CDADAM_ERR_ARG, "segment %d: k must be in [1, segment length]", r);
        total += k_per_segment[r];
    }
    DeviceGuard guard(c->device);
    CU_TRY(cudaDeviceSynchronize());
    topk_workspace_destroy(c->tk_w); topk_workspace_destroy(c->tk_s);
    c->tk_w = c->tk_s = nullptr;
    for (TopkWorkspace *w : c->seg_w) topk_workspace_destroy(w);
    for (TopkWorkspace *w : c->seg_s) topk_workspace_destroy(w);
    c->seg_w.clear(); c->seg_s.clear(); c->seg_off.clear(); c->seg_k.clear(); c->seg_at.clear();
    c->k = total;
    int rc;
    if ((rc = topk_workspace_create(&c->tk_w, c->d, total, c->n, nullptr, nullptr, false)) ||
        (rc = topk_workspace_create(&c->tk_s, c->d, total, 1, nullptr, nullptr, false)))
        return fail(rc, "top-k payload allocation failed");
    int64_t at = 0;
    for (int r = 0; r < q; ++r) {
        const int64_t len = offsets[r + 1] - offsets[r];
        TopkWorkspace *ww = nullptr, *ws = nullptr;
        if ((rc = topk_workspace_create(&ww, len, k_per_segment[r], c->n, nullptr, nullptr, true, c->d)) ||
            (rc = topk_workspace_create(&ws, len, k_per_segment[r], 1, nullptr, nullptr, true, c->d))) {
            topk_workspace_destroy(ww);
            return fail(rc, "top-k workspace allocation failed (segment %d)", r);
        }
        topk_workspace_set_error_flag(ww, c->error_flag);
        topk_workspace_set_error_flag(ws, c->error_flag);
        c->seg_w.push_back(ww); c->seg_s.push_back(ws);
        c->seg_off.push_back(offsets[r]); c->seg_k.push_back(k_per_segment[r]); c->seg_at.push_back(at);
        at += k_per_segment[r];
    }
    drop_graphs(c);
    return CDADAM_OK;
}

int cdadam_set_segments(cdadam_ctx *c, int q, const int64_t *offsets)
{
    if (!c || !offsets) return fail(CDADAM_ERR_ARG, "cdadam_set_segments: NULL argument");
    if (c->comp != CDADAM_SIGN) return fail(CDADAM_ERR_STATE, "segments apply to the scaled-sign compressor only");
    if (c->steps != 0 || c->phase != 0) return fail(CDADAM_ERR_STATE, "segments must be set before the first step");
    const int64_t dim = c->is_range ? c->range_dim : c->d;
    if (q < 1 || (int64_t)q > dim) return fail(CDADAM_ERR_ARG, "q must be in [1, d]");
    if (offsets[0] != 0 || offsets[q] != dim) return fail(CDADAM_ERR_ARG, "offsets must start at 0 and end at d");
    for (int r = 0; r < q; ++r)
        if (offsets[r + 1] <= offsets[r]) return fail(CDADAM_ERR_ARG, "offsets must be strictly increasing (segment %d)", r);
    DeviceGuard guard(c->device);
    CU_TRY(cudaDeviceSynchronize());
    std::vector<int64_t> local;
    std::vector<int32_t> gidx;
    std::vector<int64_t> glen;
    const int q_all = q;
    if (c->is_range) {             // the whole problem's segments, cut to this context's coordinates
        c->range_off_all.assign(offsets, offsets + q + 1);
        cut_segments(c, q, offsets, local, gidx, glen);
        q = (int)gidx.size();
        offsets = local.data();
    }
    int rc = c->ts.build(c->d, q, offsets, c->tile_override ? c->tile_override : choose_tile(c->d, q, false), nullptr, false);
    if (rc) return rc;
    rc = c->ts_s.build(c->d, q, offsets, c->tile_override ? c->tile_override : choose_tile(c->d, q, true), nullptr, false);
    if (rc) return rc;
    if ((rc = alloc_sign_buffers(c))) return rc;
    return c->is_range ? alloc_range_buffers(c, q_all, gidx, glen) : CDADAM_OK;
}

int cdadam_set_tile(cdadam_ctx *c, int tile)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_set_tile: NULL context");
    if (c->comp != CDADAM_SIGN && c->comp != CDADAM_TOPK)
        return fail(CDADAM_ERR_STATE, "tiles apply to the scaled-sign and top-k compressors only");
    if (c->steps != 0 || c->phase != 0) return fail(CDADAM_ERR_STATE, "the tile size must be set before the first step");
    if (tile != 0 && (tile < kSub || tile % kSub != 0 || tile > 64 * kSub))
        return fail(CDADAM_ERR_ARG, "tile must be 0 or a multiple of %d up to %d", kSub, 64 * kSub);
    if (c->comp == CDADAM_TOPK) {
        // the selection works on 4096-coordinate tiles throughout; the knob only picks the
        // kernel of the dense pass
        const int ring = tile == 0 ? 0 : tile >= 4 * kSub ? 1 : -1;
        topk_workspace_set_ring(c->tk_w, ring);
        topk_workspace_set_ring(c->tk_s, ring);
        for (TopkWorkspace *w : c->seg_w) topk_workspace_set_ring(w, ring);
        for (TopkWorkspace *w : c->seg_s) topk_workspace_set_ring(w, ring);
        return CDADAM_OK;
    }
    c->tile_override = tile;
    std::vector<int64_t> off = c->is_range ? c->range_off_all : c->ts.off;   // rebuild the tables for the current segments
    return cdadam_set_segments(c, (int)off.size() - 1, off.data());
}

int cdadam_set_wait_limit(cdadam_ctx *c, int polls)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_set_wait_limit: NULL context");
    c->wait_limit = polls < 0 ? -1 : polls;
    topk_workspace_set_wait_limit(c->tk_w, polls);
    topk_workspace_set_wait_limit(c->tk_s, polls);
    for (TopkWorkspace *w : c->seg_w) topk_workspace_set_wait_limit(w, polls);
    for (TopkWorkspace *w : c->seg_s) topk_workspace_set_wait_limit(w, polls);
    drop_graphs(c);                            // the limit is a launch argument
    return CDADAM_OK;
}

int cdadam_set_random_sets(cdadam_ctx *c, const uint32_t *workers, const uint32_t *server, void *stream)
{
    if (!c || !workers || !server) return fail(CDADAM_ERR_ARG, "cdadam_set_random_sets: NULL argument");
    if (c->comp != CDADAM_RANDK) return fail(CDADAM_ERR_STATE, "random sets apply to the rand-k compressor only");
    DeviceGuard guard(c->device);
    randk_set(c->tk_w, workers, c->error_flag, (cudaStream_t)stream);
    randk_set(c->tk_s, server, c->error_flag, (cudaStream_t)stream);
    c->sets_given = true;
    return check_launch("cdadam_set_random_sets");
}

int cdadam_set_mode(cdadam_ctx *c, int mode)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_set_mode: NULL context");
    if (mode != CDADAM_MARKOV && mode != CDADAM_EF && mode != CDADAM_NAIVE) return fail(CDADAM_ERR_ARG, "unknown mode %d", mode);
    if (mode != CDADAM_MARKOV && !c->seg_w.empty()) return fail(CDADAM_ERR_STATE, "top-k segments are available for Algorithm 1 only");
    if (c->steps != 0 || c->phase != 0) return fail(CDADAM_ERR_STATE, "the mode must be set before the first step");
    c->mode = mode;
    return CDADAM_OK;
}

int cdadam_set_lr(cdadam_ctx *c, float lr)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_set_lr: NULL context");
    c->milestones.clear();                    // an explicit step size ends a schedule
    apply_lr(c, lr);
    return CDADAM_OK;
}

int cdadam_set_weight_decay(cdadam_ctx *c, float lambda)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_set_weight_decay: NULL context");
    if (!(lambda >= 0.0f)) return fail(CDADAM_ERR_ARG, "the weight decay must be >= 0");
    c->wd = lambda;
    apply_lr(c, c->hp.lr);
    return CDADAM_OK;
}

int cdadam_set_lr_milestones(cdadam_ctx *c, float base_lr, int count, const int64_t *after_steps, float gamma)
{
    if (!c || (count > 0 && !after_steps)) return fail(CDADAM_ERR_ARG, "cdadam_set_lr_milestones: NULL argument");
    if (count < 0 || count > 64) return fail(CDADAM_ERR_ARG, "between 0 and 64 milestones");
    if (!(gamma > 0.0f && gamma <= 1.0f)) return fail(CDADAM_ERR_ARG, "gamma must be in (0, 1]: the step sizes of Algorithm 1 do not increase");
    for (int i = 0; i < count; ++i)
        if (after_steps[i] < 0 || (i > 0 && after_steps[i] <= after_steps[i - 1]))
            return fail(CDADAM_ERR_ARG, "milestones must be non-negative and increasing");
    c->base_lr = base_lr;
    c->gamma = gamma;
    c->milestones.assign(after_steps, after_steps + count);
    if (count == 0) apply_lr(c, base_lr);
    return CDADAM_OK;
}

int cdadam_get_state(cdadam_ctx *c, int name, float *dst, void *stream)
{
    if (!c || !dst) return fail(CDADAM_ERR_ARG, "cdadam_get_state: NULL argument");
    float *src = state_ptr(c, name);
    if (!src) return fail(CDADAM_ERR_ARG, "unknown state name %d", name);
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (name == CDADAM_STATE_GHAT_W && c->is_range && c->phase == 1)
        return fail(CDADAM_ERR_STATE, "cdadam_get_state: the scales of this iteration's worker messages are known after cdadam_range_server");
    if (name == CDADAM_STATE_GHAT_W && c->comp == CDADAM_SIGN && c->pending) {
        if (c->nloc > 0)
            launch_apply_sign(c->ghat_w, c->wbits + (int64_t)c->first * c->wp, c->wscale[c->cur] + (int64_t)c->first * c->ts.tb.q,
                              c->ts.tb, c->nloc, c->wp, c->mode == CDADAM_EF, st);
        int rc = check_launch("apply deferred payload");
        if (rc) return rc;
        c->pending = false;
    }
    if (name == CDADAM_STATE_GHAT_W && c->comp == CDADAM_TOPK && c->tk_w && c->nloc > 0) {
        topk_flush(c->tk_w, c->ghat_w, st);              // the last worker messages, if still to be applied
        int rc = check_launch("apply deferred payload");
        if (rc) return rc;
    }
    const size_t count = name == CDADAM_STATE_GHAT_W ? (size_t)c->nloc * c->d : (size_t)c->d;
    CU_TRY(cudaMemcpyAsync(dst, src, count * sizeof(float), cudaMemcpyDeviceToDevice, st));
    return CDADAM_OK;
}

int cdadam_set_state(cdadam_ctx *c, int name, const float *src, void *stream)
{
    if (!c || !src) return fail(CDADAM_ERR_ARG, "cdadam_set_state: NULL argument");
    float *dst = state_ptr(c, name);
    if (!dst) return fail(CDADAM_ERR_ARG, "unknown state name %d", name);
    DeviceGuard guard(c->device);
    const size_t count = name == CDADAM_STATE_GHAT_W ? (size_t)c->nloc * c->d : (size_t)c->d;
    CU_TRY(cudaMemcpyAsync(dst, src, count * sizeof(float), cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    if (name == CDADAM_STATE_GHAT_W) {                     // the given values are final
        c->pending = false;
        if (c->comp == CDADAM_TOPK) topk_forget_pending(c->tk_w, (cudaStream_t)stream);
    }
    return CDADAM_OK;
}

int cdadam_last_payload(cdadam_ctx *c, int who, const void **a, const float **b, int64_t *count)
{
    if (!c || !a || !b || !count) return fail(CDADAM_ERR_ARG, "cdadam_last_payload: NULL argument");
    if (who != CDADAM_SERVER && (who < 0 || who >= c->n)) return fail(CDADAM_ERR_ARG, "who out of range");
    if (c->steps == 0) return fail(CDADAM_ERR_STATE, "no step has run yet");
    if (c->comp == CDADAM_SIGN) {
        if (who == CDADAM_SERVER) { *a = c->sbits; *b = c->sscale; }
        else { *a = c->wbits + (int64_t)who * c->wp; *b = c->wscale[c->cur] + (int64_t)who * c->ts.tb.q; }
        *count = c->d;
        return CDADAM_OK;
    }
    if (c->comp == CDADAM_TOPK || c->comp == CDADAM_RANDK) {
        if (who != CDADAM_SERVER && c->pay_idx) {
            *a = c->pay_idx + (int64_t)who * c->k; *b = c->pay_val + (int64_t)who * c->k;
        } else {
            TopkWorkspace *w = who == CDADAM_SERVER ? c->tk_s : c->tk_w;
            topk_payload(w, who == CDADAM_SERVER ? 0 : who, (const uint32_t **)a, b);
        }
        *count = c->k;
        return CDADAM_OK;
    }
    return fail(CDADAM_ERR_STATE, "the identity compressor sends no payload");
}

int64_t cdadam_step_count(cdadam_ctx *c) { return c ? c->steps : 0; }

int cdadam_set_step_count(cdadam_ctx *c, int64_t t)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_set_step_count: NULL context");
    if (t < 0) return fail(CDADAM_ERR_ARG, "the iteration counter cannot be negative");
    if (c->phase != 0) return fail(CDADAM_ERR_STATE, "cdadam_set_step_count: a staged iteration is under way");
    c->steps = t;
    return CDADAM_OK;
}

int cdadam_device_status(cdadam_ctx *c, void *stream)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_device_status: NULL context");
    DeviceGuard guard(c->device);
    int flag = 0;
    CU_TRY(cudaMemcpyAsync(&flag, c->error_flag, sizeof flag, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (flag == 2) return fail(CDADAM_ERR_ARG, "a rand-k coordinate set was not strictly increasing or had a coordinate >= d; the state is not valid");
    if (flag) {
        c->void_state = true;
        return fail(CDADAM_ERR_TIMEOUT, "a kernel gave up waiting for an asynchronous copy; the state is not valid");
    }
    return CDADAM_OK;
}

int cdadam_launches_per_step(cdadam_ctx *c)
{
    if (!c) return 0;
    if (c->is_range && c->comp == CDADAM_TOPK) return 46;    // two staged selections of 22, aggregation, AMSGrad
    if (c->is_range) return 7;      // worker pass, sums | scales, server pass, sums | scales, update
    if (c->comp == CDADAM_SIGN) return c->fuse_finish && c->mode != CDADAM_NAIVE ? 3 : 5;
    if (c->comp == CDADAM_TOPK && !c->seg_w.empty())     // per segment: two selections and two payload copies
        return (int)c->seg_w.size() * (topk_launches_per_step(c->n) + 2) + 2;
    if (c->comp == CDADAM_TOPK) {   // (for gradient rows that are 16-byte aligned)
        // Algorithm 1: two selections (the server's with the aggregation inside its dense pass,
        // which is then one plain kernel) and AMSGrad; the comparison modes: a separate
        // aggregation kernel and their dense helpers
        const int workers_dense = topk_dense_launches(c->tk_w, c->d % 4 == 0) - 1;
        if (c->mode == CDADAM_MARKOV) return topk_launches_per_step(c->n) + 1 + workers_dense;
        return topk_launches_per_step(c->n) + 2 + (c->mode == CDADAM_EF ? 5 : 3) + workers_dense +
               topk_dense_launches(c->tk_s, c->d % 4 == 0) - 1;
    }
    if (c->comp == CDADAM_RANDK) return c->mode == CDADAM_EF ? 9 : c->mode == CDADAM_NAIVE ? 7 : 4;
    return 1;
}

int cdadam_profile_enable(cdadam_ctx *c, int on)
{
    if (!c) return fail(CDADAM_ERR_ARG, "cdadam_profile_enable: NULL context");
    c->prof_on = on != 0;
    return CDADAM_OK;
}

int cdadam_profile_read(cdadam_ctx *c, double *ms, int64_t *steps)
{
    if (!c || !ms || !steps) return fail(CDADAM_ERR_ARG, "cdadam_profile_read: NULL argument");
    DeviceGuard guard(c->device);
    const int ns = prof_slots(c), group = ns + 1;
    for (int s = 0; s < CDADAM_PROF_SLOTS; ++s) ms[s] = 0.0;
    *steps = (int64_t)(c->prof_ev.size() / group);
    if (!c->prof_ev.empty()) CU_TRY(cudaEventSynchronize(c->prof_ev.back()));
    for (int64_t t = 0; t < *steps; ++t)
        for (int s = 0; s < ns; ++s) {
            float f = 0.0f;
            CU_TRY(cudaEventElapsedTime(&f, c->prof_ev[t * group + s], c->prof_ev[t * group + s + 1]));
            ms[s] += f;
        }
    c->prof_pool.insert(c->prof_pool.end(), c->prof_ev.begin(), c->prof_ev.end());
    c->prof_ev.clear();
    return CDADAM_OK;
}

const char *cdadam_profile_name(cdadam_ctx *c, int slot)
{
    static const char *sign[] = {"k_worker_sign", "k_finalize_scales(workers)", "k_server_sign",
                                 "k_finalize_scales(server)", "k_update_sign"};
    if (c && c->comp == CDADAM_SIGN && slot == 0 && c->ts.tb.tile >= 4 * kSub && c->d % 4 == 0)
        return "k_worker_sign_ring";
    static const char *fused[] = {"k_worker_sign", "k_server_sign", "k_update_sign"};
    static const char *topk[] = {"topk_select(workers)", "topk_aggregate", "topk_select(server)", "k_amsgrad"};
    if (!c || slot < 0 || slot >= prof_slots(c)) return "";
    static const char *randk[] = {"randk_gather(workers)", "topk_aggregate", "randk_gather(server)", "k_amsgrad"};
    if (c->comp == CDADAM_RANDK) return randk[slot];
    static const char *nsign[] = {"k_pack_sign", "k_finalize_scales(workers)", "k_server_sign",
                                  "k_finalize_scales(server)", "k_update_sign"};
    if (c->comp == CDADAM_SIGN && c->mode == CDADAM_NAIVE) return nsign[slot];
    return c->comp == CDADAM_SIGN ? (c->fuse_finish ? fused[slot] : sign[slot]) : c->comp == CDADAM_TOPK ? topk[slot] : "k_step_identity";
}

int cdadam_compress_sign(const float *x, int64_t d, int q, const int64_t *offsets, uint32_t *bits,
                         float *scales, void *stream)
{
    if (!x || !bits || !scales) return fail(CDADAM_ERR_ARG, "cdadam_compress_sign: NULL argument");
    if (d < 1 || d >= ((int64_t)1 << 32)) return fail(CDADAM_ERR_ARG, "d must be in [1, 2^32)");
    const int64_t flat[2] = {0, d};
    if (!offsets) { offsets = flat; q = 1; }
    if (q < 1 || (int64_t)q > d || offsets[0] != 0 || offsets[q] != d) return fail(CDADAM_ERR_ARG, "bad segment offsets");
    for (int r = 0; r < q; ++r)
        if (offsets[r + 1] <= offsets[r]) return fail(CDADAM_ERR_ARG, "offsets must be strictly increasing");
    cudaStream_t st = (cudaStream_t)stream;
    TableSet ts;
    int rc = ts.build(d, q, offsets, choose_tile(d, q, false), st, true);
    if (rc) return rc;
    dd *part = nullptr;
    cudaError_t e = cudaMallocAsync((void **)&part, (size_t)ts.tb.nparts * sizeof(dd), st);
    if (e != cudaSuccess) { ts.release(st, true); return fail(CDADAM_ERR_ALLOC, "scratch allocation: %s", cudaGetErrorString(e)); }
    launch_pack_sign(x, bits, part, ts.tb, 1, (d + 31) / 32, aligned16(x) && d % 4 == 0, st);
    launch_finalize_scales(part, scales, ts.tb, 1, st);
    rc = check_launch("cdadam_compress_sign");
    cudaFreeAsync(part, st);
    ts.release(st, true);
    return rc;
}

int cdadam_compress_topk(const float *x, int64_t d, int64_t k, uint32_t *idx, float *val, void *stream)
{
    if (!x || !idx || !val) return fail(CDADAM_ERR_ARG, "cdadam_compress_topk: NULL argument");
    if (d < 1 || d >= ((int64_t)1 << 32) || k < 1 || k > d) return fail(CDADAM_ERR_ARG, "need 1 <= k <= d < 2^32");
    int rc = topk_compress(x, d, k, idx, val, (cudaStream_t)stream);
    if (rc) return fail(rc, "cdadam_compress_topk failed");
    return check_launch("cdadam_compress_topk");
}

}  // extern "C"
