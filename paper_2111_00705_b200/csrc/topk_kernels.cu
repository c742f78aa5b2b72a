// Top-k compressor (Appendix A: keep the k coordinates of largest magnitude) for sm_100a.
//
// Exact selection without sorting: the magnitude bits key = bits(|u|) (31 bits; for finite
// floats integer order = value order) are resolved by a three-level radix select,
//   level 1: key bits 30..20, histogram over a dense pass;
//   level 2: key bits 19..9 and level 3: key bits 8..0, histograms over the candidates only
// which yields the exact k-th largest key T.  Coordinates with key > T are kept; among those
// with key == T the ones of lowest index are kept until k is reached.  The selection lives in
// bitmaps (1 bit per coordinate), so the ordered compaction (index-increasing payload) costs
// d/8 bytes per pass instead of another pass over the data.  All counters are integer
// atomics: the result does not depend on the order of execution.
//
// Normally ONE dense pass suffices: the level-1 bucket of the previous selection, lowered by
// a margin, serves as a floor; the pass histograms only the coordinates at or above it, in
// bins of 2^11 keys counted from the floor (four level-1 buckets wide, the last bin open), and
// keeps them per 4096-coordinate tile as a short list (position in the tile, value) in index
// order.  The histogram fixes key bits 30..11 of the threshold; one pass over the lists
// (bits 10..0) fixes the rest: two levels instead of three.  Every later pass of such a row
// walks these lists, one warp per tile, with coalesced reads: k_topk_split (low-bits histogram
// and per-tile candidate records), k_scan_lists (exact threshold, per-tile counts, tie ranks
// and payload offsets, one block per row) and k_topk_emit_idx (ordered compaction with the
// values), without bitmaps.  A tile with more coordinates above the floor than its list holds
// (a selection concentrated in one tensor) is read again from the data by those passes.  If
// fewer than k coordinates lie above the floor, or the threshold lies above the fine bins,
// the classic two dense passes and the bitmap passes run instead, as a second chain of
// launches beside the first.  The state update b += u at the kept coordinates is part of the
// compaction, or, for rows selected from lists of a workspace that defers it, of the next
// selection's dense pass (one streaming pass instead of k random read-modify-writes per row).
// The server's aggregation of the workers' messages runs inside the dense pass of the server's
// selection.  The same file holds the separate sparse aggregation kernel, the rand-k path,
// which shares the payload kernels, and the staged selection over coordinate ranges.
#include "topk.h"

#include <algorithm>
#include <cstring>

#include "../../include/cdadam.h"
#include "common.cuh"

namespace cdadam {

constexpr uint32_t kFull = 0xffffffffu;
constexpr int kBins1 = 2048, kBins2 = 2048, kBins3 = 512;
constexpr int kHistStride = kBins1 + kBins2 + kBins3;
constexpr int kTileWords = 1024;      // bitmap words per block in the sparse passes
constexpr int kStashCap = 512;        // values kept per 4096-coordinate tile by the dense pass
constexpr uint32_t kGuessMargin = 1;  // level-1 buckets (1/8 octave each) kept below the last threshold bucket

struct Sel {                          // outcome of the three levels for one row
    uint32_t b1, k1, c1;              // bucket, entries still to take inside it, its size
    uint32_t b2, k2, c2;
    uint32_t b3, k3, c3;              // T = b1<<20 | b2<<9 | b3; take k3 of the c3 ties
    uint32_t pre;                     // rows whose guess held: key bits 30..11 of T (bits 10..0 zero)
    uint32_t pad[2];
};

struct TopkWorkspace {
    int64_t d, k, wp, nbt;
    int64_t stride;                   // elements between the rows of a and b (>= d)
    int rows;
    uint32_t *hist;                   // rows x kHistStride
    Sel *sel;                         // rows
    uint32_t *bm_in, *bm_cand;        // rows x wp (rows whose guess failed)
    uint32_t *floor_bucket;           // rows: guessed level-1 bucket for the next selection
    uint32_t *hit;                    // rows: 1 if the guess held in the current selection
    // lists of the coordinates at or above the guessed bucket, per 4096-coordinate tile:
    float *stash;                     // rows x nt4k x kStashCap: values u, in index order
    uint16_t *stash_pos;              // rows x nt4k x kStashCap: positions inside the tile
    uint32_t *stash_cnt;              // rows x nt4k: list lengths; above kStashCap the tile kept no
                                      // complete list and the later passes read it from a and b
    uint16_t *cand;                   // rows x nt4k x 4: low key bits of a tile's first candidates (k_topk_split)
    uint32_t *cnt_gt, *cnt_eq;        // rows x nt4k: per tile, keys above / equal to the threshold;
                                      // after the scans: payload offset / tie rank of the tile
    int64_t nt4k;                     // ceil(d / 4096)
    uint32_t *cnt_tie, *cnt_fin;      // rows x nbt
    uint32_t *idx;                    // rows x k
    float *val;                       // rows x k
    bool own_payload;
    int *error_flag;                  // device word set by a kernel whose bounded wait ran out (may be NULL)
    int ring;                         // dense pass with the prefetch ring: 0 = by size, 1 = wherever rows are aligned, -1 = never
    int wait_limit;                   // polls before a wait on an asynchronous copy gives up
    // Deferred state update (topk_workspace_set_defer): rows selected from lists do not get
    // b += u at the kept coordinates at once; the next selection's dense pass, which has the
    // tile of b in hand anyway, applies the previous payload first (pending[row] = 1 until
    // then).  topk_flush applies what is pending.
    bool defer;
    uint32_t *pending;                // rows
    // the chain of kernels for the rows whose guess failed runs beside the chain for the rows
    // selected from lists: a second stream, forked and joined with events inside topk_select
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join;
    unsigned int *tick;               // 5 x rows ticket counters of that chain's passes (zero between uses)
};

__device__ __forceinline__ uint32_t key_of(float u) { return __float_as_uint(u) & 0x7fffffffu; }

template <bool HAS_B>
__device__ __forceinline__ float diff1(const float *a, const float *b, int64_t j)
{
    return HAS_B ? __fsub_rn(a[j], b[j]) : a[j];
}

// exclusive prefix sum over the NT threads of a block; all threads must call
template <int NT>
__device__ __forceinline__ uint32_t block_excl_scan_n(uint32_t v, uint32_t &total)
{
    __shared__ uint32_t ws[NT / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) ws[warp] = inc;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) {
        const uint32_t s = ws[w];
        if (w < warp) before += s;
        all += s;
    }
    total = all;
    return before + inc - v;
}
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t &total) { return block_excl_scan_n<kBlock>(v, total); }

// ------------------------------------------------------------------------------------
// Pick the bucket that holds the `want`-th largest entry of a row's histogram: the bucket b
// with count(bins > b) < want <= count(bins >= b).  Run by one whole block for the row.
// level 0/1/2 selects which histogram and which fields of Sel are read and written.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ void pick_row(const uint32_t *hist_row, Sel *sel, int level, uint32_t k,
                                         uint32_t *floor_bucket_row)
{
    __shared__ uint32_t tot[kBlock];
    const int nb = level == 2 ? kBins3 : kBins1;
    const uint32_t *hist = hist_row + (level == 0 ? 0 : level == 1 ? kBins1 : kBins1 + kBins2);
    const uint32_t want = level == 0 ? k : level == 1 ? sel->k1 : sel->k2;
    const int per = nb / kBlock;                    // 8 or 2 contiguous bins per thread
    const int lo = threadIdx.x * per;
    uint32_t mine = 0;
    for (int t = 0; t < per; ++t) mine += __ldcg(hist + lo + t);
    __syncthreads();                                // tot may still be read by an earlier call
    tot[threadIdx.x] = mine;
    __syncthreads();
    uint32_t above = 0;                             // entries in bins owned by later threads
    for (int t = threadIdx.x + 1; t < kBlock; ++t) above += tot[t];
    for (int t = per - 1; t >= 0; --t) {
        const uint32_t c = __ldcg(hist + lo + t);
        if (above < want && above + c >= want) {
            const uint32_t bucket = lo + t, rem = want - above;
            if (level == 0) { sel->b1 = bucket; sel->k1 = rem; sel->c1 = c; }
            else if (level == 1) { sel->b2 = bucket; sel->k2 = rem; sel->c2 = c; }
            else {
                sel->b3 = bucket; sel->k3 = rem; sel->c3 = c;
                // guess for the next selection of this row: below this threshold, one bucket
                // more than after a guess that held
                *floor_bucket_row = sel->b1 > kGuessMargin + 1u ? sel->b1 - (kGuessMargin + 1u) : 1u;
            }
        }
        above += c;
    }
}

// True, for all threads of the block, in the block that is the last of `count` blocks to get
// here (the others' global writes before their call are then visible to it).  The counter
// goes back to zero.  No block waits for another.  Used by the passes of the rows whose guess
// failed, so that a row's pick or scan needs no launch of its own; those passes are rare and
// short of memory traffic, so the fence costs nothing that matters (in the dense pass of the
// common path it did: see pick_spec_row).
__device__ __forceinline__ bool last_block_of_row(unsigned int *counter, unsigned int count)
{
    __shared__ int s_is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        s_is_last = atomicAdd(counter, 1u) == count - 1u;
        if (s_is_last) *counter = 0u;
    }
    __syncthreads();
    const bool last = s_is_last != 0;
    if (last) __threadfence();
    return last;
}

// Exclusive scan of a row's nbt counts (in place, or only the total), by one whole block.
__device__ __forceinline__ void scan_row(uint32_t *cnt, int64_t nbt, uint32_t *total_out, bool in_place)
{
    uint32_t carry = 0;
    for (int64_t c = 0; c < nbt; c += kBlock) {
        const int64_t t = c + threadIdx.x;
        const uint32_t v = t < nbt ? __ldcg(cnt + t) : 0u;
        uint32_t total;
        const uint32_t ex = block_excl_scan(v, total);
        if (in_place && t < nbt) cnt[t] = carry + ex;
        carry += total;
    }
    if (total_out && threadIdx.x == 0) *total_out = carry;           // the row's sum (block-uniform)
}

// Tail of the classic passes when they run as one chain of launches (topk_select): what a
// row needs next is done by the block that finishes the row last.  tick == NULL: no tail
// (the coordinate-sharded selection picks after the histograms have been exchanged).
struct RowTail {
    unsigned int *tick;               // rows counters of this pass, or NULL
    Sel *sel;
    uint32_t *floor_bucket;
    uint32_t k;
};

// ------------------------------------------------------------------------------------
// Level 1: histogram of key >> 20 over all coordinates.  grid = (ceil(d/4096), rows).
// ------------------------------------------------------------------------------------
template <bool HAS_B>
__global__ void __launch_bounds__(kBlock)
k_topk_hist1(const float *__restrict__ a_all, const float *__restrict__ b_all,
             uint32_t *__restrict__ hist_all, const uint32_t *__restrict__ hit, int64_t d, int vec_ok, int64_t stride,
             RowTail tail)
{
    __shared__ uint32_t h[kBins1];
    if (hit[blockIdx.y]) return;                      // the guessed bucket held: nothing to redo
    for (int t = threadIdx.x; t < kBins1; t += kBlock) h[t] = 0;
    __syncthreads();
    const int row = blockIdx.y;
    const float *a = a_all + (int64_t)row * stride;
    const float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // blocks loop over tiles: the grid is small, so rows whose guess held cost almost nothing
    for (int64_t base = (int64_t)blockIdx.x * kSub; base < d; base += (int64_t)gridDim.x * kSub) {
        if (vec_ok && base + kSub <= d) {
            const int64_t wb = base + warp * kWarpSpan;
            float4 A[4], Bv[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int64_t j = wb + v * 128 + lane * 4;
                A[v] = ld_ro4(a + j);
                if (HAS_B) Bv[v] = ld_ro4(b + j);
            }
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                if (HAS_B) {
                    A[v].x = __fsub_rn(A[v].x, Bv[v].x); A[v].y = __fsub_rn(A[v].y, Bv[v].y);
                    A[v].z = __fsub_rn(A[v].z, Bv[v].z); A[v].w = __fsub_rn(A[v].w, Bv[v].w);
                }
                atomicAdd(&h[key_of(A[v].x) >> 20], 1u);
                atomicAdd(&h[key_of(A[v].y) >> 20], 1u);
                atomicAdd(&h[key_of(A[v].z) >> 20], 1u);
                atomicAdd(&h[key_of(A[v].w) >> 20], 1u);
            }
        } else {
            const int64_t end = min(base + (int64_t)kSub, d);
            for (int64_t j = base + threadIdx.x; j < end; j += kBlock)
                atomicAdd(&h[key_of(diff1<HAS_B>(a, b, j)) >> 20], 1u);
        }
    }
    __syncthreads();
    uint32_t *hist = hist_all + (int64_t)row * kHistStride;
    for (int t = threadIdx.x; t < kBins1; t += kBlock)
        if (h[t]) atomicAdd(&hist[t], h[t]);
    if (tail.tick && last_block_of_row(tail.tick + row, gridDim.x))
        pick_row(hist, tail.sel + row, 0, tail.k, tail.floor_bucket + row);
}

// ------------------------------------------------------------------------------------
// Pick the bucket that holds the `want`-th largest entry of a histogram: the bucket b with
// count(bins > b) < want <= count(bins >= b).  grid = (rows), one block.
// level 0/1/2 selects which histogram and which fields of Sel are read and written.
// ------------------------------------------------------------------------------------
// Which rows a launch of the ordered compaction takes: the rows selected from the dense pass's
// lists (the guess held) and the rows that go through the classic passes are handled by two
// chains of kernels that run side by side.
enum { kRowsListed = 1, kRowsClassic = 2 };

__global__ void __launch_bounds__(kBlock)
k_topk_pick(const uint32_t *__restrict__ hist_all, Sel *__restrict__ sel_all, int level,
            uint32_t k, const uint32_t *__restrict__ hit, uint32_t *__restrict__ floor_bucket)
{
    const int row = blockIdx.x;
    if (hit[row]) return;                             // rows selected from lists pick inside k_scan_lists
    pick_row(hist_all + (int64_t)row * kHistStride, sel_all + row, level, k, floor_bucket + row);
}

// ------------------------------------------------------------------------------------
// Second dense pass: bitmaps of "key >> 20 above the level-1 bucket" (certainly kept) and
// "inside it" (candidates), and the level-2 histogram of the candidates.
// grid = (ceil(d/4096), rows).
// ------------------------------------------------------------------------------------
template <bool HAS_B>
__global__ void __launch_bounds__(kBlock)
k_topk_mark(const float *__restrict__ a_all, const float *__restrict__ b_all,
            const Sel *__restrict__ sel_all, uint32_t *__restrict__ bm_in_all,
            uint32_t *__restrict__ bm_cand_all, uint32_t *__restrict__ hist_all,
            const uint32_t *__restrict__ hit, int64_t d, int64_t wp, int vec_ok, int64_t stride, RowTail tail)
{
    __shared__ uint32_t h[kBins2];
    if (hit[blockIdx.y]) return;
    for (int t = threadIdx.x; t < kBins2; t += kBlock) h[t] = 0;
    __syncthreads();
    const int row = blockIdx.y;
    const float *a = a_all + (int64_t)row * stride;
    const float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    uint32_t *bm_in = bm_in_all + (int64_t)row * wp, *bm_cand = bm_cand_all + (int64_t)row * wp;
    const uint32_t b1 = sel_all[row].b1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // blocks loop over tiles: the grid is small, so rows whose guess held cost almost nothing
    for (int64_t base = (int64_t)blockIdx.x * kSub; base < d; base += (int64_t)gridDim.x * kSub) {
        if (vec_ok && base + kSub <= d) {
            const int64_t wb = base + warp * kWarpSpan;
            float4 A[4], Bv[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int64_t j = wb + v * 128 + lane * 4;
                A[v] = ld_ro4(a + j);
                if (HAS_B) Bv[v] = ld_ro4(b + j);
            }
            uint32_t BI[4][4], BC[4][4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                if (HAS_B) {
                    A[v].x = __fsub_rn(A[v].x, Bv[v].x); A[v].y = __fsub_rn(A[v].y, Bv[v].y);
                    A[v].z = __fsub_rn(A[v].z, Bv[v].z); A[v].w = __fsub_rn(A[v].w, Bv[v].w);
                }
                const uint32_t kx = key_of(A[v].x), ky = key_of(A[v].y);
                const uint32_t kz = key_of(A[v].z), kw = key_of(A[v].w);
                BI[v][0] = __ballot_sync(kFull, (kx >> 20) > b1);
                BI[v][1] = __ballot_sync(kFull, (ky >> 20) > b1);
                BI[v][2] = __ballot_sync(kFull, (kz >> 20) > b1);
                BI[v][3] = __ballot_sync(kFull, (kw >> 20) > b1);
                const bool cx = (kx >> 20) == b1, cy = (ky >> 20) == b1;
                const bool cz = (kz >> 20) == b1, cw = (kw >> 20) == b1;
                BC[v][0] = __ballot_sync(kFull, cx);
                BC[v][1] = __ballot_sync(kFull, cy);
                BC[v][2] = __ballot_sync(kFull, cz);
                BC[v][3] = __ballot_sync(kFull, cw);
                if (cx) atomicAdd(&h[(kx >> 9) & (kBins2 - 1)], 1u);
                if (cy) atomicAdd(&h[(ky >> 9) & (kBins2 - 1)], 1u);
                if (cz) atomicAdd(&h[(kz >> 9) & (kBins2 - 1)], 1u);
                if (cw) atomicAdd(&h[(kw >> 9) & (kBins2 - 1)], 1u);
            }
            const uint32_t wi = warp_words(BI, lane), wc = warp_words(BC, lane);
            if (lane < 16) { bm_in[(wb >> 5) + lane] = wi; bm_cand[(wb >> 5) + lane] = wc; }
        } else {
            const int64_t end = min(base + (int64_t)kSub, d);
            for (int64_t j = base + threadIdx.x; j - lane < end; j += kBlock) {
                const bool valid = j < end;
                const uint32_t key = valid ? key_of(diff1<HAS_B>(a, b, j)) : 0u;
                const bool in = valid && (key >> 20) > b1, cand = valid && (key >> 20) == b1;
                const uint32_t wi = __ballot_sync(kFull, in), wc = __ballot_sync(kFull, cand);
                if (lane == 0) { bm_in[j >> 5] = wi; bm_cand[j >> 5] = wc; }
                if (cand) atomicAdd(&h[(key >> 9) & (kBins2 - 1)], 1u);
            }
        }
    }
    __syncthreads();
    uint32_t *hist = hist_all + (int64_t)row * kHistStride + kBins1;
    for (int t = threadIdx.x; t < kBins2; t += kBlock)
        if (h[t]) atomicAdd(&hist[t], h[t]);
    if (tail.tick && last_block_of_row(tail.tick + row, gridDim.x))
        pick_row(hist_all + (int64_t)row * kHistStride, const_cast<Sel *>(sel_all) + row, 1, 0u, tail.floor_bucket + row);
}

// Bin of a key at or above the floor key fk in the speculative pass: 2^11 keys per bin
// counted from the floor, so the 2047 regular bins span four level-1 buckets (half an
// octave) and bin 2047 takes everything above.  A threshold that falls into a regular bin
// is then known down to key bit 11, and one more pass over the lists (bits 10..0) gives it
// exactly: two levels instead of three.
__device__ __forceinline__ uint32_t fine_bin(uint32_t key, uint32_t fk) { return min((key - fk) >> 11, (uint32_t)kBins1 - 1u); }

// ------------------------------------------------------------------------------------
// Speculative single dense pass.  The threshold moves little from one iteration to the
// next, so the level-1 bucket of the previous selection, lowered by a margin, is taken as a
// floor: this pass histograms only the coordinates at or above the floor (a few percent, so
// few shared-memory atomics) and keeps them as the tile's list (position, value) in index
// order.  If at least k coordinates lie at or above the floor, the threshold bucket is found
// from this histogram and the second dense pass is not needed; otherwise the two classic
// passes run.  grid = (tiles, rows) for the tiles tile0, tile0 + 1, ... of every row.
// ------------------------------------------------------------------------------------
// Did the guess hold?  It did if the k-th largest key lies in one of the regular fine bins
// above the floor; then key bits 30..11 of the threshold follow from the histogram of those
// coordinates.  Otherwise the row's level-1 histogram is cleared for the full pass.  Run by
// one whole block for the row.  (Folding this into the dense pass - the block that finishes a
// row last takes it over - was measured twice: the memory fence before a block's ticket, in
// every thread or in the ticket-taking thread alone after a barrier, waits for the block's
// outstanding writes and cost the bandwidth-bound pass 0.2 ms either way.)
__device__ __forceinline__ void pick_spec_row(uint32_t *hist, Sel *sel, uint32_t k, uint32_t fl, uint32_t *hit_row)
{
    __shared__ uint32_t tot[kBlock];
    __shared__ uint32_t found;
    if (threadIdx.x == 0) found = 0u;
    const int per = kBins1 / kBlock, lo = threadIdx.x * per;
    uint32_t own[kBins1 / kBlock];
    uint32_t mine = 0;
#pragma unroll
    for (int t = 0; t < per; ++t) {
        own[t] = fl < (uint32_t)kBins1 ? __ldcg(hist + lo + t) : 0u;
        mine += own[t];
    }
    tot[threadIdx.x] = mine;
    __syncthreads();
    uint32_t above = 0;
    for (int t = threadIdx.x + 1; t < kBlock; ++t) above += tot[t];
    if (fl < (uint32_t)kBins1) {
#pragma unroll
        for (int t = per - 1; t >= 0; --t) {
            const uint32_t c = own[t];
            if (above < k && above + c >= k && lo + t < kBins1 - 1) {    // the last bin is open-ended: no threshold from it
                sel->pre = (fl << 20) + ((uint32_t)(lo + t) << 11);
                sel->b1 = sel->pre >> 20; sel->k1 = k - above; sel->c1 = c;
                found = 1u;
            }
            above += c;
        }
    }
    __syncthreads();
    const uint32_t ok = found;
    if (threadIdx.x == 0) *hit_row = ok;
    if (!ok)
        for (int t = threadIdx.x; t < kBins1; t += kBlock) hist[t] = 0u;
}

// grid = (rows), one block each.
__global__ void __launch_bounds__(kBlock)
k_topk_pick_spec(uint32_t *__restrict__ hist_all, Sel *__restrict__ sel_all, uint32_t k,
                 const uint32_t *__restrict__ floor_bucket, uint32_t *__restrict__ hit)
{
    const int row = blockIdx.x;
    pick_spec_row(hist_all + (int64_t)row * kHistStride, sel_all + row, k, floor_bucket[row], hit + row);
}

// Server aggregation fused into the server's dense pass (Algorithm 1: ghat += mean of the
// workers' messages, then c = C(ghat - gtil)): the n payloads whose entries a tile needs.
struct Agg {
    const uint32_t *idx;              // n x k coordinates, increasing in every row
    const float *val;                 // n x k values
    const uint32_t *tile_off;         // n x nt4k: payload offset of every 4096-coordinate tile (rows with hit)
    const uint32_t *hit;              // n: 1 = the row has tile offsets; 0 = search its coordinates
    int64_t k;
    int n, n_pow2;
};
constexpr int kAggStageWorkers = 16;  // workers whose tile entries are staged in shared memory at once
constexpr int kAggMaxWorkers = 64;    // workers that the staged path takes, batch after batch
constexpr int kAggStageCap = 64;      // entries per worker and tile that the staged path holds

__device__ __forceinline__ int64_t lower_bound_idx(const uint32_t *p, int64_t count, int64_t key)
{
    if (key >= ((int64_t)1 << 32)) return count;
    int64_t lo = 0, hi = count;
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)p[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// The payload of the previous selection that is still to be applied to a row's tile
// (deferred state update): entries [begin, end) of the row's payload arrays.
struct Pending {
    const uint32_t *pending;          // rows: 1 = the row's last payload is not in b yet
    const uint32_t *idx;              // rows x k
    const float *val;                 // rows x k
    const uint32_t *tile_off;         // rows x nt4k: payload offset of every tile's first entry
    int64_t k;
};

// APPLY: first add the previous payload's values to b at this tile's kept coordinates
// (Algorithm 1: ghat^(i) += c^(i), deferred from the previous iteration), then read b through
// the coherent path, since this block has just written to it.
// AGG (one row, the server's): a is the server aggregate ghat, read AND written.  Before
// anything else the block adds the mean of the n workers' messages to its tile of a: the
// entries of every worker inside the tile (a contiguous run of its payload) are summed per
// coordinate in the order 0, 1, ..., n-1 in shared memory, then a_j += sum_j / n where the
// sum is not zero.  The dense pass proper then works on the updated tile, which is still in
// registers: the separate aggregation kernel's pass over ghat, and its launch, are saved.
// The tile of a is loaded only after the sums are made and the tile of b after the mean is
// added, so that the kernel fits five blocks on an SM (46 registers), which hide those waits:
// measured 0.166 ms for the server stage of 25.6 M coordinates against 0.175 with the loads
// issued first and four blocks (and 0.174 with six blocks, which spill).
// With up to kAggMaxWorkers workers and kAggStageCap entries each in the tile, the entries
// are staged in shared memory, kAggStageWorkers workers at a time, and every warp adds, worker
// by worker, those among its own 512 coordinates; otherwise the block adds worker by worker
// with a barrier after each.  A row
// without a guess still gets the aggregation.
template <bool HAS_B, bool APPLY, bool AGG>
__global__ void __launch_bounds__(kBlock, AGG ? 5 : 1)
k_topk_spec(const float *__restrict__ a_all, float *b_all,
            const uint32_t *__restrict__ floor_bucket, uint32_t *__restrict__ hist_all,
            float *__restrict__ stash_all, uint16_t *__restrict__ stash_pos_all,
            uint32_t *__restrict__ stash_cnt_all, int64_t d, int vec_ok, int64_t stride, int64_t tile0,
            int64_t nt4k, Pending pd, Agg ag, float *a_rw)
{
    __shared__ uint32_t h[kBins1];
    __shared__ uint32_t wcnt[kBlock / 32];
    // flagged groups of a warp in the dense loop; with AGG, first the per-coordinate sums of the
    // warp's 512 coordinates (each warp's part is used by that warp alone, one use after the other)
    __shared__ float4 s_u[kBlock / 32][kWarpSpan / 4];
    __shared__ uint16_t s_p[kBlock / 32][kWarpSpan / 4];
    const int row = blockIdx.y;
    const uint32_t fl = floor_bucket[row];
    const bool guess = fl < (uint32_t)kBins1;
    if (!guess && !AGG) return;                       // no guess for this row (and then nothing pending)
    const uint32_t fk = fl << 20;                     // lowest key at or above the floor
    for (int t = threadIdx.x; t < kBins1; t += kBlock) h[t] = 0;
    const float *a = a_all + (int64_t)row * stride;
    float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    const int64_t tile = (int64_t)row * nt4k + tile0 + blockIdx.x;      // tiles tile0.. of the row
    if (APPLY && pd.pending[row]) {
        const int64_t t = tile0 + blockIdx.x;
        const int64_t begin = pd.tile_off[tile], end = t + 1 < nt4k ? (int64_t)pd.tile_off[tile + 1] : pd.k;
        for (int64_t e = begin + threadIdx.x; e < end; e += kBlock) {
            const uint32_t j = pd.idx[(int64_t)row * pd.k + e];
            if ((int64_t)j < d) b[j] = __fadd_rn(__ldcg(b + j), pd.val[(int64_t)row * pd.k + e]);
        }
    }
    __syncthreads();
    float *stash = stash_all + tile * kStashCap;
    uint16_t *spos = stash_pos_all + tile * kStashCap;
    const int64_t base = (tile0 + blockIdx.x) * kSub;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const bool vec_tile = vec_ok && base + kSub <= d;
    float *acc = reinterpret_cast<float *>(&s_u[0][0]);           // AGG: kSub sums, warp w owns [512 w, 512 w + 512)
    float4 A[4], Bv[4];
    auto load_tile = [&](bool want_a, bool want_b) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int64_t j = base + warp * kWarpSpan + v * 128 + lane * 4;
            if (want_a) A[v] = AGG ? ld_rw4(a + j) : ld_ro4(a + j);
            if (HAS_B && want_b) Bv[v] = APPLY ? ld_cg4(b + j) : ld_ro4(b + j);
        }
    };
    if (vec_tile && !AGG) load_tile(true, true);
    if constexpr (AGG) {
        __shared__ uint32_t s_rng[2];
        __shared__ uint16_t s_epos[kAggStageWorkers][kAggStageCap];     // staged entries: position in the tile
        __shared__ float s_eval[kAggStageWorkers][kAggStageCap];        // ... and value
        // s_first[i][w]: first staged entry of worker i at or beyond warp w's 512 coordinates
        // (w = 0 .. 8; the entries are in increasing order, so warp w's are [first[w], first[w + 1]))
        __shared__ uint8_t s_first[kAggStageWorkers][kBlock / 32 + 1];
        const int64_t t = tile0 + blockIdx.x;
        for (int e = threadIdx.x; e < kSub; e += kBlock) acc[e] = 0.0f;
        // entries of worker i inside [base, base + kSub): from the row's tile offsets, or by search
        auto range_of = [&](int i, int side) -> uint32_t {
            if (ag.hit[i]) return t + side < nt4k ? ag.tile_off[(int64_t)i * nt4k + t + side] : (uint32_t)ag.k;
            return (uint32_t)lower_bound_idx(ag.idx + (int64_t)i * ag.k, ag.k, base + (int64_t)side * kSub);
        };
        // Staged path (up to kAggMaxWorkers workers, all with tile offsets, up to kAggStageCap
        // entries each in this tile), in batches of kAggStageWorkers workers: sixteen threads
        // copy the entries of one worker to shared memory, four each (entry u = 16 r + thread),
        // and note where the entries pass from one warp's coordinates to the next one's.
        const int wi = threadIdx.x >> 4, l16 = threadIdx.x & 15;
        bool staged = ag.n <= kAggMaxWorkers;
        // entries [beg, beg + cnt) of worker i's payload lie in this tile (cnt = 0 if i >= n)
        auto entries_of = [&](int i, uint32_t &beg, uint32_t &cnt) -> bool {
            beg = 0u; cnt = 0u;
            if (i >= ag.n) return true;
            const uint32_t has = ag.hit[i];
            beg = ag.tile_off[(int64_t)i * nt4k + t];
            const uint32_t end = t + 1 < nt4k ? ag.tile_off[(int64_t)i * nt4k + t + 1] : (uint32_t)ag.k;
            cnt = end - beg;
            return has != 0u && end >= beg && cnt <= (uint32_t)kAggStageCap;
        };
        auto stage = [&](int i, uint32_t beg, uint32_t cnt) {
            uint32_t pos[4];
            float val[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {              // loads first, stores after
                const uint32_t u = l16 + 16 * r;
                pos[r] = 0xffffffffu;
                val[r] = 0.0f;
                if (u < cnt) {
                    pos[r] = ag.idx[(int64_t)i * ag.k + beg + u] - (uint32_t)base;
                    val[r] = ag.val[(int64_t)i * ag.k + beg + u];
                }
            }
            // warp of the coordinate of entry u (8 = past the tile or no entry), and of entry u - 1
            // (-1 before the first): entry u opens every warp in (that of u - 1, that of u]
            int prev_last = -1;                        // warp of entry 16 r - 1
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint32_t u = l16 + 16 * r;
                const int wq = pos[r] < (uint32_t)kSub ? (int)(pos[r] / kWarpSpan) : kBlock / 32;
                int wprev = __shfl_up_sync(kFull, wq, 1, 16);
                if (l16 == 0) wprev = prev_last;
                prev_last = __shfl_sync(kFull, wq, 15, 16);
                if (u < cnt) {
                    s_epos[wi][u] = (uint16_t)min(pos[r], 0xffffu);
                    s_eval[wi][u] = val[r];
                }
                // entries beyond cnt have wq = 8: the first of them opens the warps that are left
                if (u <= cnt)
                    for (int w8 = wprev + 1; w8 <= wq; ++w8) s_first[wi][w8] = (uint8_t)u;
            }
            if (cnt == (uint32_t)kAggStageCap && l16 == 15)      // a full list: nothing opened the rest
                for (int w8 = prev_last + 1; w8 <= kBlock / 32; ++w8) s_first[wi][w8] = (uint8_t)kAggStageCap;
        };
        // The sum of a coordinate runs over the workers in increasing order.  A warp owns the
        // sums of its 512 coordinates: it walks the staged workers in order and adds each
        // worker's entries among its coordinates (one worker sends a coordinate at most once, so
        // the lanes never meet inside a worker; __syncwarp orders one worker's additions before
        // the next one's).  No block barrier, no atomics.  Lane i holds the range of staged
        // worker i and the loop takes it by shuffle; two workers per turn, sixteen lanes each,
        // fetch their entries together and add one after the other; a range of more than
        // sixteen entries sends the pair through the plain loop.
        auto add_staged = [&](int count) {             // count staged workers (an absent one has an empty range)
            uint32_t my_lo = 0u, my_hi = 0u;
            if (lane < count) {
                my_lo = s_first[lane][warp];
                my_hi = min((uint32_t)s_first[lane][warp + 1], (uint32_t)kAggStageCap);
            }
            const int half = lane >> 4, slot = lane & 15;
            for (int i0 = 0; i0 < count; i0 += 2) {
                const int wk = i0 + half;              // (<= 16: lanes 16.. of the last odd turn find an empty range)
                const uint32_t lo = __shfl_sync(kFull, my_lo, wk), hi = __shfl_sync(kFull, my_hi, wk);
                if (__any_sync(kFull, hi > lo + 16u)) {
                    for (int t2 = 0; t2 < 2; ++t2) {
                        const uint32_t lo2 = __shfl_sync(kFull, lo, 16 * t2), hi2 = __shfl_sync(kFull, hi, 16 * t2);
                        for (uint32_t e = lo2 + lane; e < hi2; e += 32) {
                            const uint32_t q = s_epos[(i0 + t2) & (kAggStageWorkers - 1)][e];
                            if (q < (uint32_t)kSub) acc[q] = __fadd_rn(acc[q], s_eval[(i0 + t2) & (kAggStageWorkers - 1)][e]);
                        }
                        __syncwarp();
                    }
                    continue;
                }
                const uint32_t e = lo + slot;
                const uint32_t q = e < hi ? (uint32_t)s_epos[wk & (kAggStageWorkers - 1)][e] : 0xffffu;
                const bool on = q < (uint32_t)kSub;
                const float val = on ? s_eval[wk & (kAggStageWorkers - 1)][e] : 0.0f;
                if (on && half == 0) acc[q] = __fadd_rn(acc[q], val);        // the lower worker adds first
                __syncwarp();
                if (on && half == 1) acc[q] = __fadd_rn(acc[q], val);
                __syncwarp();
            }
        };
        // every batch must qualify before anything is added (the general path starts from zero sums)
        uint32_t beg0 = 0u, cnt0 = 0u;
        if (staged) {
            staged = entries_of(wi, beg0, cnt0);
            for (int w0 = kAggStageWorkers; w0 < ag.n; w0 += kAggStageWorkers) {
                uint32_t bx, cx;
                if (!entries_of(w0 + wi, bx, cx)) staged = false;
            }
        }
        stage(wi, beg0, staged ? cnt0 : 0u);          // (by all threads: it shuffles)
        if (!__syncthreads_or(!staged)) {             // (the barrier also orders the zeroing and the staging)
            add_staged(min(ag.n, kAggStageWorkers));
            for (int w0 = kAggStageWorkers; w0 < ag.n; w0 += kAggStageWorkers) {     // more than sixteen workers: batch after batch
                __syncthreads();                      // the batch before has been read by all warps
                uint32_t bx, cx;
                entries_of(w0 + wi, bx, cx);
                stage(w0 + wi, bx, cx);
                __syncthreads();
                add_staged(min(ag.n - w0, kAggStageWorkers));
            }
            if (!vec_tile) __syncthreads();           // the scalar path below reads other warps' sums
        } else {
            // general case: worker after worker over the whole block, a barrier after each
            for (int i = 0; i < ag.n; ++i) {
                if (threadIdx.x < 2) s_rng[threadIdx.x] = range_of(i, threadIdx.x);
                __syncthreads();
                const uint32_t lo = s_rng[0], hi = s_rng[1];
                for (uint32_t at = lo + threadIdx.x; at < hi; at += kBlock) {
                    const uint32_t q = ag.idx[(int64_t)i * ag.k + at] - (uint32_t)base;
                    if (q < (uint32_t)kSub) acc[q] = __fadd_rn(acc[q], ag.val[(int64_t)i * ag.k + at]);
                }
                __syncthreads();
            }
        }
        const float fn = (float)ag.n, rn = 1.0f / fn;
        auto mean = [&](float v) { return ag.n_pow2 ? __fmul_rn(v, rn) : __fdiv_rn(v, fn); };
        if (vec_tile) load_tile(true, false);         // (after the aggregation: the other blocks of the SM hide the wait)
        if (vec_tile) {
            // (the choice between the multiplication and the division is made once, outside the
            // per-coordinate code; untouched coordinates keep their bits: no addition of a zero)
            auto add_means = [&](auto mean_of) {
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int p = warp * kWarpSpan + v * 128 + lane * 4;
                    const float4 c = *reinterpret_cast<const float4 *>(acc + p);
                    if (c.x != 0.0f || c.y != 0.0f || c.z != 0.0f || c.w != 0.0f) {
                        const float sx = __fadd_rn(A[v].x, mean_of(c.x)), sy = __fadd_rn(A[v].y, mean_of(c.y));
                        const float sz = __fadd_rn(A[v].z, mean_of(c.z)), sw = __fadd_rn(A[v].w, mean_of(c.w));
                        A[v].x = c.x != 0.0f ? sx : A[v].x; A[v].y = c.y != 0.0f ? sy : A[v].y;
                        A[v].z = c.z != 0.0f ? sz : A[v].z; A[v].w = c.w != 0.0f ? sw : A[v].w;
                        st_rw4(a_rw + base + p, A[v]);
                    }
                }
            };
            if (ag.n_pow2) add_means([&](float v) { return __fmul_rn(v, rn); });
            else add_means([&](float v) { return __fdiv_rn(v, fn); });
            __syncwarp();                             // the warp's sums are read: its part of s_u is free again
            load_tile(false, true);
        } else {
            const int64_t end = min(base + (int64_t)kSub, d);
            for (int64_t j = base + threadIdx.x; j < end; j += kBlock) {
                const float c = acc[j - base];
                if (c != 0.0f) a_rw[j] = __fadd_rn(a_rw[j], mean(c));
            }
            __syncthreads();                          // the scalar pass below reads a from memory
        }
        if (!guess) return;                           // block-uniform: aggregation only
    }
    if (vec_tile) {
        // Few coordinates lie at or above the floor (a percent or two), so the per-coordinate
        // work is kept out of the dense loop: a thread only tests each of its four float4
        // groups as a whole (one vote per group), flagged groups are moved to a small list in
        // shared memory in index order, and the warp then works on that list densely - keys,
        // histogram, ranks and the writes of the tile's (position, value) list.
        const float fkf = __uint_as_float(fk);
        uint32_t FB[4];
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            if (HAS_B) {
                A[v].x = __fsub_rn(A[v].x, Bv[v].x); A[v].y = __fsub_rn(A[v].y, Bv[v].y);
                A[v].z = __fsub_rn(A[v].z, Bv[v].z); A[v].w = __fsub_rn(A[v].w, Bv[v].w);
            }
            // |u| >= floor for a finite u; true for a NaN as well, like the comparison of the key bits
            const bool f = !(fabsf(A[v].x) < fkf) || !(fabsf(A[v].y) < fkf) || !(fabsf(A[v].z) < fkf) ||
                           !(fabsf(A[v].w) < fkf);
            FB[v] = __ballot_sync(kFull, f);
        }
        uint32_t nsl = 0;                             // flagged groups of this warp, in index order
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            if ((FB[v] >> lane) & 1u) {
                const uint32_t sl = nsl + __popc(FB[v] & lt);
                s_u[warp][sl] = A[v];
                s_p[warp][sl] = (uint16_t)(warp * kWarpSpan + v * 128 + lane * 4);
            }
            nsl += __popc(FB[v]);
        }
        __syncwarp();
        // which of the four coordinates of list entry sl are at or above the floor (bit c = component c)
        auto kept_of = [&](uint32_t sl, float4 &U) -> uint32_t {
            if (sl >= nsl) return 0u;
            U = s_u[warp][sl];
            return (key_of(U.x) >= fk ? 1u : 0u) | (key_of(U.y) >= fk ? 2u : 0u) | (key_of(U.z) >= fk ? 4u : 0u) |
                   (key_of(U.w) >= fk ? 8u : 0u);
        };
        uint32_t mine = 0;
        for (uint32_t s0 = 0; s0 < nsl; s0 += 32) {   // warp-uniform
            float4 U;
            const uint32_t pm = kept_of(s0 + lane, U);
            if (pm & 1u) atomicAdd(&h[fine_bin(key_of(U.x), fk)], 1u);
            if (pm & 2u) atomicAdd(&h[fine_bin(key_of(U.y), fk)], 1u);
            if (pm & 4u) atomicAdd(&h[fine_bin(key_of(U.z), fk)], 1u);
            if (pm & 8u) atomicAdd(&h[fine_bin(key_of(U.w), fk)], 1u);
            mine += __reduce_add_sync(kFull, (uint32_t)__popc(pm));
        }
        if (lane == 0) wcnt[warp] = mine;             // the same in every lane
        __syncthreads();
        uint32_t rank = 0, total = 0;
#pragma unroll
        for (int w8 = 0; w8 < kBlock / 32; ++w8) {
            if (w8 < warp) rank += wcnt[w8];
            total += wcnt[w8];
        }
        // index order: coordinate = warp * 512 + v * 128 + lane * 4 + component = list order, then component
        for (uint32_t s0 = 0; s0 < nsl; s0 += 32) {
            float4 U;
            const uint32_t pm = kept_of(s0 + lane, U);
            const uint32_t cnt = __popc(pm);
            uint32_t inc = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += t;
            }
            uint32_t r = rank + inc - cnt;
            if (pm) {
                const uint32_t p0 = s_p[warp][s0 + lane];
                if (pm & 1u) { if (r < kStashCap) { stash[r] = U.x; spos[r] = (uint16_t)p0; } ++r; }
                if (pm & 2u) { if (r < kStashCap) { stash[r] = U.y; spos[r] = (uint16_t)(p0 + 1); } ++r; }
                if (pm & 4u) { if (r < kStashCap) { stash[r] = U.z; spos[r] = (uint16_t)(p0 + 2); } ++r; }
                if (pm & 8u) { if (r < kStashCap) { stash[r] = U.w; spos[r] = (uint16_t)(p0 + 3); } }
            }
            rank += __shfl_sync(kFull, inc, 31);
        }
        if (threadIdx.x == 0) stash_cnt_all[tile] = total;
    } else {
        const int64_t end = min(base + (int64_t)kSub, d);
        uint32_t run = 0;                             // coordinates kept so far, block-uniform
        for (int64_t j0 = base; j0 < end; j0 += kBlock) {
            const int64_t j = j0 + threadIdx.x;
            const bool valid = j < end;
            const float aj = !valid ? 0.0f : AGG ? __ldcg(a_rw + j) : a[j];
            const float u = !valid ? 0.0f : !HAS_B ? aj : __fsub_rn(aj, APPLY ? __ldcg(b + j) : b[j]);
            const uint32_t key = key_of(u);
            const bool ge = valid && key >= fk;
            const uint32_t wg = __ballot_sync(kFull, ge);
            if (ge) atomicAdd(&h[fine_bin(key, fk)], 1u);
            if (lane == 0) wcnt[warp] = __popc(wg);
            __syncthreads();
            uint32_t r = run + __popc(wg & lt), total = 0;
#pragma unroll
            for (int w8 = 0; w8 < kBlock / 32; ++w8) {
                if (w8 < warp) r += wcnt[w8];
                total += wcnt[w8];
            }
            if (ge && r < (uint32_t)kStashCap) { stash[r] = u; spos[r] = (uint16_t)(j - base); }
            run += total;
            __syncthreads();
        }
        if (threadIdx.x == 0) stash_cnt_all[tile] = run;
    }
    __syncthreads();
    uint32_t *hist = hist_all + (int64_t)row * kHistStride;
    for (int t = threadIdx.x; t < kBins1; t += kBlock)
        if (h[t]) atomicAdd(&hist[t], h[t]);
}

// ------------------------------------------------------------------------------------
// The same pass over whole tiles with a prefetch ring.  A block owns kSpecTiles consecutive
// tiles of a row; the a and b sub-tiles arrive in a two-stage shared-memory ring by bulk
// asynchronous copies (plain TMA bulk copies) issued by one thread, so the next tile is in
// flight while the block works on the current one.  Arithmetic, histogram and lists are those
// of k_topk_spec; the flagged groups are kept as positions only and read back from the stage.
// Every wait on a copy is bounded; one that runs out sets *error_flag (if given), lets the
// copies in flight land and leaves the block.  grid = (ceil(full tiles / kSpecTiles), rows);
// rows 16-byte aligned, stride % 4 == 0.
// ------------------------------------------------------------------------------------
constexpr int kSpecTiles = 7;        // (16 x 6250 tiles: 5 -> 0.911, 6 -> 0.902, 7 -> 0.901, 8 -> 0.906, 10 -> 0.901, 12 -> 0.904, 16 -> 0.912 ms per step)
constexpr int kSpecStages = 2;

template <bool HAS_B, bool APPLY>
__global__ void __launch_bounds__(kBlock, 3)
k_topk_spec_ring(const float *__restrict__ a_all, float *b_all,
                 const uint32_t *__restrict__ floor_bucket, uint32_t *__restrict__ hist_all,
                 float *__restrict__ stash_all, uint16_t *__restrict__ stash_pos_all,
                 uint32_t *__restrict__ stash_cnt_all, int64_t full_tiles, int64_t stride, int64_t nt4k,
                 int *__restrict__ error_flag, int wait_limit, Pending pd)
{
    constexpr int kStageFloats = (HAS_B ? 2 : 1) * kSub;
    extern __shared__ __align__(128) unsigned char spec_ring[];
    __shared__ __align__(8) uint64_t full[kSpecStages];
    __shared__ uint32_t h[kBins1];
    __shared__ uint32_t wcnt[kBlock / 32];
    __shared__ uint16_t s_p[kBlock / 32][kWarpSpan / 4];
    __shared__ uint32_t s_off[kSpecTiles + 1];        // APPLY: payload offsets of the block's tiles
    const int row = blockIdx.y;
    const uint32_t fl = floor_bucket[row];
    if (fl >= (uint32_t)kBins1) return;               // no guess for this row (and then nothing pending)
    const uint32_t fk = fl << 20;
    const float fkf = __uint_as_float(fk);
    for (int t = threadIdx.x; t < kBins1; t += kBlock) h[t] = 0;
    if (threadIdx.x == 0) {
        for (int st = 0; st < kSpecStages; ++st) mbar_init(&full[st], 1);
        mbar_fence_init();
    }
    const int64_t t0 = (int64_t)blockIdx.x * kSpecTiles;
    const int iters = (int)min((int64_t)kSpecTiles, full_tiles - t0);
    const bool apply = APPLY && pd.pending[row] != 0u;                 // block-uniform
    if (apply && threadIdx.x <= iters) {
        const int64_t t = t0 + threadIdx.x;
        s_off[threadIdx.x] = t < nt4k ? pd.tile_off[(int64_t)row * nt4k + t] : (uint32_t)pd.k;
    }
    __syncthreads();
    const float *a = a_all + (int64_t)row * stride;
    float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    const uint32_t *pidx = APPLY ? pd.idx + (int64_t)row * pd.k : nullptr;
    const float *pval = APPLY ? pd.val + (int64_t)row * pd.k : nullptr;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    float *ring = reinterpret_cast<float *>(spec_ring);
    // the first payload entry of this thread in the coming tile, fetched one tile ahead
    uint32_t nx_idx = 0u;
    float nx_val = 0.0f;
    auto prefetch_entry = [&](int it) {
        if (apply && it < iters) {
            const uint32_t e = s_off[it] + threadIdx.x;
            if (e < s_off[it + 1]) { nx_idx = pidx[e]; nx_val = pval[e]; }
        }
    };
    prefetch_entry(0);
    auto refill = [&](int it, int st) {                        // one thread
        float *dst = ring + (size_t)st * kStageFloats;
        mbar_arrive_expect_tx(&full[st], (uint32_t)(kStageFloats * sizeof(float)));
        bulk_copy_g2s(dst, a + (t0 + it) * kSub, kSub * sizeof(float), &full[st]);
        if (HAS_B) bulk_copy_g2s(dst + kSub, b + (t0 + it) * kSub, kSub * sizeof(float), &full[st]);
    };
    if (threadIdx.x == 0)
        for (int st = 0; st < kSpecStages && st < iters; ++st) refill(st, st);
    bool arrived = true;
    int it = 0;
    for (; it < iters; ++it) {
        const int st = it % kSpecStages;
        const bool landed = mbar_wait_bounded(&full[st], (uint32_t)(it / kSpecStages) & 1u, wait_limit);
        const float *sa = ring + (size_t)st * kStageFloats;
        float *sb = ring + (size_t)st * kStageFloats + kSub;
        if (apply) {
            // Deferred state update: the previous payload's entries of this tile are added to
            // the copy of b in the stage, and every 32-byte sector that holds one is written
            // back whole (all eight floats are at hand, so the store needs no read).
            const uint32_t tbase = (uint32_t)((t0 + it) * kSub);
            const uint32_t e0 = s_off[it], e1 = s_off[it + 1];
            const uint32_t my_pos = nx_idx - tbase;
            const bool mine = e0 + threadIdx.x < e1 && my_pos < (uint32_t)kSub;   // (a valid payload never fails the second test)
            if (mine && landed) sb[my_pos] = __fadd_rn(sb[my_pos], nx_val);
            for (uint32_t e = e0 + kBlock + threadIdx.x; e < e1 && landed; e += kBlock) {      // tiles that kept many
                const uint32_t pos = pidx[e] - tbase;
                if (pos < (uint32_t)kSub) sb[pos] = __fadd_rn(sb[pos], pval[e]);
            }
            __syncthreads();
            float *bt = b + (int64_t)tbase;
            if (mine && landed) {
                const uint32_t sec = my_pos & ~7u;
                st_rw4(bt + sec, *reinterpret_cast<const float4 *>(sb + sec));
                st_rw4(bt + sec + 4, *reinterpret_cast<const float4 *>(sb + sec + 4));
            }
            for (uint32_t e = e0 + kBlock + threadIdx.x; e < e1 && landed; e += kBlock) {
                const uint32_t sec = (pidx[e] - tbase) & ~7u;
                if (sec < (uint32_t)kSub) {
                    st_rw4(bt + sec, *reinterpret_cast<const float4 *>(sb + sec));
                    st_rw4(bt + sec + 4, *reinterpret_cast<const float4 *>(sb + sec + 4));
                }
            }
            prefetch_entry(it + 1);
        }
        // u of the group of four coordinates at tile position p
        auto group = [&](uint32_t p) -> float4 {
            float4 U = *reinterpret_cast<const float4 *>(sa + p);
            if (HAS_B) {
                const float4 Bq = *reinterpret_cast<const float4 *>(sb + p);
                U.x = __fsub_rn(U.x, Bq.x); U.y = __fsub_rn(U.y, Bq.y);
                U.z = __fsub_rn(U.z, Bq.z); U.w = __fsub_rn(U.w, Bq.w);
            }
            return U;
        };
        const int64_t tile = (int64_t)row * nt4k + t0 + it;
        float *stash = stash_all + tile * kStashCap;
        uint16_t *spos = stash_pos_all + tile * kStashCap;
        uint32_t FB[4];
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const float4 U = group((uint32_t)(warp * kWarpSpan + v * 128 + lane * 4));
            const bool f = !(fabsf(U.x) < fkf) || !(fabsf(U.y) < fkf) || !(fabsf(U.z) < fkf) || !(fabsf(U.w) < fkf);
            FB[v] = __ballot_sync(kFull, f);
        }
        uint32_t nsl = 0;                             // flagged groups of this warp, in index order
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            if ((FB[v] >> lane) & 1u)
                s_p[warp][nsl + __popc(FB[v] & lt)] = (uint16_t)(warp * kWarpSpan + v * 128 + lane * 4);
            nsl += __popc(FB[v]);
        }
        __syncwarp();
        auto kept_of = [&](uint32_t sl, float4 &U, uint32_t &p0) -> uint32_t {
            if (sl >= nsl) return 0u;
            p0 = s_p[warp][sl];
            U = group(p0);
            return (key_of(U.x) >= fk ? 1u : 0u) | (key_of(U.y) >= fk ? 2u : 0u) | (key_of(U.z) >= fk ? 4u : 0u) |
                   (key_of(U.w) >= fk ? 8u : 0u);
        };
        uint32_t mine = 0;
        for (uint32_t s0 = 0; s0 < nsl; s0 += 32) {   // warp-uniform
            float4 U;
            uint32_t p0;
            const uint32_t pm = kept_of(s0 + lane, U, p0);
            if (pm & 1u) atomicAdd(&h[fine_bin(key_of(U.x), fk)], 1u);
            if (pm & 2u) atomicAdd(&h[fine_bin(key_of(U.y), fk)], 1u);
            if (pm & 4u) atomicAdd(&h[fine_bin(key_of(U.z), fk)], 1u);
            if (pm & 8u) atomicAdd(&h[fine_bin(key_of(U.w), fk)], 1u);
            mine += __reduce_add_sync(kFull, (uint32_t)__popc(pm));
        }
        if (lane == 0) wcnt[warp] = mine;
        // the barrier also makes the outcome of the waits one decision of the whole block (a
        // thread whose wait ran out has worked on a stage that may be incomplete; everything
        // it touched so far is indexed by positions, not by data, and the results are void)
        arrived = !__syncthreads_or(!landed);
        if (!arrived) break;
        uint32_t rank = 0, total = 0;
#pragma unroll
        for (int w8 = 0; w8 < kBlock / 32; ++w8) {
            if (w8 < warp) rank += wcnt[w8];
            total += wcnt[w8];
        }
        for (uint32_t s0 = 0; s0 < nsl; s0 += 32) {
            float4 U;
            uint32_t p0 = 0;
            const uint32_t pm = kept_of(s0 + lane, U, p0);
            const uint32_t cnt = __popc(pm);
            uint32_t inc = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += t;
            }
            uint32_t r = rank + inc - cnt;
            if (pm & 1u) { if (r < kStashCap) { stash[r] = U.x; spos[r] = (uint16_t)p0; } ++r; }
            if (pm & 2u) { if (r < kStashCap) { stash[r] = U.y; spos[r] = (uint16_t)(p0 + 1); } ++r; }
            if (pm & 4u) { if (r < kStashCap) { stash[r] = U.z; spos[r] = (uint16_t)(p0 + 2); } ++r; }
            if (pm & 8u) { if (r < kStashCap) { stash[r] = U.w; spos[r] = (uint16_t)(p0 + 3); } }
            rank += __shfl_sync(kFull, inc, 31);
        }
        if (threadIdx.x == 0) stash_cnt_all[tile] = total;
        __syncthreads();                              // the stage and wcnt have been read by all
        if (threadIdx.x == 0 && it + kSpecStages < iters) {
            // the stage was also written by this block (deferred update): order those writes
            // before the asynchronous copy that refills it
            if (APPLY) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            refill(it + kSpecStages, st);
        }
    }
    if (!arrived) {
        // report, let the copies in flight (tiles it .. it + kSpecStages - 1 of this block) land
        // within the default limit before the shared memory is released, and leave together
        if (threadIdx.x == 0 && error_flag) atomicExch(error_flag, 1);
        for (int j = it; j < iters && j < it + kSpecStages; ++j)
            mbar_wait_bounded(&full[j % kSpecStages], (uint32_t)(j / kSpecStages) & 1u);
        return;
    }
    uint32_t *hist = hist_all + (int64_t)row * kHistStride;
    for (int t = threadIdx.x; t < kBins1; t += kBlock)
        if (h[t]) atomicAdd(&hist[t], h[t]);
}

// In the list passes below a warp owns kWarpTiles consecutive tiles and a block
// kListTiles; lane L reads entries L, L + 32, ... of a tile's list (coalesced).  The passes
// are bound by memory latency, so the first kPre chunks of every tile of the warp are loaded
// before any is used.  Blocks beyond the last tile return (the grid is sized for the
// bitmap passes of the rows whose guess failed).
constexpr int kTilesPerBlock = kTileWords * 32 / kSub;      // tiles per 32768-coordinate span
constexpr int kWarpTiles = 1;
constexpr int kListTiles = kWarpTiles * (kBlock / 32);
constexpr int kPre = 3;        // (lists of C3 hold about 80 entries: 2 -> 0.9023, 3 -> 0.8988, 4 -> 0.9008, 5 -> 0.9045 ms per step)

// A tile with more than kStashCap coordinates at or above the floor (the selection is
// concentrated there) has no complete list: the passes walk its coordinates in a and b
// instead ("dense" tile).  Every key a pass looks for is at or above the floor, so the
// result is that of a complete list.
struct WarpLists {
    const float *val[kWarpTiles];
    const uint16_t *pos[kWarpTiles];
    uint32_t cnt[kWarpTiles];      // list length; 0 for a dense tile
    uint32_t dense[kWarpTiles];    // coordinates of a dense tile, else 0
    int64_t tile[kWarpTiles];      // index of the tile inside its row (>= nt4k: none, cnt = 0)
};

__device__ __forceinline__ WarpLists warp_lists(const float *stash_all, const uint16_t *stash_pos_all,
                                                const uint32_t *stash_cnt_all, int row, int64_t nt4k,
                                                int64_t d)
{
    WarpLists w;
    const int64_t t0 = ((int64_t)blockIdx.x * (kBlock / 32) + (threadIdx.x >> 5)) * kWarpTiles;
#pragma unroll
    for (int m = 0; m < kWarpTiles; ++m) {
        w.tile[m] = t0 + m;
        const bool any = w.tile[m] < nt4k;
        const int64_t g = (int64_t)row * nt4k + (any ? w.tile[m] : 0);
        w.val[m] = stash_all + g * kStashCap;
        w.pos[m] = stash_pos_all + g * kStashCap;
        const uint32_t raw = any ? stash_cnt_all[g] : 0u;
        w.cnt[m] = raw <= (uint32_t)kStashCap ? raw : 0u;
        w.dense[m] = raw <= (uint32_t)kStashCap ? 0u : (uint32_t)min((int64_t)kSub, d - w.tile[m] * kSub);
    }
    return w;
}

// f(value) for every entry of the warp's lists (every coordinate of its dense tiles).
// The first kPre chunks of a list are fetched without waiting for its length (a tile's list
// has room for kStashCap >= 32 kPre entries, so the reads stay inside it; what lies beyond
// the length is not used): the pass then costs one memory latency per tile instead of two.
template <bool HAS_B, typename F>
__device__ __forceinline__ void for_each_listed(const WarpLists &w, const float *a, const float *b, F &f)
{
    const uint32_t lane = threadIdx.x & 31;
    float v[kWarpTiles][kPre];
#pragma unroll
    for (int m = 0; m < kWarpTiles; ++m)
#pragma unroll
        for (int i = 0; i < kPre; ++i) v[m][i] = w.val[m][lane + 32 * i];      // beyond the list: unused (see for_each_listed)
#pragma unroll
    for (int m = 0; m < kWarpTiles; ++m) {
#pragma unroll
        for (int i = 0; i < kPre; ++i)
            if (lane + 32 * i < w.cnt[m]) f(v[m][i]);
        for (uint32_t e = lane + 32 * kPre; e < w.cnt[m]; e += 32) f(w.val[m][e]);
        for (uint32_t e = lane; e < w.dense[m]; e += 32) f(diff1<HAS_B>(a, b, w.tile[m] * kSub + e));
    }
}

constexpr int kCandPerTile = 4;       // candidates of a tile that are kept with the tile (more: the tile is re-read)

// Per listed value: keys that share bits 30..11 with the threshold ("candidates") go to the
// histogram of bits 10..0 and, as far as there is room, into the tile's candidate slots; keys
// with higher bits 30..11 are certainly kept and only counted.
struct SplitTile {
    uint32_t *h, pre11;               // h: the row's histogram of key bits 10..0 (global)
    uint32_t *slots;                  // shared: candidates seen in this warp's tile so far
    uint16_t *cand;                   // global: the tile's kCandPerTile candidate slots (key bits 10..0)
    uint32_t above;                   // this lane's count of certainly kept values
    __device__ __forceinline__ void operator()(float v)
    {
        const uint32_t key = key_of(v), hi = key >> 11;
        if (hi == pre11) {
            // Candidates are few (one fine bin of the dense pass's histogram), so they go to
            // the row's histogram in global memory directly; the lanes that are here together
            // with the same bin send one addition between them (tie-heavy rows).
            const uint32_t bin = key & (kBins2 - 1);
            const uint32_t same = __match_any_sync(__activemask(), bin);
            if ((__ffs(same) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&h[bin], (uint32_t)__popc(same));
            const uint32_t at = atomicAdd(slots, 1u);
            if (at < (uint32_t)kCandPerTile) cand[at] = (uint16_t)bin;
        } else if (hi > pre11) {
            ++above;
        }
    }
};

// After a successful guess, one pass over the lists: the histogram of key bits 10..0 over the
// listed values that share the threshold's bits 30..11 (the pick inside k_scan_lists gives the
// exact threshold T from it), and per tile what the scan needs to place the tile's kept
// coordinates without reading the list again: the number of values certainly above T
// (cnt_gt), the number of candidates (cnt_eq) and the candidates' low key bits (cand; a tile
// with more than kCandPerTile candidates is counted again from its list by the scan).
// grid = (nbt, rows).
template <bool HAS_B>
__global__ void __launch_bounds__(kBlock)
k_topk_split(const float *__restrict__ a_all, const float *__restrict__ b_all,
             const Sel *__restrict__ sel_all, const uint32_t *__restrict__ hit,
             const float *__restrict__ stash_all, const uint16_t *__restrict__ stash_pos_all,
             const uint32_t *__restrict__ stash_cnt_all, uint32_t *__restrict__ hist_all,
             uint32_t *__restrict__ cnt_gt_all, uint32_t *__restrict__ cnt_eq_all, uint16_t *__restrict__ cand_all,
             int64_t nt4k, int64_t d, int64_t stride)
{
    __shared__ uint32_t s_slots[kBlock / 32];
    const int row = blockIdx.y;
    if (!hit[row] || (int64_t)blockIdx.x * kListTiles >= nt4k) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) s_slots[warp] = 0u;
    __syncwarp();
    const WarpLists w = warp_lists(stash_all, stash_pos_all, stash_cnt_all, row, nt4k, d);
    const int64_t g = (int64_t)row * nt4k + (w.tile[0] < nt4k ? w.tile[0] : 0);
    SplitTile f{hist_all + (int64_t)row * kHistStride + kBins1, sel_all[row].pre >> 11, &s_slots[warp],
                cand_all + g * kCandPerTile, 0u};
    for_each_listed<HAS_B>(w, a_all + (int64_t)row * stride, HAS_B ? b_all + (int64_t)row * stride : nullptr, f);
    __syncwarp();
    uint32_t above = f.above;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) above += __shfl_xor_sync(kFull, above, o);
    if (lane == 0 && w.tile[0] < nt4k) {
        cnt_gt_all[g] = above;
        cnt_eq_all[g] = s_slots[warp];
    }
}

// ------------------------------------------------------------------------------------
// Level 3 (rows whose guess failed): histogram of key & 511 over the candidates whose upper
// 22 key bits match.  grid = (blocks, rows), blocks loop over the 32768-coordinate spans; a
// thread walks the set bits of its bitmap words.
// ------------------------------------------------------------------------------------
template <bool HAS_B>
__global__ void __launch_bounds__(kBlock)
k_topk_hist3(const float *__restrict__ a_all, const float *__restrict__ b_all,
             const Sel *__restrict__ sel_all, const uint32_t *__restrict__ hit,
             const uint32_t *__restrict__ bm_cand_all, uint32_t *__restrict__ hist_all,
             int64_t wp, int64_t nbt, int64_t stride, RowTail tail)
{
    __shared__ uint32_t h[kBins3];
    const int row = blockIdx.y;
    if (hit[row]) return;                             // rows with lists have their threshold already
    for (int t = threadIdx.x; t < kBins3; t += kBlock) h[t] = 0;
    __syncthreads();
    const uint32_t *bm_cand = bm_cand_all + (int64_t)row * wp;
    const uint32_t pre = (sel_all[row].b1 << 11) | sel_all[row].b2;
    const float *a = a_all + (int64_t)row * stride;
    const float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    for (int64_t bx = blockIdx.x; bx < nbt; bx += gridDim.x) {
        const int64_t w0 = bx * kTileWords;
        for (int t = threadIdx.x; t < kTileWords && w0 + t < wp; t += kBlock) {
            uint32_t word = bm_cand[w0 + t];
            while (word) {
                const int bit = __ffs(word) - 1;
                word &= word - 1;
                const uint32_t key = key_of(diff1<HAS_B>(a, b, (w0 + t) * 32 + bit));
                if ((key >> 9) == pre) atomicAdd(&h[key & (kBins3 - 1)], 1u);
            }
        }
    }
    __syncthreads();
    uint32_t *hist = hist_all + (int64_t)row * kHistStride + kBins1 + kBins2;
    for (int t = threadIdx.x; t < kBins3; t += kBlock)
        if (h[t]) atomicAdd(&hist[t], h[t]);
    if (tail.tick && last_block_of_row(tail.tick + row, gridDim.x))
        pick_row(hist_all + (int64_t)row * kHistStride, const_cast<Sel *>(sel_all) + row, 2, 0u, tail.floor_bucket + row);
}

// ------------------------------------------------------------------------------------
// With the threshold key T known (rows whose guess failed; the rows selected from lists get
// their per-tile counts in k_topk_split and k_scan_lists): bm_in |= candidates with key > T;
// bm_cand := candidates with key == T; if all ties are needed they are merged at once,
// otherwise the per-tile tie counts feed the ordered pick below.  grid = (nbt, rows).
// ------------------------------------------------------------------------------------
template <bool HAS_B>
__global__ void __launch_bounds__(kBlock)
k_topk_resolve(const float *__restrict__ a_all, const float *__restrict__ b_all,
               const Sel *__restrict__ sel_all, const uint32_t *__restrict__ hit,
               uint32_t *__restrict__ bm_in_all, uint32_t *__restrict__ bm_cand_all,
               uint32_t *__restrict__ cnt_tie_all, int64_t wp, int64_t nbt, int64_t stride, unsigned int *tick)
{
    const int row = blockIdx.y;
    if (hit[row]) return;
    uint32_t *bm_in = bm_in_all + (int64_t)row * wp, *bm_cand = bm_cand_all + (int64_t)row * wp;
    const Sel s = sel_all[row];
    const uint32_t T = (s.b1 << 20) | (s.b2 << 9) | s.b3;
    const bool all_ties = s.k3 == s.c3;
    uint32_t nt = 0;
    const float *a = a_all + (int64_t)row * stride;
    const float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    const int64_t w0 = (int64_t)blockIdx.x * kTileWords;
    for (int t = threadIdx.x; t < kTileWords && w0 + t < wp; t += kBlock) {
        uint32_t word = bm_cand[w0 + t], keep = bm_in[w0 + t], tie = 0;
        while (word) {
            const int bit = __ffs(word) - 1;
            word &= word - 1;
            const uint32_t key = key_of(diff1<HAS_B>(a, b, (w0 + t) * 32 + bit));
            if (key > T) keep |= 1u << bit;
            else if (key == T) tie |= 1u << bit;
        }
        if (all_ties) keep |= tie;
        bm_in[w0 + t] = keep;
        bm_cand[w0 + t] = tie;
        nt += __popc(tie);
    }
    uint32_t total;
    block_excl_scan(nt, total);
    if (threadIdx.x == 0) cnt_tie_all[(int64_t)row * nbt + blockIdx.x] = total;
    // the exclusive scan of the row's tie counts, by the block that finishes the row last
    if (tick && last_block_of_row(tick + row, gridDim.x)) scan_row(cnt_tie_all + (int64_t)row * nbt, nbt, nullptr, true);
}

// Exclusive scan of the per-tile counts of the rows whose guess failed, in place
// (skip_hit: rows with lists are left alone).  grid = (rows).
__global__ void __launch_bounds__(kBlock)
k_scan_tiles(uint32_t *__restrict__ cnt_all, int64_t nbt, const uint32_t *__restrict__ hit,
             uint32_t *__restrict__ totals = nullptr, bool in_place = true)
{
    if (hit[blockIdx.x]) return;
    scan_row(cnt_all + (int64_t)blockIdx.x * nbt, nbt, totals ? totals + blockIdx.x : nullptr, in_place);
}

// Rows with lists: from the per-tile counts of keys above / equal to the threshold to, per
// tile, the rank of its first tie among the row's ties (cnt_eq) and the payload offset of its
// first kept coordinate (cnt_gt); a tile keeps its keys above T and those of its ties whose
// rank is below k3.  Every eighth tile's offset is also the offset of its 32768-coordinate
// span (cnt_fin), which the server aggregation uses.  The counts come from k_topk_split's
// per-tile records (certainly kept values, candidates and their low key bits) once this kernel
// has picked the exact threshold from the low-bits histogram.  They pass through shared memory
// in chunks of 8192 tiles (coalesced loads and stores; a row of up to 33.5 M coordinates is one
// chunk: one round of loads and two block scans); inside a chunk a thread owns 8 consecutive
// tiles (padded rows, no bank conflicts).  grid = (rows), 1024 threads: the row's scan is one
// block's serial work, so the block is as wide as it gets.  Dynamic shared memory: kScanSmemBytes.
constexpr int kScanBlock = 1024;      // one block per row does the whole scan: as wide as a block gets
constexpr int kScanPer = 8;
constexpr int kScanChunk = kScanBlock * kScanPer;
constexpr int kScanSmemBytes = 2 * (kScanChunk + kScanBlock) * (int)sizeof(uint32_t);
__device__ __forceinline__ int scan_slot(int i) { return i + i / kScanPer; }

template <bool HAS_B>
__global__ void __launch_bounds__(kScanBlock)
k_scan_lists(const float *__restrict__ a_all, const float *__restrict__ b_all,
             Sel *__restrict__ sel_all, const uint32_t *__restrict__ hit,
             const uint32_t *__restrict__ hist_all, uint32_t *__restrict__ floor_bucket,
             const float *__restrict__ stash_all, const uint32_t *__restrict__ stash_cnt_all,
             const uint16_t *__restrict__ cand_all,
             uint32_t *__restrict__ cnt_gt_all, uint32_t *__restrict__ cnt_eq_all,
             uint32_t *__restrict__ cnt_fin_all, int64_t nt4k, int64_t nbt, int64_t d, int64_t stride)
{
    extern __shared__ uint32_t scan_smem[];
    uint32_t *s_eq = scan_smem, *s_gt = scan_smem + kScanChunk + kScanBlock;
    __shared__ uint32_t s_T, s_k3, s_c3;
    const int row = blockIdx.x;
    if (!hit[row]) return;
    // The exact threshold first: the bucket of key bits 10..0 that holds the k1-th largest of
    // the candidates (the histogram k_topk_split made), as k_topk_pick does for the classic rows.
    {
        Sel *sel = sel_all + row;
        const uint32_t *hist = hist_all + (int64_t)row * kHistStride + kBins1;
        const uint32_t want = sel->k1;
        constexpr int per = kBins2 / kScanBlock;
        const int lo = threadIdx.x * per;
        uint32_t own[per];
        uint32_t mine = 0;
#pragma unroll
        for (int t = 0; t < per; ++t) { own[t] = hist[lo + t]; mine += own[t]; }
        uint32_t all;
        const uint32_t before = block_excl_scan_n<kScanBlock>(mine, all);
        uint32_t above = all - before - mine;          // entries in bins owned by later threads
#pragma unroll
        for (int t = per - 1; t >= 0; --t) {
            const uint32_t c = own[t];
            if (above < want && above + c >= want) {   // exactly one thread and bucket
                const uint32_t T = sel->pre | (uint32_t)(lo + t);
                sel->b1 = T >> 20; sel->b2 = (T >> 9) & (kBins2 - 1); sel->b3 = T & (kBins3 - 1);
                sel->k3 = want - above; sel->c3 = c;
                // guess for the next selection of this row: a little below this threshold
                floor_bucket[row] = (T >> 20) > kGuessMargin ? (T >> 20) - kGuessMargin : 1u;
                s_T = T; s_k3 = want - above; s_c3 = c;
            }
            above += c;
        }
        __syncthreads();
    }
    const uint32_t T = s_T, k3 = s_k3, Tlow = T & (kBins2 - 1);
    const bool all_ties = k3 == s_c3;
    uint32_t *gt = cnt_gt_all + (int64_t)row * nt4k, *eq = cnt_eq_all + (int64_t)row * nt4k;
    const uint2 *cand = reinterpret_cast<const uint2 *>(cand_all) + (int64_t)row * nt4k;
    uint32_t *fin = cnt_fin_all + (int64_t)row * nbt;
    const float *a = a_all + (int64_t)row * stride;
    const float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
    uint32_t carry_eq = 0, carry_keep = 0;             // block-uniform
    for (int64_t c0 = 0; c0 < nt4k; c0 += kScanChunk) {
        // all loads of the chunk first (independent, in flight together), then the counting
        uint32_t G[kScanPer], NC[kScanPer];
        uint2 C4[kScanPer];
#pragma unroll
        for (int m = 0; m < kScanPer; ++m) {
            const int64_t t = c0 + m * kScanBlock + threadIdx.x;
            const bool in = t < nt4k;
            G[m] = in ? gt[t] : 0u;
            NC[m] = in ? eq[t] : 0u;
            C4[m] = in ? cand[t] : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int m = 0; m < kScanPer; ++m) {
            const int i = m * kScanBlock + threadIdx.x;
            const int64_t t = c0 + i;
            // keys above / equal to T in tile t: the certainly kept values plus the candidates
            uint32_t g = G[m], e = 0u;
            const uint32_t lows[4] = {C4[m].x & 0xffffu, C4[m].x >> 16, C4[m].y & 0xffffu, C4[m].y >> 16};
#pragma unroll
            for (int c = 0; c < kCandPerTile; ++c) {
                const bool have = (uint32_t)c < NC[m];
                g += have && lows[c] > Tlow;
                e += have && lows[c] == Tlow;
            }
            if (NC[m] > (uint32_t)kCandPerTile) {
                // more candidates than the tile's slots hold (ties in bulk, or a selection
                // concentrated here): counted again from the tile's list, or from the data
                g = 0u; e = 0u;
                const int64_t tg = (int64_t)row * nt4k + t;
                const uint32_t raw = stash_cnt_all[tg];
                if (raw <= (uint32_t)kStashCap) {
                    const float *val = stash_all + tg * kStashCap;
                    for (uint32_t u = 0; u < raw; ++u) { const uint32_t key = key_of(val[u]); g += key > T; e += key == T; }
                } else {
                    const int64_t lo = t * kSub, hi = min(lo + (int64_t)kSub, d);
                    for (int64_t j = lo; j < hi; ++j) { const uint32_t key = key_of(diff1<HAS_B>(a, b, j)); g += key > T; e += key == T; }
                }
            }
            s_eq[scan_slot(i)] = e;
            s_gt[scan_slot(i)] = g;
        }
        __syncthreads();
        const int mine = threadIdx.x * (kScanPer + 1);  // first slot of this thread's tiles
        uint32_t sum_eq = 0;
#pragma unroll
        for (int m = 0; m < kScanPer; ++m) sum_eq += s_eq[mine + m];
        uint32_t total_eq, total_keep;
        uint32_t tie_rank = carry_eq + block_excl_scan_n<kScanBlock>(sum_eq, total_eq);
        uint32_t sum_keep = 0;
#pragma unroll
        for (int m = 0; m < kScanPer; ++m) {
            const uint32_t e = s_eq[mine + m];
            const uint32_t take = all_ties ? e : (tie_rank >= k3 ? 0u : min(e, k3 - tie_rank));
            s_eq[mine + m] = tie_rank;
            tie_rank += e;
            const uint32_t keep = s_gt[mine + m] + take;
            s_gt[mine + m] = keep;
            sum_keep += keep;
        }
        uint32_t off = carry_keep + block_excl_scan_n<kScanBlock>(sum_keep, total_keep);
#pragma unroll
        for (int m = 0; m < kScanPer; ++m) {
            const uint32_t keep = s_gt[mine + m];
            s_gt[mine + m] = off;
            off += keep;
        }
        __syncthreads();
#pragma unroll
        for (int m = 0; m < kScanPer; ++m) {
            const int i = m * kScanBlock + threadIdx.x;
            const int64_t t = c0 + i;
            if (t < nt4k) {
                const uint32_t o = s_gt[scan_slot(i)];
                eq[t] = s_eq[scan_slot(i)];
                gt[t] = o;
                if (t % kTilesPerBlock == 0) fin[t / kTilesPerBlock] = o;
            }
        }
        carry_eq += total_eq;
        carry_keep += total_keep;
        __syncthreads();
    }
}

__device__ __forceinline__ uint32_t lowest_set_bits(uint32_t word, uint32_t count)
{
    uint32_t m = 0;
    for (uint32_t t = 0; t < count && word; ++t) {
        const uint32_t lb = word & (0u - word);
        m |= lb;
        word ^= lb;
    }
    return m;
}

// ------------------------------------------------------------------------------------
// Ties (rows whose guess failed): keep those of global rank < k3 in index order (only if
// not all are kept), then count the kept coordinates of every tile.  A thread owns 4
// consecutive bitmap words.  grid = (blocks, rows), blocks loop over the spans.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBlock)
k_topk_ties(const Sel *__restrict__ sel_all, const uint32_t *__restrict__ hit,
            uint32_t *__restrict__ bm_in_all,
            const uint32_t *__restrict__ bm_cand_all, const uint32_t *__restrict__ tie_off_all,
            uint32_t *__restrict__ cnt_fin_all, int64_t wp, int64_t nbt, unsigned int *tick)
{
    const int row = blockIdx.y;
    if (hit[row]) return;                             // rows with lists have no bitmaps
    uint32_t *bm_in = bm_in_all + (int64_t)row * wp;
    const uint32_t *bm_tie = bm_cand_all + (int64_t)row * wp;
    const Sel s = sel_all[row];
    for (int64_t bx = blockIdx.x; bx < nbt; bx += gridDim.x) {       // block-uniform
    const int64_t w0 = bx * kTileWords + threadIdx.x * 4;
    uint32_t keep[4], tie[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        keep[m] = w0 + m < wp ? bm_in[w0 + m] : 0u;
        tie[m] = w0 + m < wp ? bm_tie[w0 + m] : 0u;
    }
    if (s.k3 != s.c3) {                               // block-uniform
        const uint32_t mine = __popc(tie[0]) + __popc(tie[1]) + __popc(tie[2]) + __popc(tie[3]);
        uint32_t total;
        uint32_t rank = block_excl_scan(mine, total) + tie_off_all[(int64_t)row * nbt + bx];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            if (tie[m] && rank < s.k3) {
                keep[m] |= lowest_set_bits(tie[m], s.k3 - rank);
                bm_in[w0 + m] = keep[m];
            }
            rank += __popc(tie[m]);
        }
    }
    uint32_t total;
    block_excl_scan(__popc(keep[0]) + __popc(keep[1]) + __popc(keep[2]) + __popc(keep[3]), total);
    if (threadIdx.x == 0) cnt_fin_all[(int64_t)row * nbt + bx] = total;
    }
    if (tick && last_block_of_row(tick + row, gridDim.x)) scan_row(cnt_fin_all + (int64_t)row * nbt, nbt, nullptr, true);
}

// ------------------------------------------------------------------------------------
// Ordered compaction into the payload (indices increasing).  grid = (nbt, rows).
// Rows with lists: a warp walks its tile's list in order; an entry is kept if its key is
// above T, or equal to T with tie rank below k3; positions come from ballots, and the value
// is written with the index.  Other rows: from the selection bitmap; a thread owns 4
// consecutive bitmap words, ranks come from popcount scans, values follow in k_topk_gather.
// ------------------------------------------------------------------------------------
// What the compaction does besides writing the payload.  b_rw != NULL: b_j += u_j at the kept
// coordinates (rows x stride floats, the same array the selection subtracted), unless the row
// defers it (pending != NULL and the row was selected from lists: pending[row] = 1 and the
// next dense pass applies the payload).  classic_values: rows whose guess failed get their
// values (u_j = a_j - b_j, read here) and their update in this kernel too; without it only
// their coordinates are written and k_topk_gather follows.
struct EmitUpdate {
    float *b_rw;
    uint32_t *pending;
    int classic_values;
    uint32_t *hist_clear;             // rows x kHistStride, or NULL: the row's histograms, cleared for the next selection
};

template <bool HAS_B>
__global__ void __launch_bounds__(kBlock)
k_topk_emit_idx(const float *__restrict__ a_all, const float *__restrict__ b_all,
                const uint32_t *__restrict__ bm_in_all, const uint32_t *__restrict__ fin_off_all,
                const uint32_t *__restrict__ hit, const Sel *__restrict__ sel_all,
                const float *__restrict__ stash_all, const uint16_t *__restrict__ stash_pos_all,
                const uint32_t *__restrict__ stash_cnt_all, const uint32_t *__restrict__ cnt_gt_all,
                const uint32_t *__restrict__ cnt_eq_all, uint32_t *__restrict__ idx_all,
                float *__restrict__ val_all, int64_t wp, int64_t nbt, int64_t k, int64_t nt4k, int64_t d, int64_t stride,
                int kind, EmitUpdate upd)
{
    const int row = blockIdx.y;
    if (!(kind & (hit[row] ? kRowsListed : kRowsClassic))) return;
    // Nothing reads the row's histograms after the scans before this kernel: the row's first
    // block leaves them zero for the next selection (which then needs no memset of its own in
    // front of its dense pass).
    if (upd.hist_clear && blockIdx.x == 0)
        for (int t = threadIdx.x; t < kHistStride; t += kBlock) upd.hist_clear[(int64_t)row * kHistStride + t] = 0u;
    uint32_t *idx = idx_all + (int64_t)row * k;
    float *val = val_all + (int64_t)row * k;
    float *b_rw = upd.b_rw ? upd.b_rw + (int64_t)row * stride : nullptr;
    // a row selected from lists may leave its state update to the next selection's dense pass
    const bool deferred = upd.pending != nullptr && hit[row] != 0u;
    if (upd.pending && blockIdx.x == 0 && threadIdx.x == 0) upd.pending[row] = deferred ? 1u : 0u;
    if (hit[row]) {
        if ((int64_t)blockIdx.x * kListTiles >= nt4k) return;
        const WarpLists w = warp_lists(stash_all, stash_pos_all, stash_cnt_all, row, nt4k, d);
        const float *a = a_all + (int64_t)row * stride;
        const float *b = HAS_B ? b_all + (int64_t)row * stride : nullptr;
        const Sel s = sel_all[row];
        const uint32_t T = (s.b1 << 20) | (s.b2 << 9) | s.b3;
        const bool all_ties = s.k3 == s.c3;
        const uint32_t lane = threadIdx.x & 31;
        const uint32_t lt = (1u << lane) - 1u;
        float v[kWarpTiles][kPre];
        uint32_t ps[kWarpTiles][kPre], out[kWarpTiles], tie_rank[kWarpTiles];
#pragma unroll
        for (int m = 0; m < kWarpTiles; ++m) {
            const int64_t g = (int64_t)row * nt4k + (w.tile[m] < nt4k ? w.tile[m] : 0);
            out[m] = cnt_gt_all[g];
            tie_rank[m] = cnt_eq_all[g];
#pragma unroll
            for (int i = 0; i < kPre; ++i) {
                v[m][i] = w.val[m][lane + 32 * i];       // fetched whatever the length (see for_each_listed)
                ps[m][i] = w.pos[m][lane + 32 * i];
            }
        }
#pragma unroll
        for (int m = 0; m < kWarpTiles; ++m) {
            const uint32_t base = (uint32_t)(w.tile[m] * kSub);
            // one chunk of 32 entries in index order: ballots give the tie ranks and the
            // payload positions
            auto chunk = [&](bool valid, float val_e, uint32_t pos_e) {
                const uint32_t key = key_of(val_e);
                const bool eq = valid && key == T;
                const uint32_t eqm = __ballot_sync(kFull, eq);
                const bool keep = valid && (key > T || (eq && (all_ties || tie_rank[m] + __popc(eqm & lt) < s.k3)));
                const uint32_t km = __ballot_sync(kFull, keep);
                const uint32_t at = out[m] + __popc(km & lt);
                if (keep && at < k) {
                    idx[at] = base + pos_e;
                    val[at] = val_e;
                    if (b_rw && !deferred) b_rw[base + pos_e] = __fadd_rn(b_rw[base + pos_e], val_e);   // b += u (Algorithm 1)
                }
                out[m] += __popc(km);
                tie_rank[m] += __popc(eqm);
            };
#pragma unroll
            for (int i = 0; i < kPre; ++i)
                if (32u * i < w.cnt[m]) chunk(lane + 32 * i < w.cnt[m], v[m][i], ps[m][i]);       // warp-uniform
            for (uint32_t e0 = 32 * kPre; e0 < w.cnt[m]; e0 += 32) {
                const uint32_t e = e0 + lane;
                const bool valid = e < w.cnt[m];
                chunk(valid, valid ? w.val[m][e] : 0.0f, valid ? (uint32_t)w.pos[m][e] : 0u);
            }
            for (uint32_t e0 = 0; e0 < w.dense[m]; e0 += 32) {              // a tile without a list
                const uint32_t e = e0 + lane;
                const bool valid = e < w.dense[m];
                chunk(valid, valid ? diff1<HAS_B>(a, b, w.tile[m] * kSub + e) : 0.0f, e);
            }
        }
        return;
    }
    const uint32_t *bm_in = bm_in_all + (int64_t)row * wp;
    const int64_t w0 = (int64_t)blockIdx.x * kTileWords + threadIdx.x * 4;
    uint32_t keep[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) keep[m] = w0 + m < wp ? bm_in[w0 + m] : 0u;
    uint32_t total;
    uint32_t rank = block_excl_scan(__popc(keep[0]) + __popc(keep[1]) + __popc(keep[2]) + __popc(keep[3]), total) +
                    fin_off_all[(int64_t)row * nbt + blockIdx.x];
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        uint32_t word = keep[m];
        while (word) {
            const int bit = __ffs(word) - 1;
            word &= word - 1;
            const int64_t j = (w0 + m) * 32 + bit;
            if (rank < k) {
                idx[rank] = (uint32_t)j;
                if (upd.classic_values) {             // the value u_j and the state update with it
                    const float aj = a_all[(int64_t)row * stride + j];
                    if (HAS_B) {
                        // (read through the writable pointer where there is one: this kernel writes b)
                        const float bj = b_rw ? b_rw[j] : b_all[(int64_t)row * stride + j];
                        const float u = __fsub_rn(aj, bj);
                        val[rank] = u;
                        if (b_rw) b_rw[j] = __fadd_rn(bj, u);
                    } else {
                        val[rank] = aj;
                    }
                }
            }
            ++rank;
        }
    }
}

// ------------------------------------------------------------------------------------
// Payload values and the state update at the kept coordinates (Algorithm 1: ghat^(i) += c^(i), gtil += c):
// val = u_j = a_j - b_j, b_j += u_j.  One thread per payload entry.  grid = (ceil(k/256), rows).
// Rows whose values were already written from the lists only update b.
// ------------------------------------------------------------------------------------
template <bool HAS_B, bool UPDATE_B>
__global__ void __launch_bounds__(kBlock)
k_topk_gather(const float *__restrict__ a_all, float *__restrict__ b_all,
              const uint32_t *__restrict__ idx_all, float *__restrict__ val_all,
              const uint32_t *__restrict__ have_val, int64_t d, int64_t k, int64_t stride,
              uint32_t *__restrict__ pending)
{
    const int row = blockIdx.y;
    // deferred state update: a row selected from lists (values already in the payload) keeps
    // its update for the next selection's dense pass
    const bool deferred = pending && have_val[row];
    if (pending && blockIdx.x == 0 && threadIdx.x == 0) pending[row] = deferred ? 1u : 0u;
    if (deferred) return;
    const float *a = a_all + (int64_t)row * stride;
    // (a grid smaller than the payload loops: where most rows defer, few blocks are launched)
    for (int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x; t < k; t += (int64_t)gridDim.x * kBlock) {
        const int64_t j = idx_all[(int64_t)row * k + t];
        if (j >= d) continue;                 // caller-supplied sets are checked separately
        if (have_val && have_val[row]) {      // the payload values were written with the indices
            if (HAS_B && UPDATE_B) {
                float *b = b_all + (int64_t)row * stride;
                b[j] = __fadd_rn(b[j], val_all[(int64_t)row * k + t]);
            }
            continue;
        }
        float u;
        if (HAS_B) {
            float *b = b_all + (int64_t)row * stride;
            const float bj = b[j];
            u = __fsub_rn(a[j], bj);
            if (UPDATE_B) b[j] = __fadd_rn(bj, u);
        } else {
            u = a[j];
        }
        val_all[(int64_t)row * k + t] = u;
    }
}

// Applies the payloads whose state update is still pending: b_j += u_j at the kept
// coordinates of every row with pending[row] != 0.  grid = (ceil(k/256), rows).  The flags are
// cleared by the caller afterwards.
__global__ void __launch_bounds__(kBlock)
k_topk_apply_pending(float *__restrict__ b_all, const uint32_t *__restrict__ idx_all,
                     const float *__restrict__ val_all, const uint32_t *__restrict__ pending, int64_t d,
                     int64_t k, int64_t stride)
{
    const int row = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t >= k || !pending[row]) return;
    const int64_t j = idx_all[(int64_t)row * k + t];
    if (j >= d) return;
    float *b = b_all + (int64_t)row * stride;
    b[j] = __fadd_rn(b[j], val_all[(int64_t)row * k + t]);
}

// ------------------------------------------------------------------------------------
// Sparse server aggregation (Algorithm 1): ghat_s += (sum_i c_i) / n.
//
// A block owns kAggSpan consecutive coordinates and keeps their sums in shared memory.
// Every payload is sorted by index, so worker i's entries for the block are one contiguous
// range found by binary search.  Workers are added one after the other (barrier between
// them), so each coordinate sees the binary32 sum in the order 0, 1, ..., n-1; the indices
// inside one payload are distinct, so no atomics are needed.  grid = ceil(d / kAggSpan).
// ------------------------------------------------------------------------------------
constexpr int kAggSpan = 8192;

__device__ __forceinline__ int64_t lower_bound_u32(const uint32_t *p, int64_t count, uint32_t key)
{
    int64_t lo = 0, hi = count;
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (p[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

constexpr int kAggChunk = 64;      // workers whose entry ranges are searched at once
constexpr int kAggPre = 16;        // workers whose first 256 entries are fetched before they are added

__global__ void __launch_bounds__(kBlock)
k_topk_aggregate(const uint32_t *__restrict__ idx_all, const float *__restrict__ val_all,
                 const uint32_t *__restrict__ fin_off_all, int64_t nbt, int n, int64_t k, int64_t d,
                 float *__restrict__ ghat_s, int n_pow2, const uint32_t *__restrict__ hit,
                 const uint32_t *__restrict__ tile_off_all, int64_t nt4k)
{
    __shared__ __align__(16) float acc[kAggSpan];
    __shared__ int64_t range[kAggChunk][2];
    const int64_t base = (int64_t)blockIdx.x * kAggSpan;
    const int64_t end = min(base + (int64_t)kAggSpan, d);
    const int64_t tile = base / (kTileWords * 32);          // compaction tile of this span
    for (int t = threadIdx.x; t < kAggSpan; t += kBlock) acc[t] = 0.0f;
    for (int i0 = 0; i0 < n; i0 += kAggChunk) {
        const int nc = min(kAggChunk, n - i0);
        __syncthreads();
        if (threadIdx.x < 2 * nc) {
            // entries of worker i inside [base, end): searched only among its entries of the
            // enclosing compaction tile, whose bounds are the scanned tile counts
            const int i = i0 + (threadIdx.x >> 1), side = threadIdx.x & 1;
            const uint32_t *idx = idx_all + (int64_t)i * k;
            int64_t pos;
            if (fin_off_all && hit[i] && base + kAggSpan <= d) {
                // rows selected from lists have the payload offset of every 4096-coordinate
                // tile: the span's entries are known without a search
                const int64_t t4 = (side == 0 ? base : end) / kSub;
                pos = t4 < nt4k ? (int64_t)tile_off_all[(int64_t)i * nt4k + t4] : k;
            } else {
                int64_t t_lo = 0, t_hi = k;   // without tile counts (rand-k): the whole payload
                if (fin_off_all) {
                    t_lo = fin_off_all[(int64_t)i * nbt + tile];
                    t_hi = tile + 1 < nbt ? (int64_t)fin_off_all[(int64_t)i * nbt + tile + 1] : k;
                }
                pos = t_hi;
                if (!fin_off_all || side == 0 || end < (tile + 1) * (int64_t)(kTileWords * 32))
                    pos = (side == 1 && end >= ((int64_t)1 << 32))
                              ? min(t_hi, k)
                              : t_lo + lower_bound_u32(idx + t_lo, min(t_hi, k) - t_lo, (uint32_t)(side == 0 ? base : end));
            }
            range[threadIdx.x >> 1][side] = min(pos, k);
        }
        __syncthreads();
        // The additions are ordered by worker (a barrier after each), so their operands are
        // fetched beforehand, kAggPre workers at a time: the loads of all of them are in
        // flight together instead of one memory latency per worker.
        for (int c0 = 0; c0 < nc; c0 += kAggPre) {
            uint32_t pe[kAggPre];
            float pv[kAggPre];
#pragma unroll
            for (int u = 0; u < kAggPre; ++u) {
                pe[u] = 0xffffffffu;
                pv[u] = 0.0f;
                if (c0 + u < nc) {
                    const int64_t t = range[c0 + u][0] + threadIdx.x;
                    if (t < range[c0 + u][1]) {
                        pe[u] = idx_all[(int64_t)(i0 + c0 + u) * k + t] - (uint32_t)base;
                        pv[u] = val_all[(int64_t)(i0 + c0 + u) * k + t];
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kAggPre; ++u) {                 // workers in increasing order
                if (c0 + u >= nc) break;                        // block-uniform
                if (pe[u] < (uint32_t)kAggSpan) acc[pe[u]] = __fadd_rn(acc[pe[u]], pv[u]);
                const uint32_t *idx = idx_all + (int64_t)(i0 + c0 + u) * k;
                const float *val = val_all + (int64_t)(i0 + c0 + u) * k;
                const int64_t hi = range[c0 + u][1];
                for (int64_t t = range[c0 + u][0] + kBlock + threadIdx.x; t < hi; t += kBlock) {   // dense payloads
                    const uint32_t e = idx[t] - (uint32_t)base;
                    if (e < (uint32_t)kAggSpan) acc[e] = __fadd_rn(acc[e], val[t]);
                }
                __syncthreads();
            }
        }
    }
    const float fn = (float)n, rn = 1.0f / fn;
    auto mean = [&](float a) { return n_pow2 ? __fmul_rn(a, rn) : __fdiv_rn(a, fn); };
    if (end - base == kAggSpan && ((uintptr_t)ghat_s & 15u) == 0) {
        // all loads of the span first (independent), then the additions: a loop of
        // read-modify-writes of one array would wait for each store before the next load
        constexpr int kPer = kAggSpan / 4 / kBlock;
        float4 G[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u)
            G[u] = *reinterpret_cast<const float4 *>(ghat_s + base + (int64_t)(u * kBlock + threadIdx.x) * 4);
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const int t = (u * kBlock + threadIdx.x) * 4;
            const float4 a = *reinterpret_cast<const float4 *>(&acc[t]);
            if (a.x != 0.0f || a.y != 0.0f || a.z != 0.0f || a.w != 0.0f) {     // adding an exact zero changes nothing
                if (a.x != 0.0f) G[u].x = __fadd_rn(G[u].x, mean(a.x));
                if (a.y != 0.0f) G[u].y = __fadd_rn(G[u].y, mean(a.y));
                if (a.z != 0.0f) G[u].z = __fadd_rn(G[u].z, mean(a.z));
                if (a.w != 0.0f) G[u].w = __fadd_rn(G[u].w, mean(a.w));
                *reinterpret_cast<float4 *>(ghat_s + base + t) = G[u];
            }
        }
        return;
    }
    for (int t = threadIdx.x; t < (int)(end - base); t += kBlock) {
        const float a = acc[t];
        if (a != 0.0f) ghat_s[base + t] = __fadd_rn(ghat_s[base + t], mean(a));
    }
}

// ------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------
static void free_ws(TopkWorkspace *w)
{
    cudaFree(w->hist); cudaFree(w->sel); cudaFree(w->bm_in); cudaFree(w->bm_cand);
    cudaFree(w->cnt_tie); cudaFree(w->cnt_fin);
    cudaFree(w->floor_bucket); cudaFree(w->hit); cudaFree(w->stash);
    cudaFree(w->stash_pos); cudaFree(w->stash_cnt); cudaFree(w->cnt_gt); cudaFree(w->cnt_eq);
    cudaFree(w->pending); cudaFree(w->cand); cudaFree(w->tick);
    if (w->side) cudaStreamDestroy(w->side);
    if (w->ev_fork) cudaEventDestroy(w->ev_fork);
    if (w->ev_join) cudaEventDestroy(w->ev_join);
    if (w->own_payload) { cudaFree(w->idx); cudaFree(w->val); }
    delete w;
}

int topk_workspace_create(TopkWorkspace **out, int64_t d, int64_t k, int rows, uint32_t *idx,
                          float *val, bool with_select, int64_t stride)
{
    *out = nullptr;
    TopkWorkspace *w = new TopkWorkspace();
    memset(w, 0, sizeof *w);
    w->d = d; w->k = k; w->rows = rows;
    w->stride = stride > 0 ? stride : d;
    w->wp = (d + 31) / 32;
    w->nbt = (w->wp + kTileWords - 1) / kTileWords;
    w->own_payload = idx == nullptr;
    w->idx = idx; w->val = val;
    w->wait_limit = kWaitLimit;
    bool ok = true;
    auto get = [&](void **p, size_t bytes) {
        *p = nullptr;
        if (ok && (cudaMalloc(p, bytes) != cudaSuccess || cudaMemset(*p, 0, bytes) != cudaSuccess)) ok = false;
    };
    if (with_select) {
        get((void **)&w->hist, (size_t)rows * kHistStride * 4);
        get((void **)&w->sel, (size_t)rows * sizeof(Sel));
        get((void **)&w->bm_in, (size_t)rows * w->wp * 4);
        get((void **)&w->bm_cand, (size_t)rows * w->wp * 4);
        get((void **)&w->floor_bucket, (size_t)rows * 4);
        get((void **)&w->hit, (size_t)rows * 4);
        w->nt4k = (d + kSub - 1) / kSub;
        get((void **)&w->stash, (size_t)rows * w->nt4k * kStashCap * 4);
        get((void **)&w->stash_pos, (size_t)rows * w->nt4k * kStashCap * 2);
        get((void **)&w->stash_cnt, (size_t)rows * w->nt4k * 4);
        get((void **)&w->cnt_gt, (size_t)rows * w->nt4k * 4);
        get((void **)&w->cnt_eq, (size_t)rows * w->nt4k * 4);
        if (ok && cudaMemset(w->floor_bucket, 0xff, (size_t)rows * 4) != cudaSuccess) ok = false;   // no guess yet
        get((void **)&w->cnt_tie, (size_t)rows * w->nbt * 4);
        get((void **)&w->cnt_fin, (size_t)rows * w->nbt * 4);
        get((void **)&w->pending, (size_t)rows * 4);
        get((void **)&w->cand, (size_t)rows * w->nt4k * 4 * sizeof(uint16_t));
        get((void **)&w->tick, (size_t)rows * 5 * sizeof(unsigned int));
        if (ok && (cudaStreamCreateWithFlags(&w->side, cudaStreamNonBlocking) != cudaSuccess ||
                   cudaEventCreateWithFlags(&w->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                   cudaEventCreateWithFlags(&w->ev_join, cudaEventDisableTiming) != cudaSuccess)) ok = false;
    }
    if (w->own_payload) {
        get((void **)&w->idx, (size_t)rows * k * 4);
        get((void **)&w->val, (size_t)rows * k * 4);
    }
    if (!ok) { cudaGetLastError(); free_ws(w); return CDADAM_ERR_ALLOC; }
    *out = w;
    return CDADAM_OK;
}

void topk_workspace_destroy(TopkWorkspace *w) { if (w) free_ws(w); }

void topk_workspace_set_error_flag(TopkWorkspace *w, int *error_flag) { if (w) w->error_flag = error_flag; }

void topk_workspace_set_ring(TopkWorkspace *w, int ring) { if (w) w->ring = ring; }

void topk_workspace_set_defer(TopkWorkspace *w, bool on) { if (w && w->pending) w->defer = on; }

void topk_flush(TopkWorkspace *w, float *b, cudaStream_t st)
{
    if (!w || !w->defer) return;
    const dim3 entries((unsigned)((w->k + kBlock - 1) / kBlock), (unsigned)w->rows);
    k_topk_apply_pending<<<entries, kBlock, 0, st>>>(b, w->idx, w->val, w->pending, w->d, w->k, w->stride);
    cudaMemsetAsync(w->pending, 0, (size_t)w->rows * 4, st);
}

void topk_forget_pending(TopkWorkspace *w, cudaStream_t st)
{
    if (w && w->defer) cudaMemsetAsync(w->pending, 0, (size_t)w->rows * 4, st);
}

void topk_workspace_set_wait_limit(TopkWorkspace *w, int polls) { if (w) w->wait_limit = polls < 0 ? kWaitLimit : polls; }

void topk_payload(TopkWorkspace *w, int row, const uint32_t **idx, const float **val)
{
    *idx = w->idx + (int64_t)row * w->k;
    *val = w->val + (int64_t)row * w->k;
}

constexpr int kSelectLaunches = 11;      // dense pass, pick, six for the classic chain, three for the listed chain
int topk_launches_per_step(int) { return 2 * kSelectLaunches; }    // two selections; the aggregation kernel is counted by the caller

// Whole tiles per row that the dense pass takes through the prefetch ring (0: none).
static int64_t ring_tiles(const TopkWorkspace *w, bool vec_ok)
{
    const bool ring_ok = vec_ok && w->stride % 4 == 0 && w->ring >= 0 &&
                         (w->ring > 0 || (int64_t)w->rows * (w->d / kSub) >= 32768);
    return ring_ok ? w->d / kSub : 0;
}

// Kernels of the dense pass: the ring kernel and the plain one share it when the ring takes
// the whole tiles and a ragged last tile remains.
int topk_dense_launches(const TopkWorkspace *w, bool vec_ok)
{
    const int64_t full = ring_tiles(w, vec_ok);
    return full > 0 && full < w->nt4k ? 2 : 1;
}

template <bool HAS_B>
static void select_impl(TopkWorkspace *w, const float *a, float *b, bool update_b, bool vec_ok,
                        cudaStream_t st, const Agg *agg = nullptr, float *a_rw = nullptr)
{
    const dim3 dense((unsigned)((w->d + kSub - 1) / kSub), (unsigned)w->rows);
    const dim3 sparse((unsigned)w->nbt, (unsigned)w->rows);
    // (the histograms are zero: from the allocation, then from the previous selection's compaction)
    // one dense pass with the guessed floor; the two classic passes (small looping grids)
    // do work only for rows whose guess failed
    const dim3 fallback(std::min(dense.x, std::max(148u, 148u * 4u / (unsigned)w->rows)), (unsigned)w->rows);
    // whole tiles through the prefetch ring where rows are 16-byte aligned and there are
    // tiles enough to fill the device several times over with its three blocks of seven tiles
    // per SM (measured: 16 x 6250 tiles 0.50 -> 0.47 ms, 1 x 6250 tiles 0.039 -> 0.047 ms);
    // the ragged last tile, or everything else, through the plain kernel
    const int64_t full_tiles = agg ? 0 : ring_tiles(w, vec_ok);      // the fused aggregation lives in the plain kernel
    // deferred state update: the dense pass first applies the previous selection's payload
    const bool defer = HAS_B && update_b && w->defer;
    const Pending pd = {w->pending, w->idx, w->val, w->cnt_gt, w->k};
    if (full_tiles > 0) {
        constexpr int kBytes = kSpecStages * (HAS_B ? 2 : 1) * kSub * (int)sizeof(float);
        auto kern = defer ? k_topk_spec_ring<HAS_B, HAS_B> : k_topk_spec_ring<HAS_B, false>;
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBytes);
        const dim3 groups((unsigned)((full_tiles + kSpecTiles - 1) / kSpecTiles), (unsigned)w->rows);
        kern<<<groups, kBlock, kBytes, st>>>(a, b, w->floor_bucket, w->hist, w->stash, w->stash_pos, w->stash_cnt,
                                            full_tiles, w->stride, w->nt4k, w->error_flag, w->wait_limit, pd);
    }
    if (full_tiles < w->nt4k) {
        const dim3 rest((unsigned)(w->nt4k - full_tiles), (unsigned)w->rows);
        auto kern = agg ? k_topk_spec<HAS_B, false, HAS_B> : defer ? k_topk_spec<HAS_B, HAS_B, false> : k_topk_spec<HAS_B, false, false>;
        kern<<<rest, kBlock, 0, st>>>(a, b, w->floor_bucket, w->hist, w->stash, w->stash_pos, w->stash_cnt, w->d, vec_ok,
                                     w->stride, full_tiles, w->nt4k, pd, agg ? *agg : Agg{}, a_rw);
    }
    k_topk_pick_spec<<<w->rows, kBlock, 0, st>>>(w->hist, w->sel, (uint32_t)w->k, w->floor_bucket, w->hit);
    // From here two chains run side by side (under stream capture: two branches of the graph).
    // Rows whose guess failed (none, in the steady state: six launches that find nothing to do;
    // every pick and scan is done by the block that finishes its row last) take the classic
    // passes on the side stream ...
    const dim3 fallback_sparse(std::min(sparse.x, fallback.x), (unsigned)w->rows);
    // values, state update (or its deferral) happen inside the ordered compaction
    const EmitUpdate upd = {HAS_B && update_b ? b : nullptr, defer ? w->pending : nullptr, 1, w->hist};
    cudaStream_t sd = w->side;
    cudaEventRecord(w->ev_fork, st);
    cudaStreamWaitEvent(sd, w->ev_fork, 0);
    const uint32_t k32 = (uint32_t)w->k;
    auto tail = [&](int pass) { return RowTail{w->tick + (size_t)pass * w->rows, w->sel, w->floor_bucket, k32}; };
    k_topk_hist1<HAS_B><<<fallback, kBlock, 0, sd>>>(a, b, w->hist, w->hit, w->d, vec_ok, w->stride, tail(0));
    k_topk_mark<HAS_B><<<fallback, kBlock, 0, sd>>>(a, b, w->sel, w->bm_in, w->bm_cand, w->hist, w->hit, w->d, w->wp, vec_ok, w->stride, tail(1));
    k_topk_hist3<HAS_B><<<fallback_sparse, kBlock, 0, sd>>>(a, b, w->sel, w->hit, w->bm_cand, w->hist, w->wp, w->nbt, w->stride, tail(2));
    k_topk_resolve<HAS_B><<<sparse, kBlock, 0, sd>>>(a, b, w->sel, w->hit, w->bm_in, w->bm_cand, w->cnt_tie, w->wp, w->nbt, w->stride, w->tick + (size_t)3 * w->rows);
    k_topk_ties<<<fallback_sparse, kBlock, 0, sd>>>(w->sel, w->hit, w->bm_in, w->bm_cand, w->cnt_tie, w->cnt_fin, w->wp, w->nbt, w->tick + (size_t)4 * w->rows);
    k_topk_emit_idx<HAS_B><<<sparse, kBlock, 0, sd>>>(a, b, w->bm_in, w->cnt_fin, w->hit, w->sel, w->stash, w->stash_pos, w->stash_cnt, w->cnt_gt, w->cnt_eq, w->idx, w->val, w->wp, w->nbt, w->k, w->nt4k, w->d, w->stride, kRowsClassic, upd);
    cudaEventRecord(w->ev_join, sd);
    // ... and the rows selected from the dense pass's lists take three launches on this one
    // (queued the ordinary way: with programmatic dependent launch from the pick to the
    // compaction the worker stage of 16 x 25.6 M measured 0.675 ms against 0.664)
    k_topk_split<HAS_B><<<sparse, kBlock, 0, st>>>(a, b, w->sel, w->hit, w->stash, w->stash_pos, w->stash_cnt, w->hist, w->cnt_gt, w->cnt_eq, w->cand, w->nt4k, w->d, w->stride);
    cudaFuncSetAttribute(k_scan_lists<HAS_B>, cudaFuncAttributeMaxDynamicSharedMemorySize, kScanSmemBytes);
    k_scan_lists<HAS_B><<<w->rows, kScanBlock, kScanSmemBytes, st>>>(a, b, w->sel, w->hit, w->hist, w->floor_bucket, w->stash, w->stash_cnt, w->cand, w->cnt_gt, w->cnt_eq, w->cnt_fin, w->nt4k, w->nbt, w->d, w->stride);
    k_topk_emit_idx<HAS_B><<<sparse, kBlock, 0, st>>>(a, b, w->bm_in, w->cnt_fin, w->hit, w->sel, w->stash, w->stash_pos, w->stash_cnt, w->cnt_gt, w->cnt_eq, w->idx, w->val, w->wp, w->nbt, w->k, w->nt4k, w->d, w->stride, kRowsListed, upd);
    cudaStreamWaitEvent(st, w->ev_join, 0);
}

// ------------------------------------------------------------------------------------
// Coordinate-sharded selection.  Several workspaces, one per coordinate range of the same
// rows, select the k largest of the WHOLE rows between them: the classic three levels, every
// histogram summed over the ranges before its pick (integer sums: any order gives the same
// threshold on every range), then the ties given out in coordinate order, i.e. in the order
// of the ranges: range r takes those of the k3 ties that the ranges before it left.
// The sums and counts travel through an exchange buffer of ranges x rows x kBins1 words:
// a stage writes this range's slot, the caller gathers the slots of all ranges in place,
// the next stage reads them all.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBlock)
k_range_hist_out(const uint32_t *__restrict__ hist_all, int level_off, int bins, uint32_t *__restrict__ slot)
{
    const int row = blockIdx.y, t = blockIdx.x * kBlock + threadIdx.x;
    if (t < bins) slot[(int64_t)row * kBins1 + t] = hist_all[(int64_t)row * kHistStride + level_off + t];
}

__global__ void __launch_bounds__(kBlock)
k_range_hist_sum(const uint32_t *__restrict__ x_all, int ranges, int rows, int level_off, int bins,
                 uint32_t *__restrict__ hist_all)
{
    const int row = blockIdx.y, t = blockIdx.x * kBlock + threadIdx.x;
    if (t >= bins) return;
    uint32_t sum = 0u;
    for (int r = 0; r < ranges; ++r) sum += x_all[((int64_t)r * rows + row) * kBins1 + t];
    hist_all[(int64_t)row * kHistStride + level_off + t] = sum;
}

// The ties this range may keep: k3 minus the ties of the ranges before it, at most its own.
// A row that keeps all ties (k3 == c3) is left alone.  One thread per row.
__global__ void k_range_ties_share(Sel *__restrict__ sel_all, const uint32_t *__restrict__ x_all, int range,
                                   int rows)
{
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    Sel *s = sel_all + row;
    if (s->k3 == s->c3) return;
    uint32_t before = 0u;
    for (int r = 0; r < range; ++r) before += x_all[((int64_t)r * rows + row) * kBins1];
    const uint32_t own = x_all[((int64_t)range * rows + row) * kBins1];
    const uint32_t share = before >= s->k3 ? 0u : min(own, s->k3 - before);
    s->k3 = share;
    s->c3 = 0xffffffffu;              // != k3: the ordered pick of the ties runs
}

// Payload entries beyond the range's own count are marked with the coordinate 0xffffffff
// (no vector has it: d < 2^32), which every later pass over a payload skips.
__global__ void __launch_bounds__(kBlock)
k_range_pad(uint32_t *__restrict__ idx_all, float *__restrict__ val_all, const uint32_t *__restrict__ count, int64_t k)
{
    const int row = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t < k && t >= (int64_t)count[row]) {
        idx_all[(int64_t)row * k + t] = 0xffffffffu;
        val_all[(int64_t)row * k + t] = 0.0f;
    }
}

template <bool HAS_B>
static void range_stage_impl(TopkWorkspace *w, int stage, const float *a, float *b, bool vec_ok, int64_t k_all,
                             uint32_t *x, int range, int ranges, cudaStream_t st)
{
    const dim3 dense((unsigned)((w->d + kSub - 1) / kSub), (unsigned)w->rows);
    const dim3 sparse((unsigned)w->nbt, (unsigned)w->rows);
    const dim3 fallback(std::min(dense.x, std::max(148u, 148u * 4u / (unsigned)w->rows)), (unsigned)w->rows);
    const dim3 fallback_sparse(std::min(sparse.x, fallback.x), (unsigned)w->rows);
    const dim3 bins((kBins1 + kBlock - 1) / kBlock, (unsigned)w->rows);
    uint32_t *mine = x + (int64_t)range * w->rows * kBins1;
    auto out = [&](int off, int nb) { k_range_hist_out<<<bins, kBlock, 0, st>>>(w->hist, off, nb, mine); };
    auto sum = [&](int off, int nb) { k_range_hist_sum<<<bins, kBlock, 0, st>>>(x, ranges, w->rows, off, nb, w->hist); };
    switch (stage) {
    case 0:       // level 1 of this range
        cudaMemsetAsync(w->hist, 0, (size_t)w->rows * kHistStride * 4, st);
        cudaMemsetAsync(w->hit, 0, (size_t)w->rows * 4, st);         // every row takes the classic passes
        k_topk_hist1<HAS_B><<<fallback, kBlock, 0, st>>>(a, b, w->hist, w->hit, w->d, vec_ok, w->stride, RowTail{});
        out(0, kBins1);
        break;
    case 1:       // level-1 bucket of the whole rows; level 2 of this range
        sum(0, kBins1);
        k_topk_pick<<<w->rows, kBlock, 0, st>>>(w->hist, w->sel, 0, (uint32_t)k_all, w->hit, w->floor_bucket);
        k_topk_mark<HAS_B><<<fallback, kBlock, 0, st>>>(a, b, w->sel, w->bm_in, w->bm_cand, w->hist, w->hit, w->d, w->wp, vec_ok, w->stride, RowTail{});
        out(kBins1, kBins2);
        break;
    case 2:
        sum(kBins1, kBins2);
        k_topk_pick<<<w->rows, kBlock, 0, st>>>(w->hist, w->sel, 1, 0, w->hit, w->floor_bucket);
        k_topk_hist3<HAS_B><<<fallback_sparse, kBlock, 0, st>>>(a, b, w->sel, w->hit, w->bm_cand, w->hist, w->wp, w->nbt, w->stride, RowTail{});
        out(kBins1 + kBins2, kBins3);
        break;
    case 3:       // the exact threshold; this range's ties
        sum(kBins1 + kBins2, kBins3);
        k_topk_pick<<<w->rows, kBlock, 0, st>>>(w->hist, w->sel, 2, 0, w->hit, w->floor_bucket);
        k_topk_resolve<HAS_B><<<sparse, kBlock, 0, st>>>(a, b, w->sel, w->hit, w->bm_in, w->bm_cand, w->cnt_tie, w->wp, w->nbt, w->stride, nullptr);
        // the row's number of ties in this range -> word 0 of the row's part of the slot
        cudaMemsetAsync(mine, 0, (size_t)w->rows * kBins1 * 4, st);
        k_scan_tiles<<<w->rows, kBlock, 0, st>>>(w->cnt_tie, w->nbt, w->hit, w->cnt_eq, false);
        cudaMemcpy2DAsync(mine, (size_t)kBins1 * 4, w->cnt_eq, 4, 4, (size_t)w->rows, cudaMemcpyDeviceToDevice, st);
        break;
    default: {    // the ties in the order of the ranges; ordered compaction; values and state update
        k_range_ties_share<<<(w->rows + 63) / 64, 64, 0, st>>>(w->sel, x, range, w->rows);
        k_scan_tiles<<<w->rows, kBlock, 0, st>>>(w->cnt_tie, w->nbt, w->hit);
        k_topk_ties<<<fallback_sparse, kBlock, 0, st>>>(w->sel, w->hit, w->bm_in, w->bm_cand, w->cnt_tie, w->cnt_fin, w->wp, w->nbt, nullptr);
        k_scan_tiles<<<w->rows, kBlock, 0, st>>>(w->cnt_fin, w->nbt, w->hit, w->cnt_eq);      // cnt_eq[row] = entries this range keeps
        k_topk_emit_idx<HAS_B><<<sparse, kBlock, 0, st>>>(a, b, w->bm_in, w->cnt_fin, w->hit, w->sel, w->stash, w->stash_pos, w->stash_cnt, w->cnt_gt, w->cnt_eq, w->idx, w->val, w->wp, w->nbt, w->k, w->nt4k, w->d, w->stride, kRowsClassic, EmitUpdate{nullptr, nullptr, 0, nullptr});
        const dim3 entries((unsigned)((w->k + kBlock - 1) / kBlock), (unsigned)w->rows);
        k_range_pad<<<entries, kBlock, 0, st>>>(w->idx, w->val, w->cnt_eq, w->k);
        k_topk_gather<HAS_B, HAS_B><<<entries, kBlock, 0, st>>>(a, b, w->idx, w->val, w->hit, w->d, w->k, w->stride, nullptr);
        break;
    }
    }
}

void topk_range_stage(TopkWorkspace *w, int stage, const float *a, float *b, bool vec_ok, int64_t k_all,
                      uint32_t *exchange, int range, int ranges, cudaStream_t st)
{
    if (b) range_stage_impl<true>(w, stage, a, b, vec_ok, k_all, exchange, range, ranges, st);
    else range_stage_impl<false>(w, stage, a, nullptr, vec_ok, k_all, exchange, range, ranges, st);
}

int64_t topk_range_exchange_words(const TopkWorkspace *w) { return (int64_t)w->rows * kBins1; }

void topk_select(TopkWorkspace *w, const float *a, float *b, bool update_b, bool vec_ok,
                 cudaStream_t st)
{
    if (b) select_impl<true>(w, a, b, update_b, vec_ok, st);
    else select_impl<false>(w, a, nullptr, false, vec_ok, st);
}

void topk_select_aggregated(TopkWorkspace *ws, TopkWorkspace *ww, float *ghat_s, float *gtil, int n, bool vec_ok,
                            cudaStream_t st)
{
    const Agg agg = {ww->idx, ww->val, ww->cnt_gt, ww->hit, ww->k, n, (n & (n - 1)) == 0 ? 1 : 0};
    select_impl<true>(ws, ghat_s, gtil, true, vec_ok, st, &agg, ghat_s);
}

// Payload of a segment into the payload of the whole vector: entries [at, at + k_seg) of every
// row, indices moved by the segment's offset.  grid = (ceil(k_seg/256), rows).
__global__ void __launch_bounds__(kBlock)
k_payload_concat(uint32_t *__restrict__ dst_idx, float *__restrict__ dst_val, int64_t k_all, int64_t at,
                 const uint32_t *__restrict__ src_idx, const float *__restrict__ src_val, int64_t k_seg,
                 uint32_t offset)
{
    const int row = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t >= k_seg) return;
    dst_idx[(int64_t)row * k_all + at + t] = src_idx[(int64_t)row * k_seg + t] + offset;
    dst_val[(int64_t)row * k_all + at + t] = src_val[(int64_t)row * k_seg + t];
}

void topk_payload_concat(TopkWorkspace *whole, int64_t at, TopkWorkspace *seg, int64_t offset, cudaStream_t st)
{
    const dim3 grid((unsigned)((seg->k + kBlock - 1) / kBlock), (unsigned)seg->rows);
    k_payload_concat<<<grid, kBlock, 0, st>>>(whole->idx, whole->val, whole->k, at, seg->idx, seg->val, seg->k,
                                              (uint32_t)offset);
}

void topk_aggregate(TopkWorkspace *ww, float *ghat_s, int n, cudaStream_t st)
{
    const unsigned blocks = (unsigned)((ww->d + kAggSpan - 1) / kAggSpan);
    k_topk_aggregate<<<blocks, kBlock, 0, st>>>(ww->idx, ww->val, ww->cnt_fin, ww->nbt, n, ww->k, ww->d, ghat_s, (n & (n - 1)) == 0,
                                                ww->hit, ww->cnt_gt, ww->nt4k);
}

void topk_aggregate_rows(const uint32_t *idx, const float *val, int64_t k, int64_t d, int n, float *ghat_s,
                         cudaStream_t st)
{
    const unsigned blocks = (unsigned)((d + kAggSpan - 1) / kAggSpan);
    k_topk_aggregate<<<blocks, kBlock, 0, st>>>(idx, val, nullptr, 0, n, k, d, ghat_s, (n & (n - 1)) == 0, nullptr, nullptr, 0);
}

// ---- rand-k: the coordinate sets come from the caller -------------------------------------
// Every row's set must be strictly increasing and below d; a violation sets *error_flag.
__global__ void __launch_bounds__(kBlock)
k_check_sets(const uint32_t *__restrict__ idx_all, int64_t k, int64_t d, int *__restrict__ error_flag)
{
    const int row = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t >= k) return;
    const uint32_t *idx = idx_all + (int64_t)row * k;
    if ((int64_t)idx[t] >= d || (t > 0 && idx[t - 1] >= idx[t])) atomicExch(error_flag, 2);
}

void randk_set(TopkWorkspace *w, const uint32_t *sets, int *error_flag, cudaStream_t st)
{
    cudaMemcpyAsync(w->idx, sets, (size_t)w->rows * w->k * 4, cudaMemcpyDeviceToDevice, st);
    const dim3 entries((unsigned)((w->k + kBlock - 1) / kBlock), (unsigned)w->rows);
    k_check_sets<<<entries, kBlock, 0, st>>>(w->idx, w->k, w->d, error_flag);
}

void randk_gather(TopkWorkspace *w, const float *a, float *b, bool update_b, cudaStream_t st)
{
    const dim3 entries((unsigned)((w->k + kBlock - 1) / kBlock), (unsigned)w->rows);
    if (b && update_b) k_topk_gather<true, true><<<entries, kBlock, 0, st>>>(a, b, w->idx, w->val, nullptr, w->d, w->k, w->stride, nullptr);
    else if (b) k_topk_gather<true, false><<<entries, kBlock, 0, st>>>(a, b, w->idx, w->val, nullptr, w->d, w->k, w->stride, nullptr);
    else k_topk_gather<false, false><<<entries, kBlock, 0, st>>>(a, nullptr, w->idx, w->val, nullptr, w->d, w->k, w->stride, nullptr);
}

int topk_compress(const float *x, int64_t d, int64_t k, uint32_t *idx, float *val, cudaStream_t st)
{
    TopkWorkspace *w = nullptr;
    int rc = topk_workspace_create(&w, d, k, 1, idx, val, true);
    if (rc) return rc;
    topk_select(w, x, nullptr, false, ((uintptr_t)x & 15u) == 0 && d % 4 == 0, st);
    cudaError_t e = cudaStreamSynchronize(st);
    topk_workspace_destroy(w);
    return e == cudaSuccess ? CDADAM_OK : CDADAM_ERR_CUDA;
}

}  // namespace cdadam
