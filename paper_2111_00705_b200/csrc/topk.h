// Top-k compressor (Appendix A) as an exact three-level radix select on the magnitude
// bits, for `rows` independent vectors at once, plus the sparse server aggregation.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cdadam {

struct TopkWorkspace;

// Scratch and payload buffers for selecting k of d coordinates in each of `rows` vectors.
// If idx/val are NULL the workspace owns the payload arrays (rows x k each).  stride: elements
// between consecutive rows of the vectors given to topk_select (0 = d; larger when the rows
// are segments of longer vectors).
// with_select = false allocates the payload arrays only (rand-k needs no selection scratch).
int topk_workspace_create(TopkWorkspace **w, int64_t d, int64_t k, int rows,
                          uint32_t *idx = nullptr, float *val = nullptr, bool with_select = true,
                          int64_t stride = 0);
void topk_workspace_destroy(TopkWorkspace *w);
// Device word that a selection kernel sets to 1 when a bounded wait on an asynchronous copy
// runs out (NULL: not reported).
void topk_workspace_set_error_flag(TopkWorkspace *w, int *error_flag);
// Which kernel makes the dense pass: 0 = chosen from the size (the default), 1 = the
// prefetch-ring kernel wherever rows are 16-byte aligned, -1 = the plain kernel.
void topk_workspace_set_ring(TopkWorkspace *w, int ring);
// Deferred state update for topk_select(..., update_b = true): a row selected from the dense
// pass's lists keeps b += u for the next selection, whose dense pass has the tiles of b in hand
// and applies the previous payload first (one pass over b instead of k random read-modify-
// writes per row).  Between selections b then lacks the last payload at those rows;
// topk_flush(w, b) applies what is pending (before b is read by anyone else), and
// topk_forget_pending drops it (when b is replaced from outside).
void topk_workspace_set_defer(TopkWorkspace *w, bool on);
void topk_flush(TopkWorkspace *w, float *b, cudaStream_t st);
void topk_forget_pending(TopkWorkspace *w, cudaStream_t st);
// Polls after which a bounded wait on an asynchronous copy gives up (< 0: the default).
void topk_workspace_set_wait_limit(TopkWorkspace *w, int polls);
void topk_payload(TopkWorkspace *w, int row, const uint32_t **idx, const float **val);
int topk_launches_per_step(int n);
// 1 or 2: kernels that make the dense pass of one selection in this workspace (rows aligned or not).
int topk_dense_launches(const TopkWorkspace *w, bool vec_ok);

// For every row r: u = a_r - b_r (b may be NULL: u = a_r); keep the k coordinates of
// largest |u| (ties: lower index); write their indices (increasing) and values u_j to the
// payload; if update_b, b_r[j] += u_j at the kept coordinates.  a, b: rows x d.
void topk_select(TopkWorkspace *w, const float *a, float *b, bool update_b, bool vec_ok,
                 cudaStream_t st);

// The server stage of Algorithm 1 in one selection: ghat_s += mean of the n payloads held in
// `ww` (workers added in the order 0..n-1, as topk_aggregate does), then the selection of
// ws (one row) on ghat_s - gtil with gtil updated at the kept coordinates.  The aggregation
// runs inside the dense pass of the selection, tile by tile.  ww and ws: same d, ws->rows == 1,
// ww selected by topk_select (its per-tile payload offsets are used where a row has them).
void topk_select_aggregated(TopkWorkspace *ws, TopkWorkspace *ww, float *ghat_s, float *gtil, int n, bool vec_ok,
                            cudaStream_t st);

// Coordinate-sharded selection: the workspace holds the coordinates of one range of every
// row; `ranges` such workspaces select the k_all largest of the whole rows between them.  One
// selection is the stages 0..4 in order; after each of the stages 0..3 the caller gathers
// the slots of all ranges in the exchange buffer (ranges x topk_range_exchange_words(w)
// uint32; stage s writes slot `range`, stage s + 1 reads all slots).  After stage 4 the
// payload rows hold this range's kept coordinates (increasing, relative to the range) and
// values, the rest of each row marked with the coordinate 0xffffffff; b (if given) is
// updated at the kept coordinates.  The workspace's k is the capacity of a payload row
// (min(k_all, d) is enough).  No threshold guess is used: two dense passes per selection.
void topk_range_stage(TopkWorkspace *w, int stage, const float *a, float *b, bool vec_ok, int64_t k_all,
                      uint32_t *exchange, int range, int ranges, cudaStream_t st);
int64_t topk_range_exchange_words(const TopkWorkspace *w);

// Top-k per segment: copies the payload of `seg` (a segment starting at coordinate `offset` of
// the whole vector) into entries [at, at + seg.k) of every row of `whole`'s payload, indices
// moved by `offset`.
void topk_payload_concat(TopkWorkspace *whole, int64_t at, TopkWorkspace *seg, int64_t offset, cudaStream_t st);

// Sparse server aggregation (Algorithm 1: ghat += mean of the workers' messages) from the n payloads held in `ww`:
//   ghat_s += (sum_i c_i) / n on the coordinates some worker sent, workers added in the
//   order 0, 1, ..., n-1.
void topk_aggregate(TopkWorkspace *ww, float *ghat_s, int n, cudaStream_t st);

// The same from n messages laid out as n x k arrays (coordinates increasing in every row)
// that come without the selecting side's per-tile offsets: every block finds its entries by
// binary search.
void topk_aggregate_rows(const uint32_t *idx, const float *val, int64_t k, int64_t d, int n, float *ghat_s,
                         cudaStream_t st);

// Rand-k (Appendix A): the k coordinates of every row are given by the caller.
// randk_set copies rows x k device indices into the payload and checks them (strictly
// increasing, below d; *error_flag = 2 otherwise).  randk_gather fills the payload values
// u_j = a_j - b_j (b may be NULL) and, if update_b, adds them to b at those coordinates.
void randk_set(TopkWorkspace *w, const uint32_t *sets, int *error_flag, cudaStream_t st);
void randk_gather(TopkWorkspace *w, const float *a, float *b, bool update_b, cudaStream_t st);

// Stand-alone top-k of one vector into caller buffers (allocates and frees scratch).
int topk_compress(const float *x, int64_t d, int64_t k, uint32_t *idx, float *val,
                  cudaStream_t st);

}  // namespace cdadam
