// Host-side launchers of the CD-Adam kernels.  Every launcher queues work on `st` and
// returns; errors are picked up by the caller with cudaGetLastError().
#pragma once
#include "common.cuh"

namespace cdadam {

// ---- scaled sign -------------------------------------------------------------------
// Worker pass (Algorithm 1: the workers' compression and state update) for all n workers: applies the previous payload
// (bits in wbits, scales in scale_old) to ghat_w (grads: n x d binary32 or bfloat16), forms u = g - ghat_w, packs sign(u) into
// wbits and writes per-tile double-double partial sums of |u| to wpart.  For large tiles the
// variant with a prefetch ring of bulk asynchronous copies runs; it sets *error_flag (device)
// if a bounded wait on a copy ran out (wait_limit polls; < 0 = the default).  With scale_new != NULL the block that completes a (worker, segment) also
// turns its partial sums into the scale (done: n x q zeroed counters, left zeroed), and no
// launch_finalize_scales is needed.
void launch_worker_sign(const void *grads, bool grads_bf16, float *ghat_w, uint32_t *wbits,
                        const float *scale_old, dd *wpart, const Tables &tb, int n,
                        int64_t wp, bool vec_ok, bool ef, int *error_flag, float *scale_new,
                        unsigned int *done, cudaStream_t st, int wait_limit = -1);
// Correctly rounded scale of every (row, segment) from the partial sums.  split > 1 (segments
// of very many tiles): that many blocks share a segment; split_sums holds rows x q x split
// sums, split_done rows x q zeroed counters (left zeroed).
void launch_finalize_scales(const dd *part, float *scales, const Tables &tb, int rows,
                            cudaStream_t st, int split = 1, dd *split_sums = nullptr,
                            unsigned int *split_done = nullptr);
// Coordinate-sharded iteration (the l1 norm of Appendix A's scaled sign is a sum over the
// coordinates, which several contexts may share).  launch_range_sums: this context's part of
// the l1 sum of every (row, local segment), one double-double each, into slot gidx[r] of the
// row's q_all slots.  launch_range_scales: the sums of all ranges (ranges x rows x q_all),
// added in the order of the ranges, rounded and divided by the whole segment's length glen[r]
// -> scales (rows x q_loc).
void launch_range_sums(const dd *part, dd *sums, const Tables &tb, int rows, const int32_t *gidx, int q_all,
                       cudaStream_t st);
void launch_range_scales(const dd *all, int ranges, int rows, int q_all, const int32_t *gidx, const int64_t *glen,
                         float *scales, int q_loc, cudaStream_t st);
// Server pass A (Algorithm 1: server aggregation and compression): ghat_s += mean_i decode(c_i); w = ghat_s - gtil; packs
// sign(w) into sbits and writes partial sums of |w| to spart.  sscale != NULL: the scales are
// finished in the same launch (done: q zeroed counters), as in the worker pass.
// mode: 0 Algorithm 1, 1 error feedback, 2 naive compression (w = mean; gtil is not read).
void launch_server_sign(const uint32_t *wbits, const float *wscale, float *ghat_s,
                        const float *gtil, uint32_t *sbits, dd *spart, const Tables &tb,
                        int n, int64_t wp, bool vec_ok, int mode, float *sscale, unsigned int *done,
                        cudaStream_t st);
// Server pass B and worker update (Algorithm 1: state update of gtil, AMSGrad): gtil += decode(c); AMSGrad.
void launch_update_sign(const uint32_t *sbits, const float *sscale, const float *ghat_s, float *gtil,
                        float *m, float *v, float *vhat, float *x, const Tables &tb, Hyper hp,
                        bool vec_ok, int mode, cudaStream_t st);
// ghat_w += decode(bits, scales) for all workers (applies a deferred payload).
void launch_apply_sign(float *ghat_w, const uint32_t *wbits, const float *scales,
                       const Tables &tb, int n, int64_t wp, bool ef, cudaStream_t st);
// Scaled-sign compressor without state for `rows` vectors (x rows x d, bits rows x wp, part
// rows x nparts): bits and partial sums of |x|.
void launch_pack_sign(const float *x, uint32_t *bits, dd *part, const Tables &tb, int rows,
                      int64_t wp, bool vec_ok, cudaStream_t st);

// ---- identity ----------------------------------------------------------------------
// The whole iteration with C(u) = u, one fused pass.
void launch_step_identity(const float *grads, float *ghat_w, float *ghat_s, float *gtil,
                          float *m, float *v, float *vhat, float *x, int64_t d, int n,
                          Hyper hp, int mode, cudaStream_t st);

// ---- pieces of the error-feedback iteration with the top-k compressor ---------------------
// dst[j] = (float)src[j] for count bfloat16 values (exact widening).
void launch_widen_bf16(float *dst, const void *src, int64_t count, cudaStream_t st);
// dst[j] = src[j] + dst[j] for count floats (p = g + delta, kept in the delta buffer).
void launch_add_into(float *dst, const float *src, int64_t count, bool vec_ok, cudaStream_t st);
// dst[idx[t]] = val ? val[t] : 0 for t < k, for `rows` rows (dst stride d, idx/val stride k).
void launch_scatter_set(float *dst, const uint32_t *idx, const float *val, int64_t k, int64_t d,
                        int rows, cudaStream_t st);
// dst[idx[t]] = 0 for t < rows * k: one vector, the coordinate sets of all rows.
void launch_scatter_add(float *dst, const uint32_t *idx, const float *val, int64_t k, int64_t d, cudaStream_t st);
void launch_scatter_zero_shared(float *dst, const uint32_t *idx, int64_t k, int rows, cudaStream_t st);

// ---- AMSGrad alone on a dense gradient estimate (top-k path) ------------------------------
void launch_amsgrad(const float *gtil, float *m, float *v, float *vhat, float *x, int64_t d,
                    Hyper hp, bool vec_ok, cudaStream_t st);

// Store the message cdadam_last_error() returns for the calling thread.
void set_last_error(const char *message);

}  // namespace cdadam
