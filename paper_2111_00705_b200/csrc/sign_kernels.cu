// Scaled-sign path of Algorithm 1 (CD-Adam) for sm_100a: worker pass, server pass A,
// server pass B + AMSGrad, scale finalisation, deferred-payload application.
//
// Every kernel streams its vectors exactly once.  In the worker and server passes a block
// owns one tile of the index space; the update pass uses 1024-coordinate blocks.  Tiles that
// lie inside one segment, inside [0, d) and whose rows are 16-byte aligned take the vector
// path (128-bit accesses, ballot packing, no bounds checks; for large tiles the worker pass
// prefetches through a TMA ring); all other tiles (segment boundaries, the ragged tail,
// unaligned rows) take a scalar path with the same arithmetic in the same order, so both
// paths give identical bits.  Every kernel exists for the two recursions (Markov sequences
// of Algorithm 1, classical error feedback) and the worker pass for binary32 and bfloat16
// gradients.
#include "kernels.h"

namespace cdadam {

constexpr uint32_t kFull = 0xffffffffu;

__device__ __forceinline__ float signed_scale(uint32_t bit, float s) { return bit ? s : -s; }

// ------------------------------------------------------------------------------------
// The two recursions a kernel can run (template parameter EF).
//   EF = false, Algorithm 1 (Markov compression sequence): the worker buffer holds ghat^(i);
//     ghat += c_prev, u = g - ghat; the server keeps ghat and gtil: ghat += mean,
//     w = ghat - gtil, then gtil += c and AMSGrad runs on gtil.
//   EF = true, classical error feedback (Section 4): the worker buffer holds the last
//     compressor input p_prev = g_prev + delta_prev; delta = p_prev - c_prev, u = p = g + delta;
//     the server keeps its error delta in the gtil buffer and its compressor input
//     p = mean + delta in the ghat buffer; then delta = p - c and AMSGrad runs on c.
// `stored` is what the buffer holds, `store` what is written back; the value returned is
// the compressor input.
// The server-side kernels take MODE: 0 = Algorithm 1, 1 = error feedback, 2 = naive
// compression (Section 4: no state; as error feedback with the error held at zero and
// never written; the workers' payloads come from k_pack_sign on the gradients).
// ------------------------------------------------------------------------------------
template <bool EF>
__device__ __forceinline__ float worker_step(float g, float stored, float c_prev, float &store)
{
    if (EF) {
        store = __fadd_rn(g, __fsub_rn(stored, c_prev));
        return store;
    }
    store = __fadd_rn(stored, c_prev);
    return __fsub_rn(g, store);
}
template <bool EF>
__device__ __forceinline__ float worker_input_from_memory(float g, float stored)
{
    return EF ? stored : __fsub_rn(g, stored);
}
template <bool EF>
__device__ __forceinline__ float server_step(float mean, float ghat_stored, float gt, float &store)
{
    if (EF) {
        store = __fadd_rn(mean, gt);
        return store;
    }
    store = __fadd_rn(ghat_stored, mean);
    return __fsub_rn(store, gt);
}
template <bool EF>
__device__ __forceinline__ float server_input_from_memory(float ghat_stored, float gt)
{
    return EF ? ghat_stored : __fsub_rn(ghat_stored, gt);
}
// Returns the gradient estimate AMSGrad uses; gt_store is the new content of the gtil buffer.
template <bool EF>
__device__ __forceinline__ float update_step(float gt_stored, float p, float c, float &gt_store)
{
    if (EF) {
        gt_store = __fsub_rn(p, c);
        return c;
    }
    gt_store = __fadd_rn(gt_stored, c);
    return gt_store;
}

// Gradient element types: binary32, or bfloat16 (the upper 16 bits of a binary32, so the
// conversion is exact and the arithmetic that follows is unchanged).
typedef uint16_t bf16_t;
__device__ __forceinline__ float grad_at(const float *g, int64_t j) { return g[j]; }
__device__ __forceinline__ float grad_at(const bf16_t *g, int64_t j)
{
    return __uint_as_float((uint32_t)g[j] << 16);
}
__device__ __forceinline__ float4 grad_ld4(const float *g) { return ld_ro4(g); }
__device__ __forceinline__ float4 grad_ld4(const bf16_t *g)
{
    uint2 raw;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(raw.x), "=r"(raw.y) : "l"(g));
    return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                       __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
}
// eight consecutive gradients (32-byte / 16-byte aligned)
__device__ __forceinline__ void grad_ld8(const float *g, float (&v)[8]) { ld_ro8(g, v); }
__device__ __forceinline__ void grad_ld8(const bf16_t *g, float (&v)[8])
{
    uint4 raw;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(raw.x), "=r"(raw.y), "=r"(raw.z), "=r"(raw.w) : "l"(g));
    v[0] = __uint_as_float(raw.x << 16); v[1] = __uint_as_float(raw.x & 0xffff0000u);
    v[2] = __uint_as_float(raw.y << 16); v[3] = __uint_as_float(raw.y & 0xffff0000u);
    v[4] = __uint_as_float(raw.z << 16); v[5] = __uint_as_float(raw.z & 0xffff0000u);
    v[6] = __uint_as_float(raw.w << 16); v[7] = __uint_as_float(raw.w & 0xffff0000u);
}
// four consecutive gradients from a shared-memory copy of a sub-tile
__device__ __forceinline__ float4 grad_lds4(const float *g) { return *reinterpret_cast<const float4 *>(g); }
__device__ __forceinline__ float4 grad_lds4(const bf16_t *g)
{
    const uint2 raw = *reinterpret_cast<const uint2 *>(g);
    return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                       __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
}

// ------------------------------------------------------------------------------------
// Scale of one (row, segment) without a launch of its own: every block that has written a
// partial l1 sum of the segment takes a ticket, and the block that takes the last one adds
// the partial sums (fixed thread mapping and tree, hence the same result whichever block
// it is), rounds and divides as k_finalize_scales does, and puts the counter back to zero.
// No block waits for another.  `part`, `scales` and `done` are the row's.  All threads of the
// block call it, after thread 0 has written the block's partial sum.
// ------------------------------------------------------------------------------------
__device__ __noinline__ void finish_segment(const dd *part, float *scales, unsigned int *done, int r,
                                            const int64_t *__restrict__ off,
                                            const int32_t *__restrict__ tile_first,
                                            const int64_t *__restrict__ pbase, int tile)
{
    __shared__ int is_last;
    const int64_t lo = off[r], hi = off[r + 1];
    const int64_t T0 = lo / tile, T1 = (hi - 1) / tile;
    __syncthreads();                 // the previous call's readers of is_last are done
    if (threadIdx.x == 0) {
        __threadfence();             // this block's partial sum is visible before its ticket
        is_last = atomicAdd(done + r, 1u) == (unsigned int)(T1 - T0);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    dd a0 = {0.0, 0.0}, a1 = {0.0, 0.0};
    for (int64_t T = T0 + threadIdx.x; T <= T1; T += 2 * kBlock) {
        const double2 p0 = __ldcg(reinterpret_cast<const double2 *>(part + pbase[T] + (r - tile_first[T])));
        a0 = dd_add(a0, dd{p0.x, p0.y});
        const int64_t U = T + kBlock;
        if (U <= T1) {
            const double2 p1 = __ldcg(reinterpret_cast<const double2 *>(part + pbase[U] + (r - tile_first[U])));
            a1 = dd_add(a1, dd{p1.x, p1.y});
        }
    }
    a0 = block_sum<kBlock>(dd_add(a0, a1));
    if (threadIdx.x == 0) {
        const double l1 = __dadd_rn(a0.hi, a0.lo);
        scales[r] = __double2float_rn(__ddiv_rn(l1, (double)(hi - lo)));
        done[r] = 0u;
    }
}

// Scalar path of the worker pass for one tile (segment boundaries, the ragged last tile,
// unaligned rows).  Kept out of line so that it does not shape the register allocation and
// instruction schedule of the vector path.
template <bool EF, typename G>
__device__ __noinline__ void worker_tile_scalar(const G *__restrict__ g, float *__restrict__ gh,
                                                uint32_t *__restrict__ bw, const float *__restrict__ so,
                                                dd *__restrict__ part, const int64_t *__restrict__ off,
                                                int64_t base, int64_t end, int first, int last)
{
    const int lane = threadIdx.x & 31;
    // scalar path: lane L of a warp holds coordinate (word start + L), ballot = word.
    // Four rounds are loaded before any is processed to keep several loads in flight.
    for (int64_t j0 = base + threadIdx.x; j0 - lane < end; j0 += 4 * kBlock) {
        float gv[4], hv[4], sv[4];
        uint32_t wv[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int64_t j = j0 + t * kBlock;
            gv[t] = hv[t] = sv[t] = 0.0f;
            wv[t] = 0u;
            if (j < end) {
                gv[t] = grad_at(g, j);
                hv[t] = gh[j];
                wv[t] = bw[j >> 5];
                sv[t] = so[find_segment(off, first, last, j)];
            }
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int64_t j = j0 + t * kBlock;
            if (j - lane < end) {                      // warp-uniform
                const bool valid = j < end;
                float u = -1.0f;
                if (valid) {
                    float hn;
                    u = worker_step<EF>(gv[t], hv[t], signed_scale((wv[t] >> (j & 31)) & 1u, sv[t]), hn);
                    gh[j] = hn;
                }
                const uint32_t word = __ballot_sync(kFull, valid && u >= 0.0f);
                if (lane == 0) bw[j >> 5] = word;
            }
        }
    }
    __syncthreads();
    for (int r = first; r <= last; ++r) {
        const int64_t lo = max(off[r], base), hi = min(off[r + 1], end);
        dd acc = {0.0, 0.0};
        for (int64_t j = lo + threadIdx.x; j < hi; j += kBlock)
            dd_acc(acc, fabsf(worker_input_from_memory<EF>(grad_at(g, j), gh[j])));
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) part[r - first] = acc;
    }
}

// ------------------------------------------------------------------------------------
// Worker pass.  grid = (ntiles, n).
// ------------------------------------------------------------------------------------
// The 16 coordinates a thread owns in one 4096-coordinate sub-tile: gradient, worker state
// and the previous payload's sign words.
struct WorkerRegs {
    float4 G[4], H[4];
    uint32_t ow[4];
};

template <typename G>
__device__ __forceinline__ void worker_load(WorkerRegs &r, const G *__restrict__ g,
                                            const float *__restrict__ gh,
                                            const uint32_t *__restrict__ bw, int64_t wb, int lane)
{
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        const int64_t j = wb + v * 128 + lane * 4;
        r.G[v] = grad_ld4(g + j);
        r.H[v] = ld_rw4(gh + j);
        r.ow[v] = bw[(wb >> 5) + v * 4 + (lane >> 3)];
    }
}

template <bool EF>
__device__ __forceinline__ void worker_compute(WorkerRegs &r, float *__restrict__ gh,
                                               uint32_t *__restrict__ bw, int64_t wb, int lane,
                                               float s, dd &acc)
{
    uint32_t B[4][4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        const uint32_t nib = r.ow[v] >> ((lane & 7) * 4);
        // the previous payload (sign words + scale) is applied now, then the new input formed
        float4 H;
        const float ux = worker_step<EF>(r.G[v].x, r.H[v].x, signed_scale(nib & 1u, s), H.x);
        const float uy = worker_step<EF>(r.G[v].y, r.H[v].y, signed_scale(nib & 2u, s), H.y);
        const float uz = worker_step<EF>(r.G[v].z, r.H[v].z, signed_scale(nib & 4u, s), H.z);
        const float uw = worker_step<EF>(r.G[v].w, r.H[v].w, signed_scale(nib & 8u, s), H.w);
        st_rw4(gh + wb + v * 128 + lane * 4, H);
        dd_acc(acc, fabsf(ux)); dd_acc(acc, fabsf(uy));
        dd_acc(acc, fabsf(uz)); dd_acc(acc, fabsf(uw));
        B[v][0] = __ballot_sync(kFull, ux >= 0.0f);
        B[v][1] = __ballot_sync(kFull, uy >= 0.0f);
        B[v][2] = __ballot_sync(kFull, uz >= 0.0f);
        B[v][3] = __ballot_sync(kFull, uw >= 0.0f);
    }
    const uint32_t word = warp_words(B, lane);
    if (lane < 16) bw[(wb >> 5) + lane] = word;
}

template <bool EF, typename G>
__global__ void __launch_bounds__(kBlock, 4)
k_worker_sign(const G *__restrict__ grads, float *__restrict__ ghat_w,
              uint32_t *__restrict__ wbits, const float *__restrict__ scale_old,
              dd *__restrict__ wpart, Tables tb, int64_t wp, int vec_ok,
              float *__restrict__ scale_new, unsigned int *__restrict__ done, int vec8_ok)
{
    grid_dep_launch();
    const int i = blockIdx.y;
    const int64_t T = tb.order[blockIdx.x];
    const int first = tb.tile_first[T], last = tb.tile_last[T];
    const int64_t base = T * tb.tile;
    const G *g = grads + (int64_t)i * tb.d;
    float *gh = ghat_w + (int64_t)i * tb.d;
    uint32_t *bw = wbits + (int64_t)i * wp;
    const float *so = scale_old + (int64_t)i * tb.q;

    if (!(vec_ok && first == last && base + tb.tile <= tb.d)) {
        worker_tile_scalar<EF, G>(g, gh, bw, so, wpart + (int64_t)i * tb.nparts + tb.pbase[T], tb.off, base,
                           min(base + (int64_t)tb.tile, tb.d), first, last);
    } else if (vec8_ok) {
        // Eight consecutive coordinates per thread (256-bit accesses; rows 32-byte aligned): a
        // lane's coordinates are byte (lane & 3) of word (lane >> 2) of the warp's eight sign
        // words, both of the previous payload that is applied first and of the new one, which
        // is packed as a byte per lane and joined over the word's four lanes by two shuffles.
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const float s = so[first];
        const uint32_t bsel = lane & 3u;
        dd acc = {0.0, 0.0};
        // two 2048-coordinate sub-tiles per round: both rounds of loads are in flight together
        for (int it = 0; it < tb.tile / (8 * kBlock); it += 2) {
            float Gv[2][8], H[2][8];
            uint32_t old[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t wb = base + (int64_t)(it + h) * (8 * kBlock) + warp * 256;
                grad_ld8(g + wb + lane * 8, Gv[h]);
                ld_rw8(gh + wb + lane * 8, H[h]);
                old[h] = bw[(wb >> 5) + (lane >> 2)] >> (8u * bsel);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t wb = base + (int64_t)(it + h) * (8 * kBlock) + warp * 256;
                uint32_t bits = 0u;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float hn;
                    const float u = worker_step<EF>(Gv[h][c], H[h][c], signed_scale((old[h] >> c) & 1u, s), hn);
                    H[h][c] = hn;
                    dd_acc(acc, fabsf(u));
                    bits |= (u >= 0.0f ? 1u : 0u) << c;
                }
                st_rw8(gh + wb + lane * 8, H[h]);
                uint32_t word = bits << (8u * bsel);
                word |= __shfl_xor_sync(kFull, word, 1);
                word |= __shfl_xor_sync(kFull, word, 2);
                if (bsel == 0u) bw[(wb >> 5) + (lane >> 2)] = word;
            }
        }
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) wpart[(int64_t)i * tb.nparts + tb.pbase[T]] = acc;
    } else {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const float s = so[first];
        const int iters = tb.tile / kSub;
        dd acc = {0.0, 0.0};
        for (int it = 0; it < iters; ++it) {
            WorkerRegs r;
            const int64_t wb = base + (int64_t)it * kSub + warp * kWarpSpan;
            worker_load(r, g, gh, bw, wb, lane);
            worker_compute<EF>(r, gh, bw, wb, lane, s, acc);
        }
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) wpart[(int64_t)i * tb.nparts + tb.pbase[T]] = acc;
    }
    if (scale_new)                                             // launch-uniform
        for (int r = first; r <= last; ++r)
            finish_segment(wpart + (int64_t)i * tb.nparts, scale_new + (int64_t)i * tb.q,
                           done + (int64_t)i * tb.q, r, tb.off, tb.tile_first, tb.pbase, tb.tile);
}

// ------------------------------------------------------------------------------------
// Worker pass with a prefetch ring.  grid = (ntiles, n), tile >= 4 sub-tiles.
//
// Same arithmetic as k_worker_sign.  The gradient and worker-state sub-tiles are brought
// into a two-stage shared-memory ring by bulk asynchronous copies (TMA), issued by one
// thread, so the next sub-tile is in flight while the block works on the current one; each
// thread moves its 16 coordinates from the ring to registers and the stage is refilled at
// once.  Measured at the HBM ceiling for this 8-bytes-read / 4-bytes-written mix.
// ------------------------------------------------------------------------------------
constexpr int kRingStages = 2;
constexpr int kRingStageBytes = 2 * kSub * (int)sizeof(float);    // g and ghat sub-tile: 32 KiB
constexpr int kRingSmemBytes = kRingStages * kRingStageBytes;

template <bool EF, typename G>
__global__ void __launch_bounds__(kBlock, 3)
k_worker_sign_ring(const G *__restrict__ grads, float *__restrict__ ghat_w,
                   uint32_t *__restrict__ wbits, const float *__restrict__ scale_old,
                   dd *__restrict__ wpart, Tables tb, int64_t wp, int *__restrict__ error_flag,
                   float *__restrict__ scale_new, unsigned int *__restrict__ done, int wait_limit)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t full[kRingStages];
    grid_dep_launch();
    const int i = blockIdx.y;
    const int64_t T = tb.order[blockIdx.x];
    const int first = tb.tile_first[T], last = tb.tile_last[T];
    const int64_t base = T * tb.tile;
    const G *g = grads + (int64_t)i * tb.d;
    float *gh = ghat_w + (int64_t)i * tb.d;
    uint32_t *bw = wbits + (int64_t)i * wp;
    const float *so = scale_old + (int64_t)i * tb.q;

    if (!(first == last && base + tb.tile <= tb.d)) {          // block-uniform
        worker_tile_scalar<EF, G>(g, gh, bw, so, wpart + (int64_t)i * tb.nparts + tb.pbase[T], tb.off, base,
                           min(base + (int64_t)tb.tile, tb.d), first, last);
        if (scale_new)
            for (int r = first; r <= last; ++r)
                finish_segment(wpart + (int64_t)i * tb.nparts, scale_new + (int64_t)i * tb.q,
                               done + (int64_t)i * tb.q, r, tb.off, tb.tile_first, tb.pbase, tb.tile);
        return;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int iters = tb.tile / kSub;
    if (threadIdx.x == 0) {
        for (int st = 0; st < kRingStages; ++st) mbar_init(&full[st], 1);
        mbar_fence_init();
    }
    __syncthreads();
    auto refill = [&](int it, int st) {                        // one thread
        // stage layout: the worker-state sub-tile (16 KiB), then the gradient sub-tile
        float *dst = reinterpret_cast<float *>(ring + st * kRingStageBytes);
        mbar_arrive_expect_tx(&full[st], (uint32_t)(kSub * (sizeof(float) + sizeof(G))));
        bulk_copy_g2s(dst, gh + base + (int64_t)it * kSub, kSub * sizeof(float), &full[st]);
        bulk_copy_g2s(dst + kSub, g + base + (int64_t)it * kSub, kSub * sizeof(G), &full[st]);
    };
    if (threadIdx.x == 0)
        for (int st = 0; st < kRingStages && st < iters; ++st) refill(st, st);
    const float s = so[first];
    dd acc = {0.0, 0.0};
    bool arrived = true;
    int it = 0;
    for (; it < iters; ++it) {
        const int st = it % kRingStages;
        const bool mine = mbar_wait_bounded(&full[st], (uint32_t)(it / kRingStages) & 1u, wait_limit);
        const float *src = reinterpret_cast<const float *>(ring + st * kRingStageBytes);
        const int64_t wb = base + (int64_t)it * kSub + warp * kWarpSpan;
        WorkerRegs r;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int e = warp * kWarpSpan + v * 128 + lane * 4;
            r.H[v] = *reinterpret_cast<const float4 *>(src + e);
            r.G[v] = grad_lds4(reinterpret_cast<const G *>(src + kSub) + e);
            r.ow[v] = bw[(wb >> 5) + v * 4 + (lane >> 3)];
        }
        // the stage has been read by all; the same barrier makes the outcome of the waits one
        // decision of the whole block (a thread whose wait ran out has read a stage that may
        // be incomplete: nothing of it is used)
        arrived = !__syncthreads_or(!mine);
        if (!arrived) break;
        if (threadIdx.x == 0 && it + kRingStages < iters) refill(it + kRingStages, st);
        worker_compute<EF>(r, gh, bw, wb, lane, s, acc);
    }
    if (!arrived) {
        // A copy did not complete in time: report it, give the copies still in flight (those
        // of sub-tiles it .. it + kRingStages - 1, issued and not yet consumed) a bounded
        // chance, the full default limit, to land before this block's shared memory is
        // released, and leave: all threads of the block together.  The step's results are
        // void; the scale of this segment is not finished.
        if (threadIdx.x == 0) atomicExch(error_flag, 1);
        for (int j = it; j < iters && j < it + kRingStages; ++j)
            mbar_wait_bounded(&full[j % kRingStages], (uint32_t)(j / kRingStages) & 1u);
        return;
    }
    acc = block_sum<kBlock>(acc);
    if (threadIdx.x == 0) wpart[(int64_t)i * tb.nparts + tb.pbase[T]] = acc;
    if (scale_new)
        finish_segment(wpart + (int64_t)i * tb.nparts, scale_new + (int64_t)i * tb.q,
                       done + (int64_t)i * tb.q, first, tb.off, tb.tile_first, tb.pbase, tb.tile);
}

// ------------------------------------------------------------------------------------
// Scale of (row, segment): partial sums added in a fixed order, rounded to binary64,
// divided by the segment length in binary64, rounded to binary32.  grid = (q, rows).
// ------------------------------------------------------------------------------------
constexpr int kFinBlock = 512;

__global__ void __launch_bounds__(kFinBlock)
k_finalize_scales(const dd *__restrict__ part, float *__restrict__ scales, Tables tb)
{
    grid_dep_launch();
    const int r = blockIdx.x, row = blockIdx.y;
    const int64_t lo = tb.off[r], hi = tb.off[r + 1];
    const int64_t T0 = lo / tb.tile, T1 = (hi - 1) / tb.tile;
    const dd *p = part + (int64_t)row * tb.nparts;
    dd acc = {0.0, 0.0};
    grid_dep_wait();                                   // the partial sums come from the pass before
    for (int64_t T = T0 + threadIdx.x; T <= T1; T += kFinBlock) {
        const double2 v = __ldcg(reinterpret_cast<const double2 *>(p + tb.pbase[T] + (r - tb.tile_first[T])));
        acc = dd_add(acc, dd{v.x, v.y});
    }
    acc = block_sum<kFinBlock>(acc);
    if (threadIdx.x == 0) {
        const double l1 = __dadd_rn(acc.hi, acc.lo);
        scales[(int64_t)row * tb.q + r] = __double2float_rn(__ddiv_rn(l1, (double)(hi - lo)));
    }
}

// The same for segments of very many tiles (a flat 1.5e9-coordinate buffer has 91,553):
// gridDim.z blocks share a (row, segment), each adds a contiguous run of its tiles; the block
// that finishes last (ticket) adds the gridDim.z sums in block order.  Same value whichever
// block that is; no block waits.  grid = (q, rows, split); done: rows x q zeroed counters,
// left zeroed; sums: rows x q x split.
__global__ void __launch_bounds__(kFinBlock)
k_finalize_scales_split(const dd *__restrict__ part, float *__restrict__ scales, Tables tb,
                        dd *sums, unsigned int *done)
{
    __shared__ int is_last;
    const int r = blockIdx.x, row = blockIdx.y, z = blockIdx.z, nz = gridDim.z;
    const int64_t lo = tb.off[r], hi = tb.off[r + 1];
    const int64_t T0 = lo / tb.tile, T1 = (hi - 1) / tb.tile;
    const int64_t per = (T1 - T0 + nz) / nz;              // tiles per block, rounded up
    const int64_t A = T0 + z * per, B = min(A + per, T1 + 1);
    const dd *p = part + (int64_t)row * tb.nparts;
    dd acc = {0.0, 0.0};
    grid_dep_launch();
    grid_dep_wait();                                   // the partial sums come from the pass before
    for (int64_t T = A + threadIdx.x; T < B; T += kFinBlock) {
        const double2 v = __ldcg(reinterpret_cast<const double2 *>(p + tb.pbase[T] + (r - tb.tile_first[T])));
        acc = dd_add(acc, dd{v.x, v.y});
    }
    acc = block_sum<kFinBlock>(acc);
    const int64_t slot = (int64_t)row * tb.q + r;
    if (threadIdx.x == 0) {
        sums[slot * nz + z] = acc;
        __threadfence();
        is_last = atomicAdd(done + slot, 1u) == (unsigned int)(nz - 1);
    }
    __syncthreads();
    if (!is_last || threadIdx.x != 0) return;
    __threadfence();
    dd tot = {0.0, 0.0};
    for (int i = 0; i < nz; ++i) {
        const double2 v = __ldcg(reinterpret_cast<const double2 *>(sums + slot * nz + i));
        tot = dd_add(tot, dd{v.x, v.y});
    }
    const double l1 = __dadd_rn(tot.hi, tot.lo);
    scales[slot] = __double2float_rn(__ddiv_rn(l1, (double)(hi - lo)));
    done[slot] = 0u;
}

// ------------------------------------------------------------------------------------
// Coordinate-sharded iteration.  A context that owns the coordinates [lo, hi) of every vector
// cannot finish a scale: the l1 norm of a segment is a sum over all coordinates of the
// segment, whoever owns them.  It reduces its own part of every (row, segment) to one
// double-double (k_range_sums, the tiles in the fixed order of k_finalize_scales), the
// owners' sums are brought together by the caller, and every context adds them in the order
// of the ranges and rounds (k_range_scales): binary64 nearest, divided by the length of the
// WHOLE segment, rounded to binary32.  A double-double carries about 104 bits, so the value
// that is rounded, and with it the scale, is the one a single context computes.
//   sums:   rows x q_all double-doubles of this context; a local segment r goes to slot
//           gidx[r], the slots of segments that do not meet the range stay zero
//   all:    ranges x rows x q_all, slot by slot the sums of every range
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kFinBlock)
k_range_sums(const dd *__restrict__ part, dd *__restrict__ sums, Tables tb,
             const int32_t *__restrict__ gidx, int q_all)
{
    const int r = blockIdx.x, row = blockIdx.y;
    const int64_t lo = tb.off[r], hi = tb.off[r + 1];
    const int64_t T0 = lo / tb.tile, T1 = (hi - 1) / tb.tile;
    const dd *p = part + (int64_t)row * tb.nparts;
    dd acc = {0.0, 0.0};
    for (int64_t T = T0 + threadIdx.x; T <= T1; T += kFinBlock)
        acc = dd_add(acc, p[tb.pbase[T] + (r - tb.tile_first[T])]);
    acc = block_sum<kFinBlock>(acc);
    if (threadIdx.x == 0) sums[(int64_t)row * q_all + gidx[r]] = acc;
}

__global__ void __launch_bounds__(kBlock)
k_range_scales(const dd *__restrict__ all, int ranges, int q_all, const int32_t *__restrict__ gidx,
               const int64_t *__restrict__ glen, float *__restrict__ scales, int q_loc)
{
    const int r = blockIdx.x * kBlock + threadIdx.x, row = blockIdx.y, rows = gridDim.y;
    if (r >= q_loc) return;
    dd tot = {0.0, 0.0};
    for (int z = 0; z < ranges; ++z)                   // the ranges in increasing order
        tot = dd_add(tot, all[((int64_t)z * rows + row) * q_all + gidx[r]]);
    const double l1 = __dadd_rn(tot.hi, tot.lo);
    scales[(int64_t)row * q_loc + r] = __double2float_rn(__ddiv_rn(l1, (double)glen[r]));
}

// ------------------------------------------------------------------------------------
// Server pass A.  grid = (ntiles).
//
// Vector path: a warp owns 128*VPT consecutive coordinates per iteration.  The sign words
// of up to kNC workers for that span are staged through shared memory, transposed so that a
// thread fetches the words of all its VPT coordinate groups for one worker with a single
// shared-memory load; the per-worker scales of the tile's segment sit in shared memory too.
// ------------------------------------------------------------------------------------
constexpr int kNC = 16;     // workers staged per chunk
constexpr int kTabWorkers = 8;   // workers whose sum is read from the pattern table

// Transpose of an 8x8 bit matrix held in 64 bits: bit (8 i + j) <-> bit (8 j + i)
// (three rounds of masked swaps of 1x1, 2x2 and 4x4 blocks).
__device__ __forceinline__ uint64_t transpose8x8(uint64_t x)
{
    x = (x & 0xAA55AA55AA55AA55ull) | ((x & 0x00AA00AA00AA00AAull) << 7) | ((x >> 7) & 0x00AA00AA00AA00AAull);
    x = (x & 0xCCCC3333CCCC3333ull) | ((x & 0x0000CCCC0000CCCCull) << 14) | ((x >> 14) & 0x0000CCCC0000CCCCull);
    x = (x & 0xF0F0F0F00F0F0F0Full) | ((x & 0x00000000F0F0F0F0ull) << 28) | ((x >> 28) & 0x00000000F0F0F0F0ull);
    return x;
}

template <int VPT, int MODE>
__global__ void __launch_bounds__(kBlock, 4)
k_server_sign(const uint32_t *__restrict__ wbits, const float *__restrict__ wscale,
              float *__restrict__ ghat_s, const float *__restrict__ gtil,
              uint32_t *__restrict__ sbits, dd *__restrict__ spart, Tables tb, int n,
              int64_t wp, int vec_ok, int n_pow2, float *__restrict__ sscale,
              unsigned int *__restrict__ done, int vec8_ok)
{
    constexpr bool EF = MODE != 0;
    __shared__ __align__(16) uint32_t wsm[kBlock / 32][kNC][4][VPT];   // [warp][worker][g][v]
    __shared__ float ssm[kNC];
    // tab[p]: the sequential sum over the first nt workers of +-s_i with the signs of pattern
    // p (bit i = worker i's sign bit), formed by the same additions in the same order as
    // adding worker by worker, hence the same bits
    __shared__ float tab[1 << kTabWorkers];
    const int64_t T = tb.order[blockIdx.x];
    const int first = tb.tile_first[T], last = tb.tile_last[T];
    const int64_t base = T * tb.tile;
    dd *part = spart + tb.pbase[T];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float fn = (float)n;
    const float rn = 1.0f / fn;               // exact when n is a power of two
    grid_dep_launch();
    grid_dep_wait();                          // worker sign words and scales come from the kernels before

    if (vec8_ok && first == last && base + tb.tile <= tb.d) {
        // Eight consecutive coordinates per thread (256-bit accesses; d % 8 == 0).  A lane's
        // coordinates are one byte of a sign word: byte (lane & 3) of word (lane >> 2) of the
        // warp's eight.  The lane gathers that byte from the words of workers 0..7 (PRMT),
        // one 8x8 bit transpose turns the eight bytes into the eight coordinates' sender
        // patterns, and the pattern table gives each coordinate's sum; further workers are
        // added one by one.  The new sign bits are packed as a byte per lane and joined
        // across the four lanes of a word by two shuffles (no ballots, no interleave).
        constexpr int kSpan8 = 256, kIter8 = kSpan8 * (kBlock / 32);
        const int nt = min(n, kTabWorkers);
        if (threadIdx.x < nt) ssm[threadIdx.x] = ld_cg_f32(wscale + (int64_t)threadIdx.x * tb.q + first);
        __syncthreads();
        {
            float t = 0.0f;
            for (int i = 0; i < nt; ++i) t = __fadd_rn(t, signed_scale((threadIdx.x >> i) & 1u, ssm[i]));
            tab[threadIdx.x] = t;                         // kBlock == 256 patterns (bits above nt are never set)
        }
        __syncthreads();
        const uint32_t bsel = lane & 3u;
        const uint32_t sel01 = bsel | ((bsel + 4u) << 4);     // PRMT: byte bsel of a, byte bsel of b
        dd acc = {0.0, 0.0};
        for (int it = 0; it < tb.tile / kIter8; ++it) {
            const int64_t wb = base + (int64_t)it * kIter8 + warp * kSpan8;
            const int64_t j = wb + lane * 8;
            float H[8], Gt[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) H[c] = Gt[c] = 0.0f;
            if (!EF) ld_rw8(ghat_s + j, H);               // error feedback overwrites this buffer
            if (MODE != 2) ld_ro8(gtil + j, Gt);
            const uint32_t *wrow = wbits + (wb >> 5) + (lane >> 2);
            uint32_t W[kTabWorkers];
#pragma unroll
            for (int i = 0; i < kTabWorkers; ++i) W[i] = i < nt ? ld_cg_u32(wrow + (int64_t)i * wp) : 0u;
            const uint32_t lo = __byte_perm(__byte_perm(W[0], W[1], sel01), __byte_perm(W[2], W[3], sel01), 0x5410u);
            const uint32_t hi = __byte_perm(__byte_perm(W[4], W[5], sel01), __byte_perm(W[6], W[7], sel01), 0x5410u);
            const uint64_t pat = transpose8x8(((uint64_t)hi << 32) | lo);
            const uint32_t plo = (uint32_t)pat, phi = (uint32_t)(pat >> 32);
            float a[8];
            a[0] = tab[plo & 0xFFu];         a[1] = tab[(plo >> 8) & 0xFFu];
            a[2] = tab[(plo >> 16) & 0xFFu]; a[3] = tab[plo >> 24];
            a[4] = tab[phi & 0xFFu];         a[5] = tab[(phi >> 8) & 0xFFu];
            a[6] = tab[(phi >> 16) & 0xFFu]; a[7] = tab[phi >> 24];
            for (int i = nt; i < n; ++i) {                // workers in increasing order
                const float s = ld_cg_f32(wscale + (int64_t)i * tb.q + first);
                const uint32_t byte = ld_cg_u32(wrow + (int64_t)i * wp) >> (8u * bsel);
#pragma unroll
                for (int c = 0; c < 8; ++c) a[c] = __fadd_rn(a[c], signed_scale((byte >> c) & 1u, s));
            }
            float S[8];
            uint32_t bits = 0u;
            if (n_pow2) {                                 // (decided once, outside the per-coordinate code)
#pragma unroll
                for (int c = 0; c < 8; ++c) a[c] = __fmul_rn(a[c], rn);
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c) a[c] = __fdiv_rn(a[c], fn);
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float mean = a[c];
                const float w = server_step<EF>(mean, H[c], Gt[c], S[c]);
                dd_acc(acc, fabsf(w));
                bits |= (w >= 0.0f ? 1u : 0u) << c;
            }
            st_rw8(ghat_s + j, S);
            uint32_t word = bits << (8u * bsel);
            word |= __shfl_xor_sync(kFull, word, 1);
            word |= __shfl_xor_sync(kFull, word, 2);
            if (bsel == 0u) sbits[(wb >> 5) + (lane >> 2)] = word;
        }
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) part[0] = acc;
        if (sscale) finish_segment(spart, sscale, done, first, tb.off, tb.tile_first, tb.pbase, tb.tile);
        return;
    }
    if (vec_ok && first == last && base + tb.tile <= tb.d) {
        constexpr int kSpan = 128 * VPT;                  // coordinates per warp per iteration
        constexpr int kIter = kSpan * (kBlock / 32);      // per block per iteration
        const bool multi = n > kNC;
        const int g = lane >> 3, sh = (lane & 7) * 4;
        // the table serves the first nt workers (only in the 8-coordinates-per-thread layout)
        const int nt = (multi || VPT != 2) ? 0 : min(n, kTabWorkers);
        if (!multi) {
            if (threadIdx.x < n) ssm[threadIdx.x] = ld_cg_f32(wscale + (int64_t)threadIdx.x * tb.q + first);
            __syncthreads();
            if (nt > 0) {
                if (threadIdx.x < (1 << nt)) {
                    float t = 0.0f;
                    for (int i = 0; i < nt; ++i) t = __fadd_rn(t, signed_scale((threadIdx.x >> i) & 1u, ssm[i]));
                    tab[threadIdx.x] = t;
                }
                __syncthreads();
            }
        }
        dd acc = {0.0, 0.0};
        for (int it = 0; it < tb.tile / kIter; ++it) {
            const int64_t wb = base + (int64_t)it * kIter + warp * kSpan;
            float4 H[VPT], Gt[VPT];
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                const int64_t j = wb + v * 128 + lane * 4;
                H[v] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                if (!EF) H[v] = ld_rw4(ghat_s + j);      // error feedback overwrites this buffer
                Gt[v] = MODE == 2 ? make_float4(0.0f, 0.0f, 0.0f, 0.0f) : ld_ro4(gtil + j);
            }
            float a[VPT][4];
#pragma unroll
            for (int v = 0; v < VPT; ++v) a[v][0] = a[v][1] = a[v][2] = a[v][3] = 0.0f;
            for (int i0 = 0; i0 < n; i0 += kNC) {        // workers in increasing order
                const int nc = min(kNC, n - i0);
                if (multi) {
                    __syncthreads();
                    if (threadIdx.x < nc) ssm[threadIdx.x] = ld_cg_f32(wscale + (int64_t)(i0 + threadIdx.x) * tb.q + first);
                } else {
                    __syncwarp();
                }
                for (int idx = lane; idx < nc * 4 * VPT; idx += 32) {
                    const int i = idx / (4 * VPT), wd = idx % (4 * VPT);
                    wsm[warp][i][wd & 3][wd >> 2] = ld_cg_u32(wbits + (int64_t)(i0 + i) * wp + (wb >> 5) + wd);
                }
                if (multi) __syncthreads(); else __syncwarp();
                if constexpr (VPT == 2) {
                    if (nt > 0) {
                        // byte i = worker i's sign bits of this thread's 8 coordinates; after the
                        // transpose byte j = the workers' sign bits (the pattern) of coordinate j
                        uint32_t lo = 0u, hi = 0u;
#pragma unroll
                        for (int i = 0; i < kTabWorkers; ++i) {
                            if (i < nt) {
                                const uint2 q2 = *reinterpret_cast<const uint2 *>(&wsm[warp][i][g][0]);
                                const uint32_t b8 = ((q2.x >> sh) & 0xFu) | (((q2.y >> sh) & 0xFu) << 4);
                                if (i < 4) lo |= b8 << (8 * i); else hi |= b8 << (8 * (i - 4));
                            }
                        }
                        const uint64_t pat = transpose8x8(((uint64_t)hi << 32) | lo);
                        const uint32_t plo = (uint32_t)pat, phi = (uint32_t)(pat >> 32);
                        a[0][0] = tab[plo & 0xFFu];         a[0][1] = tab[(plo >> 8) & 0xFFu];
                        a[0][2] = tab[(plo >> 16) & 0xFFu]; a[0][3] = tab[plo >> 24];
                        a[1][0] = tab[phi & 0xFFu];         a[1][1] = tab[(phi >> 8) & 0xFFu];
                        a[1][2] = tab[(phi >> 16) & 0xFFu]; a[1][3] = tab[phi >> 24];
                    }
                }
#pragma unroll 4
                for (int i = nt; i < nc; ++i) {
                    const float s = ssm[i];
                    uint32_t W[VPT];
                    if constexpr (VPT == 4) {
                        const uint4 q4 = *reinterpret_cast<const uint4 *>(&wsm[warp][i][g][0]);
                        W[0] = q4.x; W[1] = q4.y; W[2] = q4.z; W[3] = q4.w;
                    } else {
                        const uint2 q2 = *reinterpret_cast<const uint2 *>(&wsm[warp][i][g][0]);
                        W[0] = q2.x; W[1] = q2.y;
                    }
#pragma unroll
                    for (int v = 0; v < VPT; ++v) {
                        const uint32_t nib = W[v] >> sh;
                        a[v][0] = __fadd_rn(a[v][0], signed_scale(nib & 1u, s));
                        a[v][1] = __fadd_rn(a[v][1], signed_scale(nib & 2u, s));
                        a[v][2] = __fadd_rn(a[v][2], signed_scale(nib & 4u, s));
                        a[v][3] = __fadd_rn(a[v][3], signed_scale(nib & 8u, s));
                    }
                }
            }
            uint32_t B[4][4];
#pragma unroll
            for (int v = 0; v < 4; ++v) B[v][0] = B[v][1] = B[v][2] = B[v][3] = 0u;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                // sum / n: multiplication by 1/n is the same correctly rounded value as the
                // division when n is a power of two
                float m0, m1, m2, m3;
                if (n_pow2) {
                    m0 = __fmul_rn(a[v][0], rn); m1 = __fmul_rn(a[v][1], rn);
                    m2 = __fmul_rn(a[v][2], rn); m3 = __fmul_rn(a[v][3], rn);
                } else {
                    m0 = __fdiv_rn(a[v][0], fn); m1 = __fdiv_rn(a[v][1], fn);
                    m2 = __fdiv_rn(a[v][2], fn); m3 = __fdiv_rn(a[v][3], fn);
                }
                float4 S;
                const float wx = server_step<EF>(m0, H[v].x, Gt[v].x, S.x);
                const float wy = server_step<EF>(m1, H[v].y, Gt[v].y, S.y);
                const float wz = server_step<EF>(m2, H[v].z, Gt[v].z, S.z);
                const float ww = server_step<EF>(m3, H[v].w, Gt[v].w, S.w);
                st_rw4(ghat_s + wb + v * 128 + lane * 4, S);
                dd_acc(acc, fabsf(wx)); dd_acc(acc, fabsf(wy));
                dd_acc(acc, fabsf(wz)); dd_acc(acc, fabsf(ww));
                B[v][0] = __ballot_sync(kFull, wx >= 0.0f);
                B[v][1] = __ballot_sync(kFull, wy >= 0.0f);
                B[v][2] = __ballot_sync(kFull, wz >= 0.0f);
                B[v][3] = __ballot_sync(kFull, ww >= 0.0f);
            }
            const uint32_t word = warp_words(B, lane);
            if (lane < 4 * VPT) sbits[(wb >> 5) + lane] = word;
        }
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) part[0] = acc;
        if (sscale) finish_segment(spart, sscale, done, first, tb.off, tb.tile_first, tb.pbase, tb.tile);
        return;
    }

    const int64_t end = min(base + (int64_t)tb.tile, tb.d);
    for (int64_t j = base + threadIdx.x; j - lane < end; j += kBlock) {
        const bool valid = j < end;
        float w = -1.0f;
        if (valid) {
            const int r = find_segment(tb.off, first, last, j);
            float a = 0.0f;
            for (int i0 = 0; i0 < n; i0 += 8) {        // eight workers' loads in flight, then their additions in order
                uint32_t wd[8];
                float sc[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = min(i0 + u, n - 1);
                    wd[u] = ld_cg_u32(wbits + (int64_t)i * wp + (j >> 5));
                    sc[u] = ld_cg_f32(wscale + (int64_t)i * tb.q + r);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (i0 + u < n) a = __fadd_rn(a, signed_scale((wd[u] >> (j & 31)) & 1u, sc[u]));
            }
            float hn;
            w = server_step<EF>(__fdiv_rn(a, fn), EF ? 0.0f : ghat_s[j], MODE == 2 ? 0.0f : gtil[j], hn);
            ghat_s[j] = hn;
        }
        const uint32_t word = __ballot_sync(kFull, valid && w >= 0.0f);
        if (lane == 0) sbits[j >> 5] = word;
    }
    __syncthreads();
    for (int r = first; r <= last; ++r) {
        const int64_t lo = max(tb.off[r], base), hi = min(tb.off[r + 1], end);
        dd acc = {0.0, 0.0};
        for (int64_t j = lo + threadIdx.x; j < hi; j += kBlock)
            dd_acc(acc, fabsf(server_input_from_memory<EF>(ghat_s[j], EF ? 0.0f : gtil[j])));
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) part[r - first] = acc;
    }
    if (sscale)
        for (int r = first; r <= last; ++r)
            finish_segment(spart, sscale, done, r, tb.off, tb.tile_first, tb.pbase, tb.tile);
}

// ------------------------------------------------------------------------------------
// Server pass B + worker update.  grid = ceil(d / 1024): one float4 of each of the five
// vectors per thread.  This kernel has no reduction, and short blocks at full occupancy
// measured fastest for its ten streams (five read, five written).
// ------------------------------------------------------------------------------------
constexpr int kUpdSpan = kBlock * 4;

template <int MODE>
__global__ void __launch_bounds__(kBlock, 5)
k_update_sign(const uint32_t *__restrict__ sbits, const float *__restrict__ sscale,
              const float *__restrict__ ghat_s, float *__restrict__ gtil, float *__restrict__ m, float *__restrict__ v,
              float *__restrict__ vhat, float *__restrict__ x, Tables tb, Hyper hp, int vec_ok)
{
    constexpr bool EF = MODE == 1;
    const int64_t base = (int64_t)blockIdx.x * kUpdSpan;
    const int64_t T = base / tb.tile;

    if (vec_ok && base + kUpdSpan <= tb.d) {
        const int64_t j = base + threadIdx.x * 4;
        // error feedback reads the server's compressor input p (ghat buffer), not the old error;
        // naive compression reads and writes no compression state
        float4 Gt = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (MODE == 0) Gt = ld_rw4(gtil + j);           // no earlier kernel of the step writes gtil, m, v, vhat, x
        float4 M = ld_rw4(m + j), V = ld_rw4(v + j);
        float4 Vh = ld_rw4(vhat + j), X = ld_rw4(x + j);
        grid_dep_wait();                                // server sign words, scales (and p) come from the kernels before
        if (EF) Gt = ld_cg4(ghat_s + j);
        const uint32_t nib = ld_cg_u32(sbits + (j >> 5)) >> (j & 31);
        const int first = tb.tile_first[T], last = tb.tile_last[T];
        float s0, s1, s2, s3;
        s0 = s1 = s2 = s3 = ld_cg_f32(sscale + first);
        if (first != last) {                            // the tile spans several segments
            int r = find_segment(tb.off, first, last, j);
            s0 = ld_cg_f32(sscale + r);
            while (r < last && j + 1 >= tb.off[r + 1]) ++r;
            s1 = ld_cg_f32(sscale + r);
            while (r < last && j + 2 >= tb.off[r + 1]) ++r;
            s2 = ld_cg_f32(sscale + r);
            while (r < last && j + 3 >= tb.off[r + 1]) ++r;
            s3 = ld_cg_f32(sscale + r);
        }
        const float ex = update_step<MODE != 0>(Gt.x, Gt.x, signed_scale(nib & 1u, s0), Gt.x);
        const float ey = update_step<MODE != 0>(Gt.y, Gt.y, signed_scale(nib & 2u, s1), Gt.y);
        const float ez = update_step<MODE != 0>(Gt.z, Gt.z, signed_scale(nib & 4u, s2), Gt.z);
        const float ew = update_step<MODE != 0>(Gt.w, Gt.w, signed_scale(nib & 8u, s3), Gt.w);
        amsgrad1(ex, M.x, V.x, Vh.x, X.x, hp);
        amsgrad1(ey, M.y, V.y, Vh.y, X.y, hp);
        amsgrad1(ez, M.z, V.z, Vh.z, X.z, hp);
        amsgrad1(ew, M.w, V.w, Vh.w, X.w, hp);
        if (MODE != 2) st_rw4(gtil + j, Gt);
        st_rw4(m + j, M); st_rw4(v + j, V);
        st_rw4(vhat + j, Vh); st_rw4(x + j, X);
        return;
    }

    const int first = tb.tile_first[T], last = tb.tile_last[T];
    const int64_t end = min(base + (int64_t)kUpdSpan, tb.d);
    grid_dep_wait();
    for (int64_t j = base + threadIdx.x; j < end; j += kBlock) {
        const int r = find_segment(tb.off, first, last, j);
        const uint32_t bit = (ld_cg_u32(sbits + (j >> 5)) >> (j & 31)) & 1u;
        const float stored = MODE == 2 ? 0.0f : EF ? ld_cg_f32(ghat_s + j) : gtil[j];
        float gt;
        const float est = update_step<MODE != 0>(stored, stored, signed_scale(bit, ld_cg_f32(sscale + r)), gt);
        if (MODE != 2) gtil[j] = gt;
        float mm = m[j], vv = v[j], vh = vhat[j], xx = x[j];
        amsgrad1(est, mm, vv, vh, xx, hp);
        m[j] = mm; v[j] = vv; vhat[j] = vh; x[j] = xx;
    }
}

// ------------------------------------------------------------------------------------
// ghat_w += decode(bits, scales): applies a payload whose application was deferred.
// grid = (ntiles, n).
// ------------------------------------------------------------------------------------
template <bool EF>
__global__ void __launch_bounds__(kBlock)
k_apply_sign(float *__restrict__ ghat_w, const uint32_t *__restrict__ wbits,
             const float *__restrict__ scales, Tables tb, int64_t wp)
{
    const int i = blockIdx.y;
    const int64_t T = tb.order[blockIdx.x];
    const int first = tb.tile_first[T], last = tb.tile_last[T];
    const int64_t base = T * tb.tile, end = min(base + (int64_t)tb.tile, tb.d);
    float *gh = ghat_w + (int64_t)i * tb.d;
    const uint32_t *bw = wbits + (int64_t)i * wp;
    for (int64_t j = base + threadIdx.x; j < end; j += kBlock) {
        const int r = find_segment(tb.off, first, last, j);
        const uint32_t bit = (bw[j >> 5] >> (j & 31)) & 1u;
        const float c = signed_scale(bit, scales[(int64_t)i * tb.q + r]);
        gh[j] = EF ? __fsub_rn(gh[j], c) : __fadd_rn(gh[j], c);
    }
}

// ------------------------------------------------------------------------------------
// Compressor without state: sign bits of x and partial sums of |x|, for each of the rows of
// x (rows x d; bits rows x wp; partial sums rows x nparts).  grid = (ntiles, rows).
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBlock)
k_pack_sign(const float *__restrict__ x_all, uint32_t *__restrict__ bits_all, dd *__restrict__ part_all,
            Tables tb, int64_t wp, int vec_ok)
{
    const int64_t T = tb.order[blockIdx.x];
    const int first = tb.tile_first[T], last = tb.tile_last[T];
    const int64_t base = T * tb.tile;
    const float *x = x_all + (int64_t)blockIdx.y * tb.d;
    uint32_t *bits = bits_all + (int64_t)blockIdx.y * wp;
    dd *part = part_all + (int64_t)blockIdx.y * tb.nparts + tb.pbase[T];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    if (vec_ok && first == last && base + tb.tile <= tb.d) {
        dd acc = {0.0, 0.0};
        for (int it = 0; it < tb.tile / kSub; ++it) {
            const int64_t wb = base + (int64_t)it * kSub + warp * kWarpSpan;
            float4 X[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) X[v] = ld_ro4(x + wb + v * 128 + lane * 4);
            uint32_t B[4][4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                dd_acc(acc, fabsf(X[v].x)); dd_acc(acc, fabsf(X[v].y));
                dd_acc(acc, fabsf(X[v].z)); dd_acc(acc, fabsf(X[v].w));
                B[v][0] = __ballot_sync(kFull, X[v].x >= 0.0f);
                B[v][1] = __ballot_sync(kFull, X[v].y >= 0.0f);
                B[v][2] = __ballot_sync(kFull, X[v].z >= 0.0f);
                B[v][3] = __ballot_sync(kFull, X[v].w >= 0.0f);
            }
            const uint32_t word = warp_words(B, lane);
            if (lane < 16) bits[(wb >> 5) + lane] = word;
        }
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) part[0] = acc;
        return;
    }

    const int64_t end = min(base + (int64_t)tb.tile, tb.d);
    for (int64_t j = base + threadIdx.x; j - lane < end; j += kBlock) {
        const bool valid = j < end;
        const uint32_t word = __ballot_sync(kFull, valid && x[valid ? j : base] >= 0.0f);
        if (lane == 0) bits[j >> 5] = word;
    }
    for (int r = first; r <= last; ++r) {
        const int64_t lo = max(tb.off[r], base), hi = min(tb.off[r + 1], end);
        dd acc = {0.0, 0.0};
        for (int64_t j = lo + threadIdx.x; j < hi; j += kBlock) dd_acc(acc, fabsf(x[j]));
        acc = block_sum<kBlock>(acc);
        if (threadIdx.x == 0) part[r - first] = acc;
    }
}

// ------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------
template <typename G>
static void launch_worker_sign_t(const G *grads, float *ghat_w, uint32_t *wbits,
                                 const float *scale_old, dd *wpart, const Tables &tb, int n,
                                 int64_t wp, bool vec_ok, bool ef, int *error_flag, float *scale_new,
                                 unsigned int *done, cudaStream_t st, int wait_limit)
{
    dim3 grid((unsigned)tb.ntiles, (unsigned)n);
    if (vec_ok && tb.tile >= 4 * kSub) {
        auto kern = ef ? k_worker_sign_ring<true, G> : k_worker_sign_ring<false, G>;
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingSmemBytes);
        kern<<<grid, kBlock, kRingSmemBytes, st>>>(grads, ghat_w, wbits, scale_old, wpart, tb, wp, error_flag,
                                                   scale_new, done, wait_limit);
    } else {
        // 256-bit accesses: every row 32-byte aligned (state rows by d % 8; gradient rows by the
        // base address and d times the element size)
        const int vec8 = vec_ok && tb.d % 8 == 0 && ((uintptr_t)ghat_w & 31u) == 0 &&
                         ((uintptr_t)grads & (sizeof(G) == 4 ? 31u : 15u)) == 0;
        if (ef) k_worker_sign<true, G><<<grid, kBlock, 0, st>>>(grads, ghat_w, wbits, scale_old, wpart, tb, wp, vec_ok,
                                                                scale_new, done, vec8);
        else k_worker_sign<false, G><<<grid, kBlock, 0, st>>>(grads, ghat_w, wbits, scale_old, wpart, tb, wp, vec_ok,
                                                              scale_new, done, vec8);
    }
}

void launch_worker_sign(const void *grads, bool grads_bf16, float *ghat_w, uint32_t *wbits,
                        const float *scale_old, dd *wpart, const Tables &tb, int n,
                        int64_t wp, bool vec_ok, bool ef, int *error_flag, float *scale_new,
                        unsigned int *done, cudaStream_t st, int wait_limit)
{
    if (wait_limit < 0) wait_limit = kWaitLimit;
    if (grads_bf16)
        launch_worker_sign_t(static_cast<const bf16_t *>(grads), ghat_w, wbits, scale_old, wpart, tb, n, wp,
                             vec_ok, ef, error_flag, scale_new, done, st, wait_limit);
    else
        launch_worker_sign_t(static_cast<const float *>(grads), ghat_w, wbits, scale_old, wpart, tb, n, wp,
                             vec_ok, ef, error_flag, scale_new, done, st, wait_limit);
}

void launch_finalize_scales(const dd *part, float *scales, const Tables &tb, int rows,
                            cudaStream_t st, int split, dd *split_sums, unsigned int *split_done)
{
    if (split > 1) {
        dim3 grid((unsigned)tb.q, (unsigned)rows, (unsigned)split);
        launch_after(k_finalize_scales_split, grid, dim3(kFinBlock), 0, st, part, scales, tb, split_sums, split_done);
        return;
    }
    dim3 grid((unsigned)tb.q, (unsigned)rows);
    launch_after(k_finalize_scales, grid, dim3(kFinBlock), 0, st, part, scales, tb);
}

void launch_range_sums(const dd *part, dd *sums, const Tables &tb, int rows, const int32_t *gidx, int q_all,
                       cudaStream_t st)
{
    k_range_sums<<<dim3((unsigned)tb.q, (unsigned)rows), kFinBlock, 0, st>>>(part, sums, tb, gidx, q_all);
}

void launch_range_scales(const dd *all, int ranges, int rows, int q_all, const int32_t *gidx, const int64_t *glen,
                         float *scales, int q_loc, cudaStream_t st)
{
    k_range_scales<<<dim3((unsigned)((q_loc + kBlock - 1) / kBlock), (unsigned)rows), kBlock, 0, st>>>(
        all, ranges, q_all, gidx, glen, scales, q_loc);
}

void launch_server_sign(const uint32_t *wbits, const float *wscale, float *ghat_s,
                        const float *gtil, uint32_t *sbits, dd *spart, const Tables &tb,
                        int n, int64_t wp, bool vec_ok, int mode, float *sscale, unsigned int *done,
                        cudaStream_t st)
{
    const int pow2 = (n & (n - 1)) == 0;
    auto kern = mode == 2 ? k_server_sign<2, 2> : mode == 1 ? k_server_sign<2, 1> : k_server_sign<2, 0>;
    // 256-bit accesses need d % 8 == 0 (the vectors are the context's own: 256-byte aligned)
    const int vec8 = vec_ok && tb.d % 8 == 0 && (((uintptr_t)ghat_s | (uintptr_t)gtil) & 31u) == 0;
    launch_after(kern, dim3((unsigned)tb.ntiles), dim3(kBlock), 0, st, wbits, wscale, ghat_s, gtil, sbits, spart, tb, n, wp,
                 (int)vec_ok, pow2, sscale, done, vec8);
}

void launch_update_sign(const uint32_t *sbits, const float *sscale, const float *ghat_s, float *gtil,
                        float *m, float *v, float *vhat, float *x, const Tables &tb, Hyper hp,
                        bool vec_ok, int mode, cudaStream_t st)
{
    const unsigned blocks = (unsigned)((tb.d + kUpdSpan - 1) / kUpdSpan);
    auto kern = mode == 2 ? k_update_sign<2> : mode == 1 ? k_update_sign<1> : k_update_sign<0>;
    launch_after(kern, dim3(blocks), dim3(kBlock), 0, st, sbits, sscale, ghat_s, gtil, m, v, vhat, x, tb, hp, (int)vec_ok);
}

void launch_apply_sign(float *ghat_w, const uint32_t *wbits, const float *scales,
                       const Tables &tb, int n, int64_t wp, bool ef, cudaStream_t st)
{
    dim3 grid((unsigned)tb.ntiles, (unsigned)n);
    if (ef) k_apply_sign<true><<<grid, kBlock, 0, st>>>(ghat_w, wbits, scales, tb, wp);
    else k_apply_sign<false><<<grid, kBlock, 0, st>>>(ghat_w, wbits, scales, tb, wp);
}

void launch_pack_sign(const float *x, uint32_t *bits, dd *part, const Tables &tb, int rows,
                      int64_t wp, bool vec_ok, cudaStream_t st)
{
    dim3 grid((unsigned)tb.ntiles, (unsigned)rows);
    k_pack_sign<<<grid, kBlock, 0, st>>>(x, bits, part, tb, wp, vec_ok);
}

}  // namespace cdadam
