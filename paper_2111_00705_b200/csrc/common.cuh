// Shared device helpers of the CD-Adam kernels (sm_100a): double-double accumulation of
// the l1 norm, fixed-order block reductions, streaming 128-bit memory accesses, sign-bit
// packing, and the tile / segment tables.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cdadam {

constexpr int kBlock = 256;            // threads per block of every streaming kernel
constexpr int kSub = 4096;             // elements one block handles per inner iteration
constexpr int kWarpSpan = kSub / (kBlock / 32);   // 512 consecutive elements per warp

// ------------------------------------------------------------------------------------
// Tile and segment tables (device pointers).  The index space [0, d) is cut into tiles of
// `tile` elements (a multiple of kSub).  tile_first/tile_last give the first and last
// segment that overlaps a tile; a tile writes one partial l1 sum per overlapped segment at
// pbase[T] + (r - tile_first[T]).  Block b of a streaming kernel works on tile order[b]:
// the few tiles that need the slower scalar path (segment boundaries, the ragged tail) come
// first so that they overlap with the bulk instead of forming the kernel's tail.
// ------------------------------------------------------------------------------------
struct Tables {
    int64_t d;
    int q;
    int tile;
    int64_t ntiles;
    int64_t nparts;
    const int64_t *off;        // q+1 segment offsets
    const int32_t *tile_first; // ntiles
    const int32_t *tile_last;  // ntiles
    const int64_t *pbase;      // ntiles
    const int32_t *order;      // ntiles: permutation of the tiles, slow tiles first
};

// ------------------------------------------------------------------------------------
// Double-double arithmetic.  The l1 norm of a segment is accumulated as an unevaluated
// sum hi + lo of two doubles with error-free additions, so the result carries about 100
// significant bits; rounding it to binary64 gives the correctly rounded sum of the
// binary32 magnitudes whatever the launch shape.
// ------------------------------------------------------------------------------------
struct dd {
    double hi, lo;
};

// a += x  (x >= 0 exactly converted from binary32); Knuth's two-sum keeps the rounding
// error of hi + x in lo.
__device__ __forceinline__ void dd_acc(dd &a, float x)
{
    const double xd = (double)x;
    const double s = __dadd_rn(a.hi, xd);
    const double bb = __dsub_rn(s, a.hi);
    const double e = __dadd_rn(__dsub_rn(a.hi, __dsub_rn(s, bb)), __dsub_rn(xd, bb));
    a.lo = __dadd_rn(a.lo, e);
    a.hi = s;
}

// a + b, renormalised.
__device__ __forceinline__ dd dd_add(dd a, dd b)
{
    const double s = __dadd_rn(a.hi, b.hi);
    const double bb = __dsub_rn(s, a.hi);
    double e = __dadd_rn(__dsub_rn(a.hi, __dsub_rn(s, bb)), __dsub_rn(b.hi, bb));
    e = __dadd_rn(e, __dadd_rn(a.lo, b.lo));
    dd r;
    r.hi = __dadd_rn(s, e);
    r.lo = __dsub_rn(e, __dsub_rn(r.hi, s));
    return r;
}

__device__ __forceinline__ dd dd_shfl_down(dd a, int delta)
{
    dd r;
    r.hi = __shfl_down_sync(0xffffffffu, a.hi, delta);
    r.lo = __shfl_down_sync(0xffffffffu, a.lo, delta);
    return r;
}

// Sum over the block in a fixed tree order; the result is valid in thread 0.
// All threads of the block must call it.  `NT` = block size (multiple of 32, <= 1024).
template <int NT>
__device__ __forceinline__ dd block_sum(dd a)
{
    __shared__ double sh_hi[NT / 32], sh_lo[NT / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int delta = 16; delta >= 1; delta >>= 1) a = dd_add(a, dd_shfl_down(a, delta));
    __syncthreads();   // protects sh_* against the previous call's readers
    if (lane == 0) { sh_hi[warp] = a.hi; sh_lo[warp] = a.lo; }
    __syncthreads();
    if (warp == 0) {
        dd b;
        b.hi = lane < NT / 32 ? sh_hi[lane] : 0.0;
        b.lo = lane < NT / 32 ? sh_lo[lane] : 0.0;
#pragma unroll
        for (int delta = 16; delta >= 1; delta >>= 1) b = dd_add(b, dd_shfl_down(b, delta));
        a = b;
    }
    return a;
}

// ------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel queued with launch_after() may be scheduled while
// the kernel before it in the stream is still running: its blocks start, run up to
// grid_dep_wait() and stop there until the earlier kernel has finished and its writes are
// visible.  Everything a kernel reads that an earlier kernel of the same step writes must
// therefore be read after grid_dep_wait(); what precedes it (table look-ups, loads of
// vectors no earlier kernel of the step writes) overlaps the earlier kernel's tail and the
// launch latency.  grid_dep_launch() in the earlier kernel lets the next one be scheduled as
// soon as all of its own blocks have started.  Both are no-ops in a kernel launched the
// ordinary way.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... P, typename... A>
inline cudaError_t launch_after(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

// ------------------------------------------------------------------------------------
// 128-bit global memory accesses.  Read-only streams (gradients, payload bits) use the
// non-coherent path without L1 allocation; read-modify-write state uses streaming
// (evict-first) loads and stores: every vector is touched once per kernel.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ float4 ld_ro4(const float *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_rw4(const float *p)
{
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void st_rw4(float *p, float4 v)
{
    __stcs(reinterpret_cast<float4 *>(p), v);
}
__device__ __forceinline__ uint32_t ld_ro_u32(const uint32_t *p) { return __ldg(p); }
// 256-bit accesses (eight consecutive floats of one thread, 32-byte aligned): a warp then
// covers 1 KiB of a vector with whole 32-byte sectors per thread.
__device__ __forceinline__ void ld_ro8(const float *p, float (&v)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}
__device__ __forceinline__ void ld_rw8(const float *p, float (&v)[8])
{
    asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p) : "memory");
}
__device__ __forceinline__ void st_rw8(float *p, const float (&v)[8])
{
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]),
                 "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}
// Coherent (L2) loads for what the kernel queued just before wrote: under programmatic
// dependent launch this grid is already resident while that kernel runs, so such data is not
// read-only for this grid's lifetime and must not go through the non-coherent path.
__device__ __forceinline__ uint32_t ld_cg_u32(const uint32_t *p) { return __ldcg(p); }
__device__ __forceinline__ float ld_cg_f32(const float *p) { return __ldcg(p); }
__device__ __forceinline__ float4 ld_cg4(const float *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }

// ------------------------------------------------------------------------------------
// Plain bulk asynchronous copies (TMA, one-dimensional, one destination block) global -> shared, completed
// on an mbarrier.  Addresses and sizes must be multiples of 16 bytes.  Every wait is
// bounded: a barrier that does not complete makes the caller report an error and leave.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, int arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals));
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n.reg .pred p;\n"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                 "selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return done != 0;
}
constexpr int kWaitLimit = 1 << 22;     // try_wait attempts before a wait gives up (default)
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, int limit = kWaitLimit)
{
    for (int spin = 0; spin < limit; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_copy_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes,
                                              uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

// ------------------------------------------------------------------------------------
// Sign-bit packing.  In the vector kernels lane L of a warp holds the four consecutive
// coordinates 4L..4L+3 of a 128-coordinate group, so the ballot over component c has bit L
// = sign of coordinate 4L + c.  Word g (coordinates 32g..32g+31) of the group is the
// 4-way bit interleave of byte g of the four ballots.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t spread4(uint32_t t)   // bit j (j < 8) -> bit 4j
{
    t = (t | (t << 12)) & 0x000F000Fu;
    t = (t | (t << 6)) & 0x03030303u;
    t = (t | (t << 3)) & 0x11111111u;
    return t;
}
__device__ __forceinline__ uint32_t interleave_word(uint32_t b0, uint32_t b1, uint32_t b2,
                                                    uint32_t b3, int g)
{
    const int sh = 8 * g;
    return spread4((b0 >> sh) & 0xFFu) | (spread4((b1 >> sh) & 0xFFu) << 1) |
           (spread4((b2 >> sh) & 0xFFu) << 2) | (spread4((b3 >> sh) & 0xFFu) << 3);
}

// Lane L < 16 returns word L of the warp's 512-coordinate span: B[v][c] is the ballot of
// component c in 128-coordinate group v (identical in all lanes).
__device__ __forceinline__ uint32_t warp_words(const uint32_t (&B)[4][4], int lane)
{
    const int v = (lane >> 2) & 3;
    uint32_t b[4];
#pragma unroll
    for (int c = 0; c < 4; ++c)
        b[c] = v == 0 ? B[0][c] : v == 1 ? B[1][c] : v == 2 ? B[2][c] : B[3][c];
    return interleave_word(b[0], b[1], b[2], b[3], lane & 3);
}

// Segment that holds coordinate j, searched in [lo, hi] (both inclusive, off[lo] <= j).
__device__ __forceinline__ int find_segment(const int64_t *off, int lo, int hi, int64_t j)
{
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (off[mid] <= j) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ------------------------------------------------------------------------------------
// AMSGrad update of one coordinate (the last four assignments of Algorithm 1): nu inside the root, no bias
// correction, one rounding per operation, no fused multiply-add.  With a weight decay
// lambda (Section 6; decoupled form) x also loses (alpha lambda) x_t.
// ------------------------------------------------------------------------------------
struct Hyper {
    float beta1, beta2, omb1, omb2, lr, nu;   // omb = 1 - beta, rounded once in binary32
    float lrwd;                               // alpha * lambda, rounded once in binary32
    int decay;                                // lambda != 0
};

__device__ __forceinline__ void amsgrad1(float gt, float &m, float &v, float &vh, float &x,
                                         const Hyper &hp)
{
    m = __fadd_rn(__fmul_rn(hp.beta1, m), __fmul_rn(hp.omb1, gt));
    v = __fadd_rn(__fmul_rn(hp.beta2, v), __fmul_rn(hp.omb2, __fmul_rn(gt, gt)));
    vh = vh >= v ? vh : v;
    const float xo = x;
    x = __fsub_rn(xo, __fdiv_rn(__fmul_rn(hp.lr, m), __fsqrt_rn(__fadd_rn(vh, hp.nu))));
    if (hp.decay) x = __fsub_rn(x, __fmul_rn(hp.lrwd, xo));
}

}  // namespace cdadam
