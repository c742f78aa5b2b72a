// cdadam_compress_sign_static: the flat scaled-sign compressor for callers that must not
// allocate device memory.
//
// Some users of this library run where a device allocation is not allowed: inside a
// region that must not synchronise the device (cudaMalloc and cudaFree may), in a process
// whose memory pool is owned and fully reserved by a framework, or under a real-time
// budget where an allocator call is an unbounded delay.  For them the per-tile partial
// sums of the l1 norm, the only scratch memory the compressor needs, live in a fixed array
// in the library's own device image instead of in memory taken from the allocator.
//
// The array is a file-scope device variable; its name in host code is only a handle.  The
// device address is looked up once per device with cudaGetSymbolAddress and that pointer
// is what the kernels receive.
#include <cstdio>
#include <mutex>

#include "../../include/cdadam.h"
#include "common.cuh"
#include "kernels.h"

namespace cdadam {

constexpr int kStaticTile = 4 * kSub;                                   // 16,384 coordinates
constexpr int64_t kStaticMaxParts = CDADAM_STATIC_MAX_D / kStaticTile;  // 16,384 partial sums
constexpr uint32_t kFullMask = 0xffffffffu;

// 256 KiB per device that loads the library, held until the process exits.
static __device__ __align__(256) dd g_static_parts[kStaticMaxParts];

// One block per tile: sign bits of x and the tile's double-double sum of |x| -> parts[T].
__global__ void __launch_bounds__(kBlock)
k_pack_sign_flat(const float *__restrict__ x, uint32_t *__restrict__ bits, dd *__restrict__ parts,
                 int64_t d, int vec_ok)
{
    const int64_t base = (int64_t)blockIdx.x * kStaticTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    dd acc = {0.0, 0.0};
    if (vec_ok && base + kStaticTile <= d) {
        for (int it = 0; it < kStaticTile / kSub; ++it) {
            const int64_t wb = base + (int64_t)it * kSub + warp * kWarpSpan;
            float4 X[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) X[v] = ld_ro4(x + wb + v * 128 + lane * 4);
            uint32_t B[4][4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                dd_acc(acc, fabsf(X[v].x)); dd_acc(acc, fabsf(X[v].y));
                dd_acc(acc, fabsf(X[v].z)); dd_acc(acc, fabsf(X[v].w));
                B[v][0] = __ballot_sync(kFullMask, X[v].x >= 0.0f);
                B[v][1] = __ballot_sync(kFullMask, X[v].y >= 0.0f);
                B[v][2] = __ballot_sync(kFullMask, X[v].z >= 0.0f);
                B[v][3] = __ballot_sync(kFullMask, X[v].w >= 0.0f);
            }
            const uint32_t word = warp_words(B, lane);
            if (lane < 16) bits[(wb >> 5) + lane] = word;
        }
    } else {
        const int64_t end = min(base + (int64_t)kStaticTile, d);
        for (int64_t j = base + threadIdx.x; j - lane < end; j += kBlock) {
            const bool valid = j < end;
            const float xv = valid ? x[j] : -1.0f;
            const uint32_t word = __ballot_sync(kFullMask, valid && xv >= 0.0f);
            if (lane == 0) bits[j >> 5] = word;
            if (valid) dd_acc(acc, fabsf(xv));
        }
    }
    acc = block_sum<kBlock>(acc);
    if (threadIdx.x == 0) parts[blockIdx.x] = acc;
}

// One block: the partial sums in a fixed order -> the correctly rounded scale.
__global__ void __launch_bounds__(512)
k_finalize_flat(const dd *__restrict__ parts, int64_t nparts, int64_t d, float *__restrict__ scale)
{
    dd acc = {0.0, 0.0};
    for (int64_t t = threadIdx.x; t < nparts; t += 512) acc = dd_add(acc, parts[t]);
    acc = block_sum<512>(acc);
    if (threadIdx.x == 0)
        *scale = __double2float_rn(__ddiv_rn(__dadd_rn(acc.hi, acc.lo), (double)d));
}

}  // namespace cdadam

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
cdadam::dd *g_parts_ptr[kMaxDevices] = {};

}  // namespace

extern "C" {

int cdadam_compress_sign_static(const float *x, int64_t d, uint32_t *bits, float *scale,
                                void *stream)
{
    using namespace cdadam;
    char msg[256];
    if (!x || !bits || !scale) {
        snprintf(msg, sizeof msg, "cdadam_compress_sign_static: NULL argument");
        set_last_error(msg);
        return CDADAM_ERR_ARG;
    }
    if (d < 1 || d > CDADAM_STATIC_MAX_D) {
        snprintf(msg, sizeof msg,
                 "cdadam_compress_sign_static: d = %lld is outside [1, %lld], the size the built-in "
                 "scratch array covers", (long long)d, (long long)CDADAM_STATIC_MAX_D);
        set_last_error(msg);
        return CDADAM_ERR_ARG;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        snprintf(msg, sizeof msg, "cdadam_compress_sign_static: no usable CUDA device");
        set_last_error(msg);
        return CDADAM_ERR_CUDA;
    }
    dd *parts = nullptr;
    {
        // set-up, once per device, with that device current: the device address of the array
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_parts_ptr[dev]) {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_parts);
            if (e != cudaSuccess || !p) {
                snprintf(msg, sizeof msg, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
                set_last_error(msg);
                return CDADAM_ERR_CUDA;
            }
            g_parts_ptr[dev] = static_cast<dd *>(p);
        }
        parts = g_parts_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t ntiles = (d + kStaticTile - 1) / kStaticTile;
    const int vec_ok = (((uintptr_t)x & 15u) == 0 && d % 4 == 0) ? 1 : 0;
    // every partial sum below ntiles is overwritten by its tile, none is accumulated into, so
    // nothing has to be cleared between calls
    k_pack_sign_flat<<<(unsigned)ntiles, kBlock, 0, st>>>(x, bits, parts, d, vec_ok);
    k_finalize_flat<<<1, 512, 0, st>>>(parts, ntiles, d, scale);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(msg, sizeof msg, "cdadam_compress_sign_static: %s", cudaGetErrorString(e));
        set_last_error(msg);
        return CDADAM_ERR_CUDA;
    }
    return CDADAM_OK;
}

}  // extern "C"
