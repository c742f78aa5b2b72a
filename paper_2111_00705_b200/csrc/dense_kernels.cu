// Dense kernels that need no compressor state: the identity-compressor iteration of
// Algorithm 1 fused into one pass, and the AMSGrad update alone (used after the top-k
// payload has been scattered into gtil).
#include "kernels.h"

namespace cdadam {

// C(u) = u: every line of Algorithm 1 for one coordinate, workers in increasing order.
// EF: the same with classical error feedback, whose error terms stay exactly zero.
template <int MODE>      // 0 = Algorithm 1, 1 = error feedback, 2 = naive (no state)
__global__ void __launch_bounds__(kBlock)
k_step_identity(const float *__restrict__ grads, float *__restrict__ ghat_w,
                float *__restrict__ ghat_s, float *__restrict__ gtil, float *__restrict__ m,
                float *__restrict__ v, float *__restrict__ vhat, float *__restrict__ x,
                int64_t d, int n, Hyper hp)
{
    constexpr bool EF = MODE == 1;
    const float fn = (float)n;
    for (int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x; j < d;
         j += (int64_t)gridDim.x * kBlock) {
        float a = 0.0f;
        for (int i = 0; i < n; ++i) {
            const int64_t p = (int64_t)i * d + j;
            if (MODE == 2) { a = __fadd_rn(a, grads[p]); continue; }
            const float gh = ghat_w[p];
            const float u = EF ? __fadd_rn(grads[p], gh) : __fsub_rn(grads[p], gh);   // c^(i) = u
            ghat_w[p] = EF ? __fsub_rn(u, u) : __fadd_rn(gh, u);
            a = __fadd_rn(a, u);
        }
        float gt;
        if (MODE == 2) {
            gt = __fdiv_rn(a, fn);
        } else if (EF) {
            gt = __fadd_rn(__fdiv_rn(a, fn), gtil[j]);         // c = p, the error p - c is zero
            gtil[j] = __fsub_rn(gt, gt);
        } else {
            const float hs = __fadd_rn(ghat_s[j], __fdiv_rn(a, fn));
            ghat_s[j] = hs;
            const float gt0 = gtil[j];
            gt = __fadd_rn(gt0, __fsub_rn(hs, gt0));           // c = w
            gtil[j] = gt;
        }
        float mm = m[j], vv = v[j], vh = vhat[j], xx = x[j];
        amsgrad1(gt, mm, vv, vh, xx, hp);
        m[j] = mm; v[j] = vv; vhat[j] = vh; x[j] = xx;
    }
}

// One float4 of each of the five vectors per thread, no loop: short blocks at full occupancy
// keep the most loads in flight for 5 read and 4 written streams.  grid = ceil(d / 1024).
__global__ void __launch_bounds__(kBlock, 5)
k_amsgrad(const float *__restrict__ gtil, float *__restrict__ m, float *__restrict__ v,
          float *__restrict__ vhat, float *__restrict__ x, int64_t d, Hyper hp, int vec_ok)
{
    const int64_t j = ((int64_t)blockIdx.x * kBlock + threadIdx.x) * 4;
    if (vec_ok && j + 4 <= d) {
        const float4 G = ld_ro4(gtil + j);
        float4 M = ld_rw4(m + j), V = ld_rw4(v + j), Vh = ld_rw4(vhat + j), X = ld_rw4(x + j);
        amsgrad1(G.x, M.x, V.x, Vh.x, X.x, hp);
        amsgrad1(G.y, M.y, V.y, Vh.y, X.y, hp);
        amsgrad1(G.z, M.z, V.z, Vh.z, X.z, hp);
        amsgrad1(G.w, M.w, V.w, Vh.w, X.w, hp);
        st_rw4(m + j, M); st_rw4(v + j, V); st_rw4(vhat + j, Vh); st_rw4(x + j, X);
        return;
    }
    const int64_t end = j + 4 < d ? j + 4 : d;
    for (int64_t i = j; i < end; ++i) {
        float mm = m[i], vv = v[i], vh = vhat[i], xx = x[i];
        amsgrad1(gtil[i], mm, vv, vh, xx, hp);
        m[i] = mm; v[i] = vv; vhat[i] = vh; x[i] = xx;
    }
}

static unsigned grid_for(int64_t items)
{
    int64_t blocks = (items + kBlock - 1) / kBlock;
    const int64_t cap = 148 * 16;
    return (unsigned)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

void launch_step_identity(const float *grads, float *ghat_w, float *ghat_s, float *gtil,
                          float *m, float *v, float *vhat, float *x, int64_t d, int n,
                          Hyper hp, int mode, cudaStream_t st)
{
    if (mode == 2) k_step_identity<2><<<grid_for(d), kBlock, 0, st>>>(grads, ghat_w, ghat_s, gtil, m, v, vhat, x, d, n, hp);
    else if (mode == 1) k_step_identity<1><<<grid_for(d), kBlock, 0, st>>>(grads, ghat_w, ghat_s, gtil, m, v, vhat, x, d, n, hp);
    else k_step_identity<0><<<grid_for(d), kBlock, 0, st>>>(grads, ghat_w, ghat_s, gtil, m, v, vhat, x, d, n, hp);
}

// exact widening bfloat16 -> binary32
__global__ void __launch_bounds__(kBlock)
k_widen_bf16(float *__restrict__ dst, const uint16_t *__restrict__ src, int64_t count)
{
    for (int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x; j < count; j += (int64_t)gridDim.x * kBlock)
        dst[j] = __uint_as_float((uint32_t)src[j] << 16);
}

void launch_widen_bf16(float *dst, const void *src, int64_t count, cudaStream_t st)
{
    k_widen_bf16<<<grid_for(count), kBlock, 0, st>>>(dst, static_cast<const uint16_t *>(src), count);
}

// dst = src + dst
__global__ void __launch_bounds__(kBlock)
k_add_into(float *__restrict__ dst, const float *__restrict__ src, int64_t count, int vec_ok)
{
    const int64_t nvec = vec_ok ? count / 4 : 0;
    const int64_t stride = (int64_t)gridDim.x * kBlock;
    const int64_t t0 = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    for (int64_t q = t0; q < nvec; q += stride) {
        const float4 a = ld_ro4(src + q * 4);
        float4 b = ld_rw4(dst + q * 4);
        b.x = __fadd_rn(a.x, b.x); b.y = __fadd_rn(a.y, b.y);
        b.z = __fadd_rn(a.z, b.z); b.w = __fadd_rn(a.w, b.w);
        st_rw4(dst + q * 4, b);
    }
    for (int64_t j = nvec * 4 + t0; j < count; j += stride) dst[j] = __fadd_rn(src[j], dst[j]);
}

void launch_add_into(float *dst, const float *src, int64_t count, bool vec_ok, cudaStream_t st)
{
    k_add_into<<<grid_for(vec_ok ? count / 4 : count), kBlock, 0, st>>>(dst, src, count, vec_ok);
}

__global__ void __launch_bounds__(kBlock)
k_scatter_set(float *__restrict__ dst, const uint32_t *__restrict__ idx, const float *__restrict__ val,
              int64_t k, int64_t d)
{
    const int row = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t < k) dst[(int64_t)row * d + idx[(int64_t)row * k + t]] = val ? val[(int64_t)row * k + t] : 0.0f;
}

// dst[idx[row][t]] = 0 for every row: one vector, the coordinate sets of all rows
__global__ void __launch_bounds__(kBlock)
k_scatter_zero_shared(float *__restrict__ dst, const uint32_t *__restrict__ idx, int64_t k)
{
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t < k) dst[idx[(int64_t)blockIdx.y * k + t]] = 0.0f;
}

void launch_scatter_zero_shared(float *dst, const uint32_t *idx, int64_t k, int rows, cudaStream_t st)
{
    dim3 grid((unsigned)((k + kBlock - 1) / kBlock), (unsigned)rows);
    k_scatter_zero_shared<<<grid, kBlock, 0, st>>>(dst, idx, k);
}

void launch_scatter_set(float *dst, const uint32_t *idx, const float *val, int64_t k, int64_t d,
                        int rows, cudaStream_t st)
{
    dim3 grid((unsigned)((k + kBlock - 1) / kBlock), (unsigned)rows);
    k_scatter_set<<<grid, kBlock, 0, st>>>(dst, idx, val, k, d);
}

// dst[idx[t]] += val[t] for one message of k distinct coordinates (a worker applying the
// server's top-k message to its copy of gtil); coordinates >= d are skipped.
__global__ void __launch_bounds__(kBlock)
k_scatter_add(float *__restrict__ dst, const uint32_t *__restrict__ idx, const float *__restrict__ val,
              int64_t k, int64_t d)
{
    const int64_t t = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (t >= k) return;
    const int64_t j = idx[t];
    if (j < d) dst[j] = __fadd_rn(dst[j], val[t]);
}

void launch_scatter_add(float *dst, const uint32_t *idx, const float *val, int64_t k, int64_t d, cudaStream_t st)
{
    k_scatter_add<<<(unsigned)((k + kBlock - 1) / kBlock), kBlock, 0, st>>>(dst, idx, val, k, d);
}

void launch_amsgrad(const float *gtil, float *m, float *v, float *vhat, float *x, int64_t d,
                    Hyper hp, bool vec_ok, cudaStream_t st)
{
    k_amsgrad<<<(unsigned)((d + 4 * kBlock - 1) / (4 * kBlock)), kBlock, 0, st>>>(gtil, m, v, vhat, x, d, hp, vec_ok);
}

}  // namespace cdadam
