// Layer glue around the ternary contractions (Sec. 2.4: a ternary block is conv, affine,
// ReLU, pooling; Algorithm 1 back-propagates through them the standard way).  All tensors
// are NHWC bf16; arithmetic is fp32; every kernel is a plain bandwidth-bound sweep with
// 16-byte accesses along the channel dimension where the channel count allows it.
#include <cuda_bf16.h>

#include "common.cuh"

namespace {

constexpr int kT = 256;

inline int blocks_for(long long items, int sm_count)
{
    long long b = (items + kT - 1) / kT;
    const long long cap = (long long)sm_count * 16;
    if (b > cap) b = cap;
    if (b < 1) b = 1;
    return (int)b;
}

// ---- im2col: rows = output pixels, columns = (r, s, c), zero outside the image and past K
__global__ void __launch_bounds__(kT)
im2col_kernel(const __nv_bfloat16 *__restrict__ X, twn_conv_desc_t d, long long Ho, long long Wo,
              __nv_bfloat16 *__restrict__ out, long long ldk)
{
    const long long K = (long long)d.kh * d.kw * d.Cin;
    const long long chunks = ldk / 8;                 // 8 columns (16 bytes) per thread
    const long long total = d.B * Ho * Wo * chunks;
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < total; i += (long long)gridDim.x * kT) {
        const long long m = i / chunks;
        const int k0 = (int)(i - m * chunks) * 8;
        const long long wo = m % Wo, ho = (m / Wo) % Ho, b = m / (Wo * Ho);
        __align__(16) __nv_bfloat16 v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int k = k0 + e;
            __nv_bfloat16 x = __float2bfloat16_rn(0.0f);
            if (k < K) {
                const int c = k % (int)d.Cin, t = k / (int)d.Cin;
                const int s = t % d.kw, r = t / d.kw;
                const long long h = ho * d.stride_h - d.pad_h + r, w = wo * d.stride_w - d.pad_w + s;
                if (h >= 0 && h < d.H && w >= 0 && w < d.W) x = X[((b * d.H + h) * d.W + w) * d.Cin + c];
            }
            v[e] = x;
        }
        *reinterpret_cast<uint4 *>(out + m * ldk + k0) = *reinterpret_cast<const uint4 *>(v);
    }
}

// ---- max pooling, window k x k, -inf padding; the first maximum in scan order wins
__global__ void __launch_bounds__(kT)
maxpool_fwd_kernel(const __nv_bfloat16 *__restrict__ X, long long B, long long H, long long W, long long C,
                   int k, int stride, int pad, long long Ho, long long Wo,
                   __nv_bfloat16 *__restrict__ Y, uint8_t *__restrict__ idx)
{
    const long long total = B * Ho * Wo * C;
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < total; i += (long long)gridDim.x * kT) {
        const long long c = i % C, wo = (i / C) % Wo, ho = (i / (C * Wo)) % Ho, b = i / (C * Wo * Ho);
        float best = -INFINITY;
        int arg = 0;
        __nv_bfloat16 bestv = __float2bfloat16_rn(0.0f);
        for (int r = 0; r < k; ++r) {
            const long long h = ho * stride - pad + r;
            if (h < 0 || h >= H) continue;
            for (int s = 0; s < k; ++s) {
                const long long w = wo * stride - pad + s;
                if (w < 0 || w >= W) continue;
                const __nv_bfloat16 xv = X[((b * H + h) * W + w) * C + c];
                const float x = __bfloat162float(xv);
                if (x > best) { best = x; bestv = xv; arg = r * k + s; }
            }
        }
        Y[i] = bestv;
        if (idx) idx[i] = (uint8_t)arg;
    }
}

// gather form: an input pixel collects the gradient of every window whose maximum it was
__global__ void __launch_bounds__(kT)
maxpool_bwd_kernel(const __nv_bfloat16 *__restrict__ dY, const uint8_t *__restrict__ idx, long long B, long long H,
                   long long W, long long C, int k, int stride, int pad, long long Ho, long long Wo,
                   __nv_bfloat16 *__restrict__ dX)
{
    const long long total = B * H * W * C;
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < total; i += (long long)gridDim.x * kT) {
        const long long c = i % C, w = (i / C) % W, h = (i / (C * W)) % H, b = i / (C * W * H);
        float g = 0.0f;
        for (int r = 0; r < k; ++r) {
            const long long hn = h + pad - r;
            if (hn < 0 || hn % stride != 0) continue;
            const long long ho = hn / stride;
            if (ho >= Ho) continue;
            for (int s = 0; s < k; ++s) {
                const long long wn = w + pad - s;
                if (wn < 0 || wn % stride != 0) continue;
                const long long wo = wn / stride;
                if (wo >= Wo) continue;
                const long long o = ((b * Ho + ho) * Wo + wo) * C + c;
                if (idx[o] == r * k + s) g += __bfloat162float(dY[o]);
            }
        }
        dX[i] = __float2bfloat16_rn(g);
    }
}

// ---- global average pooling [B,H,W,C] -> [B,C] and its backward
__global__ void __launch_bounds__(kT)
avgpool_fwd_kernel(const __nv_bfloat16 *__restrict__ X, long long B, long long HW, long long C,
                   __nv_bfloat16 *__restrict__ Y)
{
    const long long total = B * C;
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < total; i += (long long)gridDim.x * kT) {
        const long long c = i % C, b = i / C;
        float s = 0.0f;
        for (long long p = 0; p < HW; ++p) s += __bfloat162float(X[(b * HW + p) * C + c]);
        Y[i] = __float2bfloat16_rn(s / (float)HW);
    }
}

__global__ void __launch_bounds__(kT)
avgpool_bwd_kernel(const __nv_bfloat16 *__restrict__ dY, long long B, long long HW, long long C,
                   __nv_bfloat16 *__restrict__ dX)
{
    const long long total = B * HW * C;
    const float inv = 1.0f / (float)HW;
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < total; i += (long long)gridDim.x * kT) {
        const long long c = i % C, b = i / (C * HW);
        dX[i] = __float2bfloat16_rn(__bfloat162float(dY[b * C + c]) * inv);
    }
}

// ---- backward through y = relu(z * scale[c] + shift[c] (+ residual)):
//   dPre = dY * [Y > 0]  (or dY when Y is NULL: no ReLU),  dZ = dPre * scale[c]
__global__ void __launch_bounds__(kT)
act_bwd_kernel(const __nv_bfloat16 *__restrict__ dY, const __nv_bfloat16 *__restrict__ Y,
               const float *__restrict__ scale, long long n, long long C,
               __nv_bfloat16 *__restrict__ dZ, __nv_bfloat16 *__restrict__ dPre)
{
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < n; i += (long long)gridDim.x * kT) {
        float g = __bfloat162float(dY[i]);
        if (Y && !(__bfloat162float(Y[i]) > 0.0f)) g = 0.0f;
        if (dPre) dPre[i] = __float2bfloat16_rn(g);
        if (dZ) dZ[i] = __float2bfloat16_rn(scale ? g * __ldg(scale + i % C) : g);
    }
}

int pool_extent(long long in, int k, int stride, int pad) { return (int)((in + 2 * pad - k) / stride + 1); }

}  // namespace

extern "C" int twn_im2col(const twn_conv_desc_t *d, const void *X, void *Xcol, int64_t ldk, twn_stream_t stream)
{
    TWN_REQUIRE(d && X && Xcol, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->B > 0 && d->H > 0 && d->W > 0 && d->Cin > 0 && d->kh > 0 && d->kw > 0 && d->stride_h > 0 &&
                    d->stride_w > 0 && d->pad_h >= 0 && d->pad_w >= 0, TWN_ERR_INVALID_ARG);
    const long long K = (long long)d->kh * d->kw * d->Cin;
    TWN_REQUIRE(ldk >= K && ldk % 8 == 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(Xcol, 16) && twn_aligned(X, 2), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long Ho = (d->H + 2 * d->pad_h - d->kh) / d->stride_h + 1, Wo = (d->W + 2 * d->pad_w - d->kw) / d->stride_w + 1;
    TWN_REQUIRE(Ho > 0 && Wo > 0, TWN_ERR_INVALID_ARG);
    const long long items = d->B * Ho * Wo * (ldk / 8);
    im2col_kernel<<<blocks_for(items, dev.sm_count), kT, 0, twn_cu(stream)>>>(
        static_cast<const __nv_bfloat16 *>(X), *d, Ho, Wo, static_cast<__nv_bfloat16 *>(Xcol), ldk);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_maxpool2d_fwd(const void *X, int64_t B, int64_t H, int64_t W, int64_t C, int k, int stride,
                                 int pad, void *Y, uint8_t *argmax, twn_stream_t stream)
{
    TWN_REQUIRE(X && Y && B > 0 && H > 0 && W > 0 && C > 0 && k > 0 && k <= 15 && stride > 0 && pad >= 0 && pad < k,
                TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long Ho = pool_extent(H, k, stride, pad), Wo = pool_extent(W, k, stride, pad);
    TWN_REQUIRE(Ho > 0 && Wo > 0, TWN_ERR_INVALID_ARG);
    maxpool_fwd_kernel<<<blocks_for(B * Ho * Wo * C, dev.sm_count), kT, 0, twn_cu(stream)>>>(
        static_cast<const __nv_bfloat16 *>(X), B, H, W, C, k, stride, pad, Ho, Wo, static_cast<__nv_bfloat16 *>(Y), argmax);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_maxpool2d_bwd(const void *dY, const uint8_t *argmax, int64_t B, int64_t H, int64_t W, int64_t C,
                                 int k, int stride, int pad, void *dX, twn_stream_t stream)
{
    TWN_REQUIRE(dY && argmax && dX && B > 0 && H > 0 && W > 0 && C > 0 && k > 0 && k <= 15 && stride > 0 &&
                    pad >= 0 && pad < k, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long Ho = pool_extent(H, k, stride, pad), Wo = pool_extent(W, k, stride, pad);
    TWN_REQUIRE(Ho > 0 && Wo > 0, TWN_ERR_INVALID_ARG);
    maxpool_bwd_kernel<<<blocks_for(B * H * W * C, dev.sm_count), kT, 0, twn_cu(stream)>>>(
        static_cast<const __nv_bfloat16 *>(dY), argmax, B, H, W, C, k, stride, pad, Ho, Wo, static_cast<__nv_bfloat16 *>(dX));
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_avgpool_fwd(const void *X, int64_t B, int64_t HW, int64_t C, void *Y, twn_stream_t stream)
{
    TWN_REQUIRE(X && Y && B > 0 && HW > 0 && C > 0, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    avgpool_fwd_kernel<<<blocks_for(B * C, dev.sm_count), kT, 0, twn_cu(stream)>>>(
        static_cast<const __nv_bfloat16 *>(X), B, HW, C, static_cast<__nv_bfloat16 *>(Y));
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_avgpool_bwd(const void *dY, int64_t B, int64_t HW, int64_t C, void *dX, twn_stream_t stream)
{
    TWN_REQUIRE(dY && dX && B > 0 && HW > 0 && C > 0, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    avgpool_bwd_kernel<<<blocks_for(B * HW * C, dev.sm_count), kT, 0, twn_cu(stream)>>>(
        static_cast<const __nv_bfloat16 *>(dY), B, HW, C, static_cast<__nv_bfloat16 *>(dX));
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_act_bwd(const void *dY, const void *Y, const float *scale, int64_t n, int64_t C, void *dZ,
                           void *dPre, twn_stream_t stream)
{
    TWN_REQUIRE(dY && n >= 0 && C > 0 && (dZ || dPre), TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    if (n == 0) return TWN_OK;
    act_bwd_kernel<<<blocks_for(n, dev.sm_count), kT, 0, twn_cu(stream)>>>(
        static_cast<const __nv_bfloat16 *>(dY), static_cast<const __nv_bfloat16 *>(Y), scale, n, C,
        static_cast<__nv_bfloat16 *>(dZ), static_cast<__nv_bfloat16 *>(dPre));
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}
