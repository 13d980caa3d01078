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

// Index arithmetic is 32-bit whenever the tensors allow it (64-bit division is an order of
// magnitude slower on the GPU); `I` is int or long long.

// ---- im2col: rows = output pixels, columns = (r, s, c), zero outside the image and past K
template <typename I>
__global__ void __launch_bounds__(kT)
im2col_kernel(const __nv_bfloat16 *__restrict__ X, twn_conv_desc_t d, I Ho, I Wo,
              __nv_bfloat16 *__restrict__ out, I ldk)
{
    const int K = d.kh * d.kw * (int)d.Cin, Cin = (int)d.Cin;
    const I chunks = ldk / 8;                 // 8 columns (16 bytes) per thread
    const I total = (I)d.B * Ho * Wo * chunks;
    const I H = (I)d.H, W = (I)d.W;
    for (I i = (I)blockIdx.x * kT + threadIdx.x; i < total; i += (I)gridDim.x * kT) {
        const I m = i / chunks;
        const int k0 = (int)(i - m * chunks) * 8;
        const I wo = m % Wo, t1 = m / Wo, ho = t1 % Ho, b = t1 / Ho;
        int t = k0 / Cin, c = k0 - t * Cin;
        int r = t / d.kw, sx = t - r * d.kw;
        __align__(16) __nv_bfloat16 v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            __nv_bfloat16 x = __float2bfloat16_rn(0.0f);
            if (k0 + e < K) {
                const I h = ho * d.stride_h - d.pad_h + r, w = wo * d.stride_w - d.pad_w + sx;
                if (h >= 0 && h < H && w >= 0 && w < W) x = X[((b * H + h) * W + w) * Cin + c];
            }
            v[e] = x;
            if (++c == Cin) { c = 0; if (++sx == d.kw) { sx = 0; ++r; } }
        }
        *reinterpret_cast<uint4 *>(out + m * ldk + k0) = *reinterpret_cast<const uint4 *>(v);
    }
}

// Patch variant for short rows (small Cin): a block takes 64 consecutive output pixels of one
// output row.  The input window they read (kh rows of (63*stride_w + kw) pixels) is copied to
// shared memory with zeros outside the image; the shared-memory offset of every patch column is
// tabulated once; then each warp writes whole patch rows, one 16-byte chunk per lane, so that a
// store instruction covers a contiguous run of the output.
constexpr int kPatchPix = 64;
constexpr int kPatchMaxElems = 12288;   // window elements (24 KB)
constexpr int kPatchMaxCols = 1024;     // ldk

__global__ void __launch_bounds__(kT)
im2col_patch_kernel(const __nv_bfloat16 *__restrict__ X, twn_conv_desc_t d, int Ho, int Wo, int wseg,
                    __nv_bfloat16 *__restrict__ out, int ldk, int win_w)
{
    extern __shared__ __align__(16) unsigned char smem_patch[];
    __nv_bfloat16 *win = reinterpret_cast<__nv_bfloat16 *>(smem_patch);       // [kh][win_w * Cin] (+1 zero at the end)
    int *tab = reinterpret_cast<int *>(smem_patch + ((size_t)(d.kh * win_w * (int)d.Cin + 1) * 2 + 15) / 16 * 16);
    const int Cin = (int)d.Cin, K = d.kh * d.kw * Cin, row_el = win_w * Cin, zero_at = d.kh * row_el;
    int blk = blockIdx.x;
    const int seg = blk % wseg; blk /= wseg;
    const int ho = blk % Ho, b = blk / Ho;
    const int wo0 = seg * kPatchPix;
    const int h0 = ho * d.stride_h - d.pad_h, w0 = wo0 * d.stride_w - d.pad_w;
    const int H = (int)d.H, W = (int)d.W;
    for (int i = threadIdx.x; i < zero_at + 1; i += kT) {
        const int r = i / row_el, j = i - r * row_el;
        const int w = w0 + j / Cin, h = h0 + r;
        __nv_bfloat16 x = __float2bfloat16_rn(0.0f);
        if (i < zero_at && h >= 0 && h < H && w >= 0 && w < W)
            x = X[(((long long)b * H + h) * W + w0) * Cin + j];
        win[i] = x;
    }
    for (int k = threadIdx.x; k < ldk; k += kT) {
        int off = zero_at;                       // columns K..ldk-1 read the zero
        if (k < K) {
            const int t = k / Cin, c = k - t * Cin, r = t / d.kw, sx = t - r * d.kw;
            off = r * row_el + sx * Cin + c;
        }
        tab[k] = off;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunks = ldk >> 3;
    const int step = d.stride_w * Cin;           // window elements between neighbouring output pixels
    const int npix = Wo - wo0 < kPatchPix ? Wo - wo0 : kPatchPix;
    __nv_bfloat16 *const orow = out + (((long long)b * Ho + ho) * Wo + wo0) * ldk;
    for (int ch = lane; ch < chunks; ch += 32) {
        int o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = tab[ch * 8 + e];
        for (int p = warp; p < npix; p += kT / 32) {
            __align__(16) __nv_bfloat16 v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = win[o[e] == zero_at ? zero_at : o[e] + p * step];
            *reinterpret_cast<uint4 *>(orow + (long long)p * ldk + ch * 8) = *reinterpret_cast<const uint4 *>(v);
        }
    }
}

__device__ __forceinline__ void unpack8(const uint4 v, float (&f)[8])
{
    const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 t = __bfloat1622float2(p[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    uint4 v;
    __nv_bfloat162 *p = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
}

// ---- max pooling, window k x k, -inf padding; the first maximum in scan order wins.
// V = 8: eight channels per thread with 16-byte accesses (C % 8 == 0); V = 1: any C.
template <typename I, int V>
__global__ void __launch_bounds__(kT)
maxpool_fwd_kernel(const __nv_bfloat16 *__restrict__ X, I B, I H, I W, I C,
                   int k, int stride, int pad, I Ho, I Wo,
                   __nv_bfloat16 *__restrict__ Y, uint8_t *__restrict__ idx)
{
    const I Cv = C / V;
    const I total = B * Ho * Wo * Cv;
    for (I i = (I)blockIdx.x * kT + threadIdx.x; i < total; i += (I)gridDim.x * kT) {
        const I cv = i % Cv, t1 = i / Cv, wo = t1 % Wo, t2 = t1 / Wo, ho = t2 % Ho, b = t2 / Ho;
        float best[V];
        int arg[V];
#pragma unroll
        for (int e = 0; e < V; ++e) { best[e] = -INFINITY; arg[e] = 0; }
        for (int r = 0; r < k; ++r) {
            const I h = ho * stride - pad + r;
            if (h < 0 || h >= H) continue;
            for (int s = 0; s < k; ++s) {
                const I w = wo * stride - pad + s;
                if (w < 0 || w >= W) continue;
                const __nv_bfloat16 *src = X + ((b * H + h) * W + w) * C + cv * V;
                float x[V];
                if (V == 8) {
                    float t8[8];
                    unpack8(__ldg(reinterpret_cast<const uint4 *>(src)), t8);
#pragma unroll
                    for (int e = 0; e < V; ++e) x[e] = t8[e];
                } else {
                    x[0] = __bfloat162float(src[0]);
                }
#pragma unroll
                for (int e = 0; e < V; ++e)
                    if (x[e] > best[e]) { best[e] = x[e]; arg[e] = r * k + s; }
            }
        }
        const I o = ((b * Ho + ho) * Wo + wo) * C + cv * V;
        if (V == 8) {
            float t8[8];
#pragma unroll
            for (int e = 0; e < V; ++e) t8[e] = best[e] == -INFINITY ? 0.0f : best[e];
            *reinterpret_cast<uint4 *>(Y + o) = pack8(t8);     // exact: the values are bf16 already
            if (idx) {
                uint2 a;
                a.x = arg[0] | (arg[1 % V] << 8) | (arg[2 % V] << 16) | (arg[3 % V] << 24);
                a.y = arg[4 % V] | (arg[5 % V] << 8) | (arg[6 % V] << 16) | (arg[7 % V] << 24);
                *reinterpret_cast<uint2 *>(idx + o) = a;
            }
        } else {
            Y[o] = __float2bfloat16_rn(best[0] == -INFINITY ? 0.0f : best[0]);
            if (idx) idx[o] = (uint8_t)arg[0];
        }
    }
}

// t[e] = 0 where the pooled value (the window's maximum, i.e. the ReLU output at the arg-max) is not positive
__device__ __forceinline__ void gate8(float (&t)[8], const uint4 pooled)
{
    float p[8];
    unpack8(pooled, p);
#pragma unroll
    for (int e = 0; e < 8; ++e) t[e] = p[e] > 0.0f ? t[e] : 0.0f;
}

// gather form: an input pixel collects the gradient of every window whose maximum it was
template <typename I, int V>
__global__ void __launch_bounds__(kT)
maxpool_bwd_kernel(const __nv_bfloat16 *__restrict__ dY, const uint8_t *__restrict__ idx, I B, I H,
                   I W, I C, int k, int stride, int pad, I Ho, I Wo,
                   __nv_bfloat16 *__restrict__ dX, const __nv_bfloat16 *__restrict__ pooled,
                   const float *__restrict__ scale)
{
    const I Cv = C / V;
    const I total = B * H * W * Cv;
    for (I i = (I)blockIdx.x * kT + threadIdx.x; i < total; i += (I)gridDim.x * kT) {
        const I cv = i % Cv, t1 = i / Cv, w = t1 % W, t2 = t1 / W, h = t2 % H, b = t2 / H;
        float g[V];
#pragma unroll
        for (int e = 0; e < V; ++e) g[e] = 0.0f;
        for (int r = 0; r < k; ++r) {
            const I hn = h + pad - r;
            if (hn < 0 || hn % stride != 0) continue;
            const I ho = hn / stride;
            if (ho >= Ho) continue;
            for (int s = 0; s < k; ++s) {
                const I wn = w + pad - s;
                if (wn < 0 || wn % stride != 0) continue;
                const I wo = wn / stride;
                if (wo >= Wo) continue;
                const I o = ((b * Ho + ho) * Wo + wo) * C + cv * V;
                const int want = r * k + s;
                if (V == 8) {
                    const uint2 a = __ldg(reinterpret_cast<const uint2 *>(idx + o));
                    float t8[8];
                    unpack8(__ldg(reinterpret_cast<const uint4 *>(dY + o)), t8);
                    if (pooled) gate8(t8, __ldg(reinterpret_cast<const uint4 *>(pooled + o)));
#pragma unroll
                    for (int e = 0; e < V; ++e) {
                        const int ai = ((e < 4 ? a.x : a.y) >> (8 * (e & 3))) & 0xFF;
                        if (ai == want) g[e] += t8[e];
                    }
                } else {
                    if (idx[o] == want && (!pooled || __bfloat162float(pooled[o]) > 0.0f)) g[0] += __bfloat162float(dY[o]);
                }
            }
        }
        const I o = ((b * H + h) * W + w) * C + cv * V;
        if (scale) {
#pragma unroll
            for (int e = 0; e < V; ++e) g[e] *= __ldg(scale + cv * V + e);
        }
        if (V == 8) {
            float t8[8];
#pragma unroll
            for (int e = 0; e < V; ++e) t8[e] = g[e];
            *reinterpret_cast<uint4 *>(dX + o) = pack8(t8);
        } else {
            dX[o] = __float2bfloat16_rn(g[0]);
        }
    }
}

// 0xFFFF in each half where the bf16 value of a is greater than (equal to) that of b; false for NaN
__device__ __forceinline__ uint32_t greater_mask(uint32_t a, uint32_t b)
{
    return __hgt2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
}
__device__ __forceinline__ uint32_t equal_mask(uint32_t a, uint32_t b)
{
    return __heq2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
}

// Variants of the two pooling kernels for the common case (8 channels per thread, 32-bit
// indices).  The forward one takes one window per thread over the flat index; in the backward one
// a block walks whole image rows, and a power-of-two stride turns the window search into shifts.
// These sweeps are otherwise bound by their index arithmetic, not by memory.
__global__ void __launch_bounds__(kT)
maxpool_fwd_vec_kernel(const __nv_bfloat16 *__restrict__ X, int B, int H, int W, int C, int k, int stride, int pad,
                        int Ho, int Wo, __nv_bfloat16 *__restrict__ Y, uint8_t *__restrict__ idx)
{
    const int Cv = C >> 3, per_row = Wo * Cv, total = B * Ho * per_row;
    // one window (8 channels) per thread over the flat index: every block has the same work
    for (int it = blockIdx.x * kT + threadIdx.x; it < total; it += gridDim.x * kT) {
        const int row = it / per_row, i = it - row * per_row;
        const int b = row / Ho, ho = row - b * Ho;
        const int h_lo = ho * stride - pad;
        const int wo = i / Cv, cv = i - wo * Cv;
        const int w_lo = wo * stride - pad;
        float best[8];
        int arg[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { best[e] = -INFINITY; arg[e] = 0; }
        if (k <= 3) {
            // all (up to nine) window elements are requested before the first comparison, so
            // their latencies overlap; an element outside the image reads as -inf and never wins
            uint4 v[9];
#pragma unroll
            for (int q = 0; q < 9; ++q) {
                const int r = q / 3, sx = q - 3 * r;
                const int h = h_lo + r, w = w_lo + sx;
                const bool ok = r < k && sx < k && h >= 0 && h < H && w >= 0 && w < W;
                v[q] = ok ? __ldg(reinterpret_cast<const uint4 *>(X + ((size_t)(b * H + h) * W + w) * C + cv * 8))
                          : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // bf16 -inf
            }
            // two channels per register: the comparison yields a mask per bf16 half, and the
            // maximum and its tap (16 bits each until the end) are selected with it
            uint32_t bp[4], ap[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) { bp[p] = 0xFF80FF80u; ap[p] = 0u; }
#pragma unroll
            for (int q = 0; q < 9; ++q) {
                const int r = q / 3, sx = q - 3 * r;
                const uint32_t tap2 = (uint32_t)(r * k + sx) * 0x00010001u;
                const uint32_t x4[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const uint32_t m = greater_mask(x4[p], bp[p]);      // false for NaN, as x > best is
                    bp[p] = (x4[p] & m) | (bp[p] & ~m);
                    ap[p] = (tap2 & m) | (ap[p] & ~m);
                }
            }
            // a maximum still at -inf is written as zero
#pragma unroll
            for (int p = 0; p < 4; ++p) bp[p] &= ~equal_mask(bp[p], 0xFF80FF80u);
            const size_t o = ((size_t)row * Wo + wo) * C + cv * 8;
            *reinterpret_cast<uint4 *>(Y + o) = make_uint4(bp[0], bp[1], bp[2], bp[3]);
            if (idx) {
                uint2 a;        // the low byte of each 16-bit tap
                asm("prmt.b32 %0, %1, %2, 0x6420;" : "=r"(a.x) : "r"(ap[0]), "r"(ap[1]));
                asm("prmt.b32 %0, %1, %2, 0x6420;" : "=r"(a.y) : "r"(ap[2]), "r"(ap[3]));
                *reinterpret_cast<uint2 *>(idx + o) = a;
            }
            continue;
        } else
        for (int r = 0; r < k; ++r) {
            const int h = h_lo + r;
            if (h < 0 || h >= H) continue;
            const __nv_bfloat16 *rowp = X + ((size_t)(b * H + h) * W) * C + cv * 8;
            for (int sx = 0; sx < k; ++sx) {
                const int w = w_lo + sx;
                if (w < 0 || w >= W) continue;
                float x[8];
                unpack8(__ldg(reinterpret_cast<const uint4 *>(rowp + (size_t)w * C)), x);
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (x[e] > best[e]) { best[e] = x[e]; arg[e] = r * k + sx; }
            }
        }
        const size_t o = ((size_t)row * Wo + wo) * C + cv * 8;
        float t8[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) t8[e] = best[e] == -INFINITY ? 0.0f : best[e];
        *reinterpret_cast<uint4 *>(Y + o) = pack8(t8);     // exact: the values are bf16 already
        if (idx) {
            uint2 a;
            a.x = arg[0] | (arg[1] << 8) | (arg[2] << 16) | (arg[3] << 24);
            a.y = arg[4] | (arg[5] << 8) | (arg[6] << 16) | (arg[7] << 24);
            *reinterpret_cast<uint2 *>(idx + o) = a;
        }
    }
}

// bit 7 of each byte of the result is set where that byte of t is zero (exact for every byte value)
__device__ __forceinline__ uint32_t zero_bytes(uint32_t t)
{
    return ~(((t & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | t);
}
// bytes of the result, low to high: sign of byte s0 of z twice, sign of byte s1 twice (prmt's replicate mode)
template <uint32_t SEL>
__device__ __forceinline__ uint32_t pair_mask(uint32_t z)
{
    uint32_t m;
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(m) : "r"(z), "r"(SEL));
    return m;
}
// g += the bf16 values of d whose arg-max byte equals the tap (want4 = the tap in all four bytes)
__device__ __forceinline__ void add_matching(float (&g)[8], const uint2 a, const uint4 d, uint32_t want4)
{
    const uint32_t zx = zero_bytes(a.x ^ want4), zy = zero_bytes(a.y ^ want4);
    const uint32_t v0 = d.x & pair_mask<0x9988u>(zx), v1 = d.y & pair_mask<0xBBAAu>(zx);
    const uint32_t v2 = d.z & pair_mask<0x9988u>(zy), v3 = d.w & pair_mask<0xBBAAu>(zy);
    g[0] += __uint_as_float(v0 << 16); g[1] += __uint_as_float(v0 & 0xFFFF0000u);
    g[2] += __uint_as_float(v1 << 16); g[3] += __uint_as_float(v1 & 0xFFFF0000u);
    g[4] += __uint_as_float(v2 << 16); g[5] += __uint_as_float(v2 & 0xFFFF0000u);
    g[6] += __uint_as_float(v3 << 16); g[7] += __uint_as_float(v3 & 0xFFFF0000u);
}
// 0xFFFF in each half whose bf16 value is greater than zero (false for NaN)
__device__ __forceinline__ uint32_t positive_mask(uint32_t pair)
{
    return greater_mask(pair, 0u);
}

// k = 3, stride 2, pad 1.  An even input row (column) lies in one window, at tap 1; an odd one in
// two, at tap 2 of the window before and tap 0 of the window after.  One thread takes a 2 x 2 block
// of input pixels (8 channels): the four windows around it are loaded once, gated once, and feed
// 1 + 2 + 2 + 4 pixel-window pairs with no divergence.
__global__ void __launch_bounds__(kT)
maxpool_bwd_k3s2_kernel(const __nv_bfloat16 *__restrict__ dY, const uint8_t *__restrict__ idx, int B, int H, int W,
                        int C, int Ho, int Wo, __nv_bfloat16 *__restrict__ dX,
                        const __nv_bfloat16 *__restrict__ pooled, const float *__restrict__ scale)
{
    const int Cv = C >> 3, Hb = (H + 1) >> 1, Wb = (W + 1) >> 1;
    const int items = B * Hb * Wb * Cv;
    for (int it = blockIdx.x * kT + threadIdx.x; it < items; it += gridDim.x * kT) {
        int t = it / Cv;
        const int cv = it - t * Cv;
        const int i = t % Wb;
        t /= Wb;
        const int j = t % Hb, b = t / Hb;
        uint2 a[4];
        uint4 d[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int ho = j + (q >> 1), wo = i + (q & 1);
            const bool ok = ho < Ho && wo < Wo;
            const size_t o = ok ? ((size_t)(b * Ho + ho) * Wo + wo) * C + cv * 8 : 0;
            // an absent window's 0xFF bytes match no tap
            a[q] = ok ? __ldg(reinterpret_cast<const uint2 *>(idx + o)) : make_uint2(0xFFFFFFFFu, 0xFFFFFFFFu);
            d[q] = ok ? __ldg(reinterpret_cast<const uint4 *>(dY + o)) : make_uint4(0u, 0u, 0u, 0u);
            if (pooled) {
                const uint4 pl = ok ? __ldg(reinterpret_cast<const uint4 *>(pooled + o)) : make_uint4(0u, 0u, 0u, 0u);
                d[q].x &= positive_mask(pl.x); d[q].y &= positive_mask(pl.y);
                d[q].z &= positive_mask(pl.z); d[q].w &= positive_mask(pl.w);
            }
        }
        float4 s0 = make_float4(1.0f, 1.0f, 1.0f, 1.0f), s1 = s0;
        if (scale) {
            s0 = __ldg(reinterpret_cast<const float4 *>(scale + cv * 8));
            s1 = __ldg(reinterpret_cast<const float4 *>(scale + cv * 8 + 4));
        }
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
#pragma unroll
            for (int pc = 0; pc < 2; ++pc) {
                const int h = 2 * j + pr, w = 2 * i + pc;
                float g[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) g[e] = 0.0f;
                // later windows first, as the general kernels add them
#pragma unroll
                for (int dj = pr; dj >= 0; --dj) {
#pragma unroll
                    for (int di = pc; di >= 0; --di) {
                        const int r = pr == 0 ? 1 : (dj == 0 ? 2 : 0), sx = pc == 0 ? 1 : (di == 0 ? 2 : 0);
                        add_matching(g, a[dj * 2 + di], d[dj * 2 + di], (uint32_t)(r * 3 + sx) * 0x01010101u);
                    }
                }
                if (scale) {
                    g[0] *= s0.x; g[1] *= s0.y; g[2] *= s0.z; g[3] *= s0.w;
                    g[4] *= s1.x; g[5] *= s1.y; g[6] *= s1.z; g[7] *= s1.w;
                }
                if (h < H && w < W)
                    *reinterpret_cast<uint4 *>(dX + ((size_t)(b * H + h) * W + w) * C + cv * 8) = pack8(g);
            }
        }
    }
}

__global__ void __launch_bounds__(kT)
maxpool_bwd_rows_kernel(const __nv_bfloat16 *__restrict__ dY, const uint8_t *__restrict__ idx, int B, int H, int W,
                        int C, int k, int stride, int lg_stride, int pad, int Ho, int Wo,
                        __nv_bfloat16 *__restrict__ dX, const __nv_bfloat16 *__restrict__ pooled,
                        const float *__restrict__ scale)
{
    const int Cv = C >> 3, per_row = W * Cv;
    // window row / column that covers input coordinate x with tap t: (x + pad - t) / stride when divisible
    auto window = [&](int xn, int limit) -> int {
        if (xn < 0) return -1;
        int q;
        if (lg_stride >= 0) {
            if (xn & (stride - 1)) return -1;
            q = xn >> lg_stride;
        } else {
            q = xn / stride;
            if (q * stride != xn) return -1;
        }
        return q < limit ? q : -1;
    };
    for (int row = blockIdx.x; row < B * H; row += gridDim.x) {
        const int b = row / H, h = row - b * H;
        if (k <= 2 * stride) {
            // At most two windows per dimension cover a pixel: their argmax bytes and gradients
            // (up to four of each) are loaded before any of them is used, so the loads overlap.
            int hos[2] = {0, 0}, rs[2] = {0, 0}, nh = 0;
            for (int r = 0; r < k; ++r) {
                const int ho = window(h + pad - r, Ho);
                if (ho >= 0 && nh < 2) { hos[nh] = ho; rs[nh] = r; ++nh; }
            }
            for (int i = threadIdx.x; i < per_row; i += kT) {
                const int w = i / Cv, cv = i - w * Cv;
                int wos[2] = {0, 0}, sxs[2] = {0, 0}, nw = 0;
                for (int sx = 0; sx < k; ++sx) {
                    const int wo = window(w + pad - sx, Wo);
                    if (wo >= 0 && nw < 2) { wos[nw] = wo; sxs[nw] = sx; ++nw; }
                }
                uint2 a[4];
                uint4 d[4], pl[4];
                int want[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int ih = q >> 1, iw = q & 1;
                    const bool ok = ih < nh && iw < nw;
                    const size_t o = ((size_t)(b * Ho + hos[ih]) * Wo + wos[iw]) * C + cv * 8;   // in range also when !ok
                    a[q] = ok ? __ldg(reinterpret_cast<const uint2 *>(idx + o)) : make_uint2(0xFFFFFFFFu, 0xFFFFFFFFu);
                    d[q] = ok ? __ldg(reinterpret_cast<const uint4 *>(dY + o)) : make_uint4(0u, 0u, 0u, 0u);
                    if (pooled) pl[q] = ok ? __ldg(reinterpret_cast<const uint4 *>(pooled + o)) : make_uint4(0u, 0u, 0u, 0u);
                    want[q] = rs[ih] * k + sxs[iw];     // < 255: an absent window's 0xFF bytes never match
                }
                float g[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) g[e] = 0.0f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float t8[8];
                    unpack8(d[q], t8);
                    if (pooled) gate8(t8, pl[q]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int ai = ((e < 4 ? a[q].x : a[q].y) >> (8 * (e & 3))) & 0xFF;
                        if (ai == want[q]) g[e] += t8[e];
                    }
                }
                if (scale) {
                    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(scale + cv * 8));
                    const float4 s1 = __ldg(reinterpret_cast<const float4 *>(scale + cv * 8 + 4));
                    g[0] *= s0.x; g[1] *= s0.y; g[2] *= s0.z; g[3] *= s0.w;
                    g[4] *= s1.x; g[5] *= s1.y; g[6] *= s1.z; g[7] *= s1.w;
                }
                *reinterpret_cast<uint4 *>(dX + ((size_t)row * W + w) * C + cv * 8) = pack8(g);
            }
            continue;
        }
        for (int i = threadIdx.x; i < per_row; i += kT) {
            const int w = i / Cv, cv = i - w * Cv;
            float g[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = 0.0f;
            for (int r = 0; r < k; ++r) {
                const int ho = window(h + pad - r, Ho);
                if (ho < 0) continue;
                for (int sx = 0; sx < k; ++sx) {
                    const int wo = window(w + pad - sx, Wo);
                    if (wo < 0) continue;
                    const size_t o = ((size_t)(b * Ho + ho) * Wo + wo) * C + cv * 8;
                    const int want = r * k + sx;
                    const uint2 a = __ldg(reinterpret_cast<const uint2 *>(idx + o));
                    float t8[8];
                    unpack8(__ldg(reinterpret_cast<const uint4 *>(dY + o)), t8);
                    if (pooled) gate8(t8, __ldg(reinterpret_cast<const uint4 *>(pooled + o)));
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int ai = ((e < 4 ? a.x : a.y) >> (8 * (e & 3))) & 0xFF;
                        if (ai == want) g[e] += t8[e];
                    }
                }
            }
            if (scale) {
#pragma unroll
                for (int e = 0; e < 8; ++e) g[e] *= __ldg(scale + cv * 8 + e);
            }
            *reinterpret_cast<uint4 *>(dX + ((size_t)row * W + w) * C + cv * 8) = pack8(g);
        }
    }
}

// ---- folded input of a stride-2 layer with very few channels (the first layer of ResNet-18):
// the 2 x 2 pixel block at (2i - pad_h, 2j - pad_w) becomes the 4*Cin <= 16 channels of folded
// pixel (i, j), so that the stride-2 k x k layer is a stride-1 ceil(k/2) x ceil(k/2) layer and the
// four folded pixels a filter row touches are 64 consecutive bf16 (one tensor-core k-block).
// CIN > 0 fixes the channel count at compile time (the 16 values then stay in registers)
template <int CIN>
__global__ void __launch_bounds__(kT)
fold_input_kernel(const __nv_bfloat16 *__restrict__ X, int B, int H, int W, int Cin_rt, int pad_h, int pad_w, int Hf,
                  int Wf, __nv_bfloat16 *__restrict__ Xf)
{
    const int Cin = CIN > 0 ? CIN : Cin_rt;
    const int total = B * Hf * Wf;
    for (int p = blockIdx.x * kT + threadIdx.x; p < total; p += gridDim.x * kT) {
        const int j = p % Wf, t = p / Wf, i = t % Hf, b = t / Hf;
        __align__(16) __nv_bfloat16 v[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = __float2bfloat16_rn(0.0f);
#pragma unroll
        for (int dy = 0; dy < 2; ++dy) {
            const int h = 2 * i + dy - pad_h;
#pragma unroll
            for (int dx = 0; dx < 2; ++dx) {
                const int w = 2 * j + dx - pad_w;
                if (h < 0 || h >= H || w < 0 || w >= W) continue;
                const __nv_bfloat16 *src = X + ((size_t)(b * H + h) * W + w) * Cin;
                if (CIN > 0) {
#pragma unroll
                    for (int c = 0; c < CIN; ++c) v[(dy * 2 + dx) * CIN + c] = src[c];
                } else {
                    for (int c = 0; c < Cin; ++c) v[(dy * 2 + dx) * Cin + c] = src[c];
                }
            }
        }
        uint4 *dst = reinterpret_cast<uint4 *>(Xf + (size_t)p * 16);
        dst[0] = reinterpret_cast<const uint4 *>(v)[0];
        dst[1] = reinterpret_cast<const uint4 *>(v)[1];
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

// 8 channels per thread (C a multiple of 8, 32-bit indices).  Forward: a block takes 32 channel
// groups of one image, its 8 warps share the pixels, the partial sums meet in shared memory in a
// fixed order.  Backward: one 16-byte store per thread.
__global__ void __launch_bounds__(kT)
avgpool_fwd_vec_kernel(const __nv_bfloat16 *__restrict__ X, int HW, int C, int groups, __nv_bfloat16 *__restrict__ Y)
{
    __shared__ float part[kT / 32][32][9];
    const int Cv = C >> 3, b = blockIdx.x / groups, cv = (blockIdx.x - b * groups) * 32 + (threadIdx.x & 31);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float s[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) s[e] = 0.0f;
    if (cv < Cv)
        for (int p = warp; p < HW; p += kT / 32) {
            float x[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(X + ((size_t)b * HW + p) * C + cv * 8)), x);
#pragma unroll
            for (int e = 0; e < 8; ++e) s[e] += x[e];
        }
#pragma unroll
    for (int e = 0; e < 8; ++e) part[warp][lane][e] = s[e];
    __syncthreads();
    const int col = threadIdx.x & 31, e = threadIdx.x >> 5;     // 256 threads = 32 groups x 8 channels
    const int c = ((blockIdx.x - b * groups) * 32 + col) * 8 + e;
    if (c < C) {
        float t = 0.0f;
#pragma unroll
        for (int w = 0; w < kT / 32; ++w) t += part[w][col][e];
        Y[(size_t)b * C + c] = __float2bfloat16_rn(t / (float)HW);
    }
}

__global__ void __launch_bounds__(kT)
avgpool_bwd_vec_kernel(const __nv_bfloat16 *__restrict__ dY, int total, int HW, int C, __nv_bfloat16 *__restrict__ dX)
{
    const int Cv = C >> 3;
    const float inv = 1.0f / (float)HW;
    for (int i = blockIdx.x * kT + threadIdx.x; i < total; i += gridDim.x * kT) {
        const int pix = i / Cv, cv = i - pix * Cv, b = pix / HW;
        float g[8];
        unpack8(__ldg(reinterpret_cast<const uint4 *>(dY + (size_t)b * C + cv * 8)), g);
#pragma unroll
        for (int e = 0; e < 8; ++e) g[e] *= inv;
        *reinterpret_cast<uint4 *>(dX + (size_t)i * 8) = pack8(g);
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

// eight elements per thread (C % 8 == 0, 16-byte aligned tensors)
__global__ void __launch_bounds__(kT)
act_bwd_vec_kernel(const uint4 *__restrict__ dY, const uint4 *__restrict__ Y, const float *__restrict__ scale,
                   long long n8, int C8, uint4 *__restrict__ dZ, uint4 *__restrict__ dPre)
{
    for (long long i = (long long)blockIdx.x * kT + threadIdx.x; i < n8; i += (long long)gridDim.x * kT) {
        float g[8];
        unpack8(__ldg(dY + i), g);
        if (Y) {
            float y[8];
            unpack8(__ldg(Y + i), y);
#pragma unroll
            for (int e = 0; e < 8; ++e) if (!(y[e] > 0.0f)) g[e] = 0.0f;
        }
        if (dPre) dPre[i] = pack8(g);
        if (dZ) {
            if (scale) {
                const int c0 = (int)(i % C8) * 8;
                const float4 s0 = __ldg(reinterpret_cast<const float4 *>(scale + c0));
                const float4 s1 = __ldg(reinterpret_cast<const float4 *>(scale + c0 + 4));
                g[0] *= s0.x; g[1] *= s0.y; g[2] *= s0.z; g[3] *= s0.w;
                g[4] *= s1.x; g[5] *= s1.y; g[6] *= s1.z; g[7] *= s1.w;
            }
            dZ[i] = pack8(g);
        }
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
    const bool small = items * 8 < 0x7fffffffLL && d->B * d->H * d->W * d->Cin < 0x7fffffffLL;
    const long long win_w = (long long)(kPatchPix - 1) * d->stride_w + d->kw;
    const long long wseg = (Wo + kPatchPix - 1) / kPatchPix;
    if (d->kh * win_w * d->Cin <= kPatchMaxElems && ldk <= kPatchMaxCols && d->B * Ho * wseg < 0x7fffffffLL) {
        const size_t smem = ((size_t)(d->kh * win_w * d->Cin + 1) * 2 + 15) / 16 * 16 + (size_t)ldk * sizeof(int);
        im2col_patch_kernel<<<(int)(d->B * Ho * wseg), kT, smem, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(X), *d, (int)Ho, (int)Wo, (int)wseg, static_cast<__nv_bfloat16 *>(Xcol),
            (int)ldk, (int)win_w);
    } else if (small)
        im2col_kernel<int><<<blocks_for(items, dev.sm_count), kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(X), *d, (int)Ho, (int)Wo, static_cast<__nv_bfloat16 *>(Xcol), (int)ldk);
    else
        im2col_kernel<long long><<<blocks_for(items, dev.sm_count), kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(X), *d, Ho, Wo, static_cast<__nv_bfloat16 *>(Xcol), (long long)ldk);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_fold_dims(const twn_conv_desc_t *d, int64_t *Hf, int64_t *Wf, int64_t *ldf)
{
    TWN_REQUIRE(d != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->B > 0 && d->H > 0 && d->W > 0 && d->Cin > 0 && d->Cout > 0 && d->kh > 0 && d->kw > 0 &&
                    d->pad_h >= 0 && d->pad_w >= 0, TWN_ERR_INVALID_ARG);
    // foldable: stride 2 both ways, at most 8 x 8 taps, the 2 x 2 block fits 16 channels
    TWN_REQUIRE(d->stride_h == 2 && d->stride_w == 2 && d->kh <= 8 && d->kw <= 8 && 4 * d->Cin <= 16,
                TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->H + 2 * d->pad_h >= d->kh && d->W + 2 * d->pad_w >= d->kw, TWN_ERR_INVALID_ARG);
    const int64_t Ho = (d->H + 2 * d->pad_h - d->kh) / 2 + 1, Wo = (d->W + 2 * d->pad_w - d->kw) / 2 + 1;
    const int64_t rf = (d->kh + 1) / 2;
    if (Hf) *Hf = Ho + rf - 1;
    if (Wf) *Wf = Wo + 3;         // the 64-element window of the last output pixel ends inside the row
    if (ldf) *ldf = rf * 64;
    return TWN_OK;
}

extern "C" int twn_fold_input(const twn_conv_desc_t *d, const void *X, void *Xf, twn_stream_t stream)
{
    int64_t Hf, Wf;
    int rc = twn_fold_dims(d, &Hf, &Wf, nullptr);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(X && Xf, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(X, 2) && twn_aligned(Xf, 16), TWN_ERR_MISALIGNED);
    TWN_REQUIRE(d->B * Hf * Wf * 16 < 0x7fffffffLL && d->B * d->H * d->W * d->Cin < 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const int grid = blocks_for(d->B * Hf * Wf, dev.sm_count * 4);
    if (d->Cin == 3)
        fold_input_kernel<3><<<grid, kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(X), (int)d->B, (int)d->H, (int)d->W, 3, d->pad_h, d->pad_w, (int)Hf,
            (int)Wf, static_cast<__nv_bfloat16 *>(Xf));
    else
        fold_input_kernel<0><<<grid, kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(X), (int)d->B, (int)d->H, (int)d->W, (int)d->Cin, d->pad_h, d->pad_w,
            (int)Hf, (int)Wf, static_cast<__nv_bfloat16 *>(Xf));
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
    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(X);
    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(Y);
    const bool small = B * H * W * C < 0x7fffffffLL;
    const bool vec = C % 8 == 0 && twn_aligned(X, 16) && twn_aligned(Y, 16) && twn_aligned(argmax, 8);
    cudaStream_t s = twn_cu(stream);
    if (vec && small) {
        maxpool_fwd_vec_kernel<<<blocks_for(B * Ho * Wo * (C / 8), dev.sm_count * 4), kT, 0, s>>>(x, (int)B, (int)H, (int)W, (int)C, k, stride, pad, (int)Ho, (int)Wo,
                                                    y, argmax);
    }
    else if (vec)
        maxpool_fwd_kernel<long long, 8><<<blocks_for(B * Ho * Wo * C / 8, dev.sm_count), kT, 0, s>>>(
            x, B, H, W, C, k, stride, pad, Ho, Wo, y, argmax);
    else
        maxpool_fwd_kernel<long long, 1><<<blocks_for(B * Ho * Wo * C, dev.sm_count), kT, 0, s>>>(
            x, B, H, W, C, k, stride, pad, Ho, Wo, y, argmax);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

namespace {

int maxpool_bwd_launch(const void *dY, const uint8_t *argmax, const void *pooled_v, const float *scale, int64_t B,
                       int64_t H, int64_t W, int64_t C, int k, int stride, int pad, void *dX, twn_stream_t stream)
{
    TWN_REQUIRE(dY && argmax && dX && B > 0 && H > 0 && W > 0 && C > 0 && k > 0 && k <= 15 && stride > 0 &&
                    pad >= 0 && pad < k, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long Ho = pool_extent(H, k, stride, pad), Wo = pool_extent(W, k, stride, pad);
    TWN_REQUIRE(Ho > 0 && Wo > 0, TWN_ERR_INVALID_ARG);
    const __nv_bfloat16 *dy = static_cast<const __nv_bfloat16 *>(dY);
    const __nv_bfloat16 *pooled = static_cast<const __nv_bfloat16 *>(pooled_v);
    __nv_bfloat16 *dx = static_cast<__nv_bfloat16 *>(dX);
    const bool small = B * H * W * C < 0x7fffffffLL;
    const bool vec = C % 8 == 0 && twn_aligned(dY, 16) && twn_aligned(dX, 16) && twn_aligned(argmax, 8) &&
                     twn_aligned(pooled_v, 16) && twn_aligned(scale, 16);
    cudaStream_t s = twn_cu(stream);
    if (vec && small && k == 3 && stride == 2 && pad == 1) {
        const long long items = B * ((H + 1) / 2) * ((W + 1) / 2) * (C / 8);
        maxpool_bwd_k3s2_kernel<<<blocks_for(items, dev.sm_count * 4), kT, 0, s>>>(
            dy, argmax, (int)B, (int)H, (int)W, (int)C, (int)Ho, (int)Wo, dx, pooled, scale);
    }
    else if (vec && small) {
        const long long rows = B * H;
        const int grid = (int)(rows < dev.sm_count * 16LL ? rows : dev.sm_count * 16LL);
        int lg = -1;
        for (int i = 0; i < 8; ++i) if ((1 << i) == stride) lg = i;
        maxpool_bwd_rows_kernel<<<grid, kT, 0, s>>>(dy, argmax, (int)B, (int)H, (int)W, (int)C, k, stride, lg, pad,
                                                    (int)Ho, (int)Wo, dx, pooled, scale);
    }
    else if (vec)
        maxpool_bwd_kernel<long long, 8><<<blocks_for(B * H * W * C / 8, dev.sm_count), kT, 0, s>>>(
            dy, argmax, B, H, W, C, k, stride, pad, Ho, Wo, dx, pooled, scale);
    else
        maxpool_bwd_kernel<long long, 1><<<blocks_for(B * H * W * C, dev.sm_count), kT, 0, s>>>(
            dy, argmax, B, H, W, C, k, stride, pad, Ho, Wo, dx, pooled, scale);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

}  // namespace

extern "C" int twn_maxpool2d_bwd(const void *dY, const uint8_t *argmax, int64_t B, int64_t H, int64_t W, int64_t C,
                                 int k, int stride, int pad, void *dX, twn_stream_t stream)
{
    return maxpool_bwd_launch(dY, argmax, nullptr, nullptr, B, H, W, C, k, stride, pad, dX, stream);
}

extern "C" int twn_maxpool2d_bwd_act(const void *dY, const uint8_t *argmax, const void *pooled, const float *scale,
                                     int64_t B, int64_t H, int64_t W, int64_t C, int k, int stride, int pad,
                                     void *dZ, twn_stream_t stream)
{
    TWN_REQUIRE(pooled != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(pooled, 2) && twn_aligned(scale, 4), TWN_ERR_MISALIGNED);
    return maxpool_bwd_launch(dY, argmax, pooled, scale, B, H, W, C, k, stride, pad, dZ, stream);
}

extern "C" int twn_avgpool_fwd(const void *X, int64_t B, int64_t HW, int64_t C, void *Y, twn_stream_t stream)
{
    TWN_REQUIRE(X && Y && B > 0 && HW > 0 && C > 0, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long groups = (C / 8 + 31) / 32;
    if (C % 8 == 0 && twn_aligned(X, 16) && B * HW * C < 0x7fffffffLL && B * groups < 0x7fffffffLL)
        avgpool_fwd_vec_kernel<<<(int)(B * groups), kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(X), (int)HW, (int)C, (int)groups, static_cast<__nv_bfloat16 *>(Y));
    else
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
    if (C % 8 == 0 && twn_aligned(dY, 16) && twn_aligned(dX, 16) && B * HW * C < 0x7fffffffLL)
        avgpool_bwd_vec_kernel<<<blocks_for(B * HW * C / 8, dev.sm_count), kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(dY), (int)(B * HW * C / 8), (int)HW, (int)C,
            static_cast<__nv_bfloat16 *>(dX));
    else
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
    const bool vec = C % 8 == 0 && n % 8 == 0 && twn_aligned(dY, 16) && twn_aligned(Y, 16) && twn_aligned(dZ, 16) &&
                     twn_aligned(dPre, 16) && twn_aligned(scale, 16);
    if (vec)
        act_bwd_vec_kernel<<<blocks_for(n / 8, dev.sm_count), kT, 0, twn_cu(stream)>>>(
            static_cast<const uint4 *>(dY), static_cast<const uint4 *>(Y), scale, n / 8, (int)(C / 8),
            static_cast<uint4 *>(dZ), static_cast<uint4 *>(dPre));
    else
        act_bwd_kernel<<<blocks_for(n, dev.sm_count), kT, 0, twn_cu(stream)>>>(
            static_cast<const __nv_bfloat16 *>(dY), static_cast<const __nv_bfloat16 *>(Y), scale, n, C,
            static_cast<__nv_bfloat16 *>(dZ), static_cast<__nv_bfloat16 *>(dPre));
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

namespace {

// Batch normalisation in training mode, from the sums the convolution's epilogue produced:
// mean = sum/n, var = sumsq/n - mean^2 (biased), scale = gamma / sqrt(var + eps), shift = beta - mean * scale.
__global__ void __launch_bounds__(kT)
bn_finalize_kernel(const double *__restrict__ sum, const double *__restrict__ sumsq, long long n, int C,
                   const float *__restrict__ gamma, const float *__restrict__ beta, double eps,
                   float *__restrict__ scale, float *__restrict__ shift, double *__restrict__ mean,
                   double *__restrict__ var)
{
    const int c = blockIdx.x * kT + threadIdx.x;
    if (c >= C) return;
    const double m = sum[c] / (double)n;
    double v = sumsq[c] / (double)n - m * m;
    if (v < 0.0) v = 0.0;
    const double sc = (gamma ? (double)gamma[c] : 1.0) / sqrt(v + eps);
    if (scale) scale[c] = (float)sc;
    if (shift) shift[c] = (float)((beta ? (double)beta[c] : 0.0) - m * sc);
    if (mean) mean[c] = m;
    if (var) var[c] = v;
}

}  // namespace

extern "C" int twn_bn_finalize(const double *sum, const double *sumsq, int64_t n, int64_t C, const float *gamma,
                               const float *beta, double eps, float *scale, float *shift, double *mean, double *var,
                               twn_stream_t stream)
{
    TWN_REQUIRE(sum && sumsq && n > 0 && C > 0 && C <= 0x7fffffffLL && eps >= 0.0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(sum, 8) && twn_aligned(sumsq, 8) && twn_aligned(mean, 8) && twn_aligned(var, 8) &&
                    twn_aligned(gamma, 4) && twn_aligned(beta, 4) && twn_aligned(scale, 4) && twn_aligned(shift, 4),
                TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    bn_finalize_kernel<<<(int)((C + kT - 1) / kT), kT, 0, twn_cu(stream)>>>(sum, sumsq, n, (int)C, gamma, beta, eps, scale,
                                                                          shift, mean, var);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}
