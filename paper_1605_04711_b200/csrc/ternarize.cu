// Threshold ternarization fused with 2-bit packing (Sec. 2.3: Eq. 3, Eq. 5 and the
// threshold rule; Algorithm 1, first loop), plus the standalone pack / unpack /
// re-layout kernels.
//
// Two sweeps over the fp32 master weights, both bound by HBM bandwidth:
//   sweep 1  S = sum |W_i| in fp64  ->  delta = factor * S / n
//   sweep 2  codes by Eq. 3, packed 16 per word; sum and count of the kept set
//            ->  alpha (Eq. 5)
// Sweep 2 walks the tensor back to front so that what sweep 1 read last is still
// in L2.  Both reductions have a fixed order: per-thread strided partial sums,
// a shuffle tree per warp, a shared-memory tree per block, one partial per block
// in the workspace, and the block that finishes last folds the partials in index
// order.  No floating-point atomics, no waiting on other blocks.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxBlocks = 2048;
// workspace: [0,256) tickets, then four arrays of kMaxBlocks 8-byte partials
constexpr size_t kWorkspaceBytes = 256 + 4 * size_t(kMaxBlocks) * 8;

struct Workspace {
    unsigned int *ticket1;
    unsigned int *ticket2;
    double *part_sum;
    double *part_kept;
    unsigned long long *part_pos;
    unsigned long long *part_neg;
};

__host__ __device__ inline Workspace carve(void *ws)
{
    char *b = static_cast<char *>(ws);
    Workspace w;
    w.ticket1 = reinterpret_cast<unsigned int *>(b);
    w.ticket2 = reinterpret_cast<unsigned int *>(b + 64);
    w.part_sum = reinterpret_cast<double *>(b + 256);
    w.part_kept = w.part_sum + kMaxBlocks;
    w.part_pos = reinterpret_cast<unsigned long long *>(w.part_kept + kMaxBlocks);
    w.part_neg = w.part_pos + kMaxBlocks;
    return w;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide sum with a fixed order; the result is valid in thread 0.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T *smem /* kWarps entries */)
{
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    T r = T(0);
    if (warp == 0) {
        r = lane < kWarps ? smem[lane] : T(0);
        r = warp_sum(r);
    }
    return r;
}

// Returns true in every thread of the block that took the last of `grid` tickets.
__device__ __forceinline__ bool last_block(unsigned int *ticket, unsigned int grid)
{
    __shared__ bool is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == grid - 1);
    __syncthreads();
    return is_last;
}

// ---- sweep 1 -------------------------------------------------------------
// `vb` of `vg`: this block's index and the number of blocks that work on this tensor (the whole
// grid for a single tensor, a slice of it when several tensors share one launch).
__device__ __forceinline__ void sum_abs_body(const float *__restrict__ W, long long n, double factor, const Workspace ws,
                                             twn_stats_t *__restrict__ stats, unsigned int vb, unsigned int vg)
{
    __shared__ double red[kWarps];
    const long long n4 = n >> 2;
    const float4 *W4 = reinterpret_cast<const float4 *>(W);
    const long long stride = (long long)vg * kThreads;
    long long i = (long long)vb * kThreads + threadIdx.x;

    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    for (; i + 3 * stride < n4; i += 4 * stride) {
        const float4 v0 = __ldg(W4 + i);
        const float4 v1 = __ldg(W4 + i + stride);
        const float4 v2 = __ldg(W4 + i + 2 * stride);
        const float4 v3 = __ldg(W4 + i + 3 * stride);
        a0 += (double)fabsf(v0.x); a1 += (double)fabsf(v0.y); a2 += (double)fabsf(v0.z); a3 += (double)fabsf(v0.w);
        a0 += (double)fabsf(v1.x); a1 += (double)fabsf(v1.y); a2 += (double)fabsf(v1.z); a3 += (double)fabsf(v1.w);
        a0 += (double)fabsf(v2.x); a1 += (double)fabsf(v2.y); a2 += (double)fabsf(v2.z); a3 += (double)fabsf(v2.w);
        a0 += (double)fabsf(v3.x); a1 += (double)fabsf(v3.y); a2 += (double)fabsf(v3.z); a3 += (double)fabsf(v3.w);
    }
    for (; i < n4; i += stride) {
        const float4 v = __ldg(W4 + i);
        a0 += (double)fabsf(v.x); a1 += (double)fabsf(v.y); a2 += (double)fabsf(v.z); a3 += (double)fabsf(v.w);
    }
    // scalar tail (n % 4 elements), by the first threads of block 0
    if (vb == 0) {
        const long long t = (n4 << 2) + threadIdx.x;
        if (t < n) a0 += (double)fabsf(__ldg(W + t));
    }
    const double bsum = block_sum((a0 + a1) + (a2 + a3), red);
    if (threadIdx.x == 0) ws.part_sum[vb] = bsum;

    if (last_block(ws.ticket1, vg)) {
        double s = 0.0;
        for (int b = threadIdx.x; b < (int)vg; b += kThreads) s += __ldcg(ws.part_sum + b);
        s = block_sum(s, red);
        if (threadIdx.x == 0) {
            const double delta = n > 0 ? factor * (s / (double)n) : 0.0;
            stats->sum_abs = s;
            stats->delta = delta;
            stats->status = isfinite(s) ? TWN_OK : TWN_ERR_NONFINITE;
            stats->reserved = 0;
            *ws.ticket1 = 0u;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
sum_abs_kernel(const float *__restrict__ W, long long n, double factor, void *ws_raw,
               twn_stats_t *__restrict__ stats)
{
    sum_abs_body(W, n, factor, carve(ws_raw), stats, blockIdx.x, gridDim.x);
}

// ---- parameter update fused with sweep 1 of the next iteration -------------
// Last step of Algorithm 1 (UpdateParameters: SGD with momentum and L2 weight decay on the fp32
// master weights, Sec. 3):
//     g = dW + wd * W;   V' = mu * V + g;   W' = W - lr * V'
// every operation a separately rounded fp32 operation in this order (no fused multiply-add), so
// the result is defined to the bit.  The next iteration starts by ternarizing W', whose
// threshold needs sum |W'|: it is accumulated here while W' is still in registers, which saves
// the first sweep of that ternarization (one read of the weights).
__device__ __forceinline__ float sgd_one(float w, float g, float &v, float lr, float mu, float wd)
{
    const float grad = __fadd_rn(g, __fmul_rn(wd, w));
    v = __fadd_rn(__fmul_rn(mu, v), grad);
    return __fsub_rn(w, __fmul_rn(lr, v));
}

// `vb` of `vg`: this block's index among the blocks that work on this tensor.
__device__ __forceinline__ void sgd_update_body(float *__restrict__ W, const float *__restrict__ dW, float *__restrict__ V,
                                                long long n, float lr, float mu, float wd, double factor,
                                                const Workspace ws, twn_stats_t *__restrict__ stats, unsigned int vb,
                                                unsigned int vg)
{
    __shared__ double red[kWarps];
    const long long n4 = n >> 2;
    float4 *W4 = reinterpret_cast<float4 *>(W);
    float4 *V4 = reinterpret_cast<float4 *>(V);
    const float4 *G4 = reinterpret_cast<const float4 *>(dW);
    const long long stride = (long long)vg * kThreads;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll 2
    for (long long i = (long long)vb * kThreads + threadIdx.x; i < n4; i += stride) {
        float4 w = W4[i], v = V4[i];
        const float4 g = __ldg(G4 + i);
        w.x = sgd_one(w.x, g.x, v.x, lr, mu, wd);
        w.y = sgd_one(w.y, g.y, v.y, lr, mu, wd);
        w.z = sgd_one(w.z, g.z, v.z, lr, mu, wd);
        w.w = sgd_one(w.w, g.w, v.w, lr, mu, wd);
        W4[i] = w;
        V4[i] = v;
        a0 += (double)fabsf(w.x); a1 += (double)fabsf(w.y); a2 += (double)fabsf(w.z); a3 += (double)fabsf(w.w);
    }
    if (vb == 0) {
        const long long t = (n4 << 2) + threadIdx.x;
        if (t < n) {
            float v = V[t];
            const float w = sgd_one(W[t], __ldg(dW + t), v, lr, mu, wd);
            W[t] = w;
            V[t] = v;
            a0 += (double)fabsf(w);
        }
    }
    const double bsum = block_sum((a0 + a1) + (a2 + a3), red);
    if (threadIdx.x == 0) ws.part_sum[vb] = bsum;
    if (last_block(ws.ticket1, vg)) {
        double s = 0.0;
        for (int b = threadIdx.x; b < (int)vg; b += kThreads) s += __ldcg(ws.part_sum + b);
        s = block_sum(s, red);
        if (threadIdx.x == 0) {
            if (stats) {
                stats->sum_abs = s;
                stats->delta = n > 0 ? factor * (s / (double)n) : 0.0;
                stats->status = isfinite(s) ? TWN_OK : TWN_ERR_NONFINITE;
                stats->reserved = 0;
            }
            *ws.ticket1 = 0u;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
sgd_update_kernel(float *__restrict__ W, const float *__restrict__ dW, float *__restrict__ V, long long n,
                  float lr, float mu, float wd, double factor, void *ws_raw, twn_stats_t *__restrict__ stats)
{
    sgd_update_body(W, dW, V, n, lr, mu, wd, factor, carve(ws_raw), stats, blockIdx.x, gridDim.x);
}

// ---- sweep 2 -------------------------------------------------------------
// 2-bit field of one weight: bit 0 = kept, bit 1 = negative  (00 / 01 / 11).
__device__ __forceinline__ uint32_t code2(float w, float thr, double &kept_sum)
{
    const float a = fabsf(w);
    const bool keep = a > thr;
    if (keep) kept_sum += (double)a;
    return keep ? (w < 0.0f ? 3u : 1u) : 0u;
}

// Bit position of element e (0..15) inside its word: even elements fill the low
// half-word, odd elements the high half-word, each from the top down, so that a left
// shift by 2*(e/2) brings the element's field to the top two bits of its half-word.
__host__ __device__ __forceinline__ int field_pos(int e) { return 14 - 2 * (e >> 1) + 16 * (e & 1); }

// Four consecutive weights -> one byte: low nibble = fields of elements 0 (upper) and 2,
// high nibble = fields of elements 1 (upper) and 3.
__device__ __forceinline__ uint32_t code8(const float4 v, float thr, double &k0, double &k1)
{
    uint32_t c = code2(v.x, thr, k0) << 2;
    c |= code2(v.z, thr, k0);
    c |= code2(v.y, thr, k1) << 6;
    c |= code2(v.w, thr, k1) << 4;
    return c;
}

// Bytes B0..B3 (as produced by code8 for four consecutive float4) -> the word of
// those 16 elements: low half = low nibbles, high half = high nibbles, B0's on top.
__device__ __forceinline__ uint32_t bytes_to_word(uint32_t r)
{
    r = __byte_perm(r, 0u, 0x0123);
    uint32_t lo = r & 0x0F0F0F0Fu, hi = (r >> 4) & 0x0F0F0F0Fu;
    lo = (lo | (lo >> 4)) & 0x00FF00FFu;
    lo = (lo | (lo >> 8)) & 0x0000FFFFu;
    hi = (hi | (hi >> 4)) & 0x00FF00FFu;
    hi = (hi | (hi >> 8)) & 0x0000FFFFu;
    return lo | (hi << 16);
}

// inverse: word -> bytes B0..B3
__device__ __forceinline__ uint32_t word_to_bytes(uint32_t w)
{
    uint32_t lo = w & 0xFFFFu, hi = w >> 16;
    lo = (lo | (lo << 8)) & 0x00FF00FFu;
    lo = (lo | (lo << 4)) & 0x0F0F0F0Fu;
    hi = (hi | (hi << 8)) & 0x00FF00FFu;
    hi = (hi | (hi << 4)) & 0x0F0F0F0Fu;
    return __byte_perm(lo | (hi << 4), 0u, 0x0123);
}

// int8 image of the four fields of a code8 byte, in element order:
// 00 -> 0x00, 01 -> 0x01, 11 -> 0xFF
__device__ __forceinline__ uint32_t fields_to_i8x4(uint32_t c8)
{
    uint32_t r = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const uint32_t f = (c8 >> (2 - 2 * (e >> 1) + 4 * (e & 1))) & 3u;
        const uint32_t b = (f & 1u) ? ((f & 2u) ? 0xFFu : 0x01u) : 0u;
        r |= b << (8 * e);
    }
    return r;
}

// Fast path geometry: a "unit" is 512 consecutive weights = 128 float4 = 32 words,
// handled by one warp: lane l loads float4 (unit*128 + j*32 + l) for j = 0..3, so
// every load instruction covers 512 contiguous bytes.  A 4x4 byte transpose inside
// each group of four lanes then leaves lane l with the four bytes of word
// unit*32 + (l%4)*8 + l/4, and the warp stores one contiguous 128-byte line.
__device__ __forceinline__ void code_pack_body(const float *__restrict__ W, long long rows, long long cols,
                                               long long ld_codes, long long fast_units, uint32_t *__restrict__ packed,
                                               int8_t *__restrict__ codes_i8, const Workspace ws,
                                               twn_stats_t *__restrict__ stats, unsigned int vb, unsigned int vg)
{
    __shared__ double red[kWarps];
    __shared__ unsigned long long redu[kWarps];
    const long long n = rows * cols;
    // delta rounded toward -inf: for any float w,  w > delta  <=>  w > thr
    const float thr = __double2float_rd(stats->delta);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double k0 = 0.0, k1 = 0.0;
    unsigned long long npos = 0, nneg = 0;

    // -- fast units, back to front
    const long long gwarps = (long long)vg * kWarps;
    const float4 *W4 = reinterpret_cast<const float4 *>(W);
    for (long long u = fast_units - 1 - ((long long)vb * kWarps + warp); u >= 0; u -= gwarps) {
        const long long f0 = u * 128 + lane;
        const float4 v0 = __ldg(W4 + f0);
        const float4 v1 = __ldg(W4 + f0 + 32);
        const float4 v2 = __ldg(W4 + f0 + 64);
        const float4 v3 = __ldg(W4 + f0 + 96);
        const uint32_t c0 = code8(v0, thr, k0, k1);
        const uint32_t c1 = code8(v1, thr, k0, k1);
        const uint32_t c2 = code8(v2, thr, k0, k1);
        const uint32_t c3 = code8(v3, thr, k0, k1);
        uint32_t r = c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
        const uint32_t neg = __popc((r >> 1) & 0x55555555u);
        nneg += neg;
        npos += __popc(r & 0x55555555u) - neg;
        if (codes_i8) {
            uint32_t *o = reinterpret_cast<uint32_t *>(codes_i8) + f0;
            o[0] = fields_to_i8x4(c0);
            o[32] = fields_to_i8x4(c1);
            o[64] = fields_to_i8x4(c2);
            o[96] = fields_to_i8x4(c3);
        }
        // 4x4 byte transpose across lanes l^2 then l^1
        const uint32_t y = __shfl_xor_sync(0xffffffffu, r, 2);
        r = __byte_perm(r, y, (lane & 2) ? 0x3276 : 0x5410);
        const uint32_t z = __shfl_xor_sync(0xffffffffu, r, 1);
        r = __byte_perm(r, z, (lane & 1) ? 0x3715 : 0x6240);
        packed[u * 32 + (lane & 3) * 8 + (lane >> 2)] = bytes_to_word(r);
    }

    // -- everything else, one thread per word: the tail of a flat tensor, ragged rows, padding
    const long long wpr = ld_codes >> 4;
    const long long total_words = rows * wpr;
    const long long first_word = fast_units * 32;
    for (long long w = first_word + (long long)vb * kThreads + threadIdx.x; w < total_words;
         w += (long long)vg * kThreads) {
        const long long r = w / wpr;
        const long long j0 = (w - r * wpr) << 4;
        uint32_t word = 0;
#pragma unroll 4
        for (int e = 0; e < 16; ++e) {
            const long long j = j0 + e;
            if (j < cols) {
                const float v = __ldg(W + r * cols + j);
                const uint32_t c = code2(v, thr, k0);
                word |= c << field_pos(e);
                if (codes_i8) codes_i8[r * cols + j] = (int8_t)((c & 1u) ? ((c & 2u) ? -1 : 1) : 0);
            }
        }
        const uint32_t neg = __popc((word >> 1) & 0x55555555u);
        nneg += neg;
        npos += __popc(word & 0x55555555u) - neg;
        packed[w] = word;
    }

    const double bk = block_sum(k0 + k1, red);
    const unsigned long long bp = block_sum(npos, redu);
    const unsigned long long bn = block_sum(nneg, redu);
    if (threadIdx.x == 0) {
        ws.part_kept[vb] = bk;
        ws.part_pos[vb] = bp;
        ws.part_neg[vb] = bn;
    }
    if (last_block(ws.ticket2, vg)) {
        double s = 0.0;
        unsigned long long p = 0, q = 0;
        for (int b = threadIdx.x; b < (int)vg; b += kThreads) {
            s += __ldcg(ws.part_kept + b);
            p += __ldcg(ws.part_pos + b);
            q += __ldcg(ws.part_neg + b);
        }
        s = block_sum(s, red);
        p = block_sum(p, redu);
        q = block_sum(q, redu);
        if (threadIdx.x == 0) {
            const unsigned long long kept = p + q;
            stats->sum_abs_kept = s;
            stats->alpha = kept > 0 ? s / (double)kept : 0.0;
            stats->n_pos = p;
            stats->n_neg = q;
            stats->n_zero = (unsigned long long)n - kept;
            *ws.ticket2 = 0u;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
code_pack_kernel(const float *__restrict__ W, long long rows, long long cols, long long ld_codes,
                 long long fast_units, uint32_t *__restrict__ packed, int8_t *__restrict__ codes_i8,
                 void *ws_raw, twn_stats_t *__restrict__ stats)
{
    code_pack_body(W, rows, cols, ld_codes, fast_units, packed, codes_i8, carve(ws_raw), stats, blockIdx.x, gridDim.x);
}

// ---- several tensors in one launch ------------------------------------------
// A training step ternarizes every layer (Algorithm 1, first loop).  One launch per sweep for
// all of them: the blocks of the grid are dealt out to the tensors in proportion to their size,
// and each tensor keeps its own tickets and partials, so its results are bit-identical to those
// of a call of its own.
constexpr int kMaxBatch = 32;
struct BatchItem {
    const float *W;
    long long rows, cols, ld_codes, fast_units;
    uint32_t *packed;
    int8_t *codes_i8;
    twn_stats_t *stats;
};
struct BatchParams {
    int count;
    unsigned int first_block[kMaxBatch + 1];   // blocks [first_block[t], first_block[t+1]) work on tensor t
    BatchItem item[kMaxBatch];
};

// Slice t of a batch workspace: the tickets of all tensors come first (256 bytes each, so that one
// small memset clears them), then the partials.
__host__ __device__ inline Workspace carve_batch(void *ws, int t, int count)
{
    char *b = static_cast<char *>(ws);
    Workspace w;
    w.ticket1 = reinterpret_cast<unsigned int *>(b + (size_t)t * 256);
    w.ticket2 = reinterpret_cast<unsigned int *>(b + (size_t)t * 256 + 64);
    char *p = b + (size_t)count * 256 + (size_t)t * (4 * size_t(kMaxBlocks) * 8);
    w.part_sum = reinterpret_cast<double *>(p);
    w.part_kept = w.part_sum + kMaxBlocks;
    w.part_pos = reinterpret_cast<unsigned long long *>(w.part_kept + kMaxBlocks);
    w.part_neg = w.part_pos + kMaxBlocks;
    return w;
}

__device__ __forceinline__ int batch_tensor_of(const BatchParams &P, unsigned int block)
{
    int t = 0;
    while (t + 1 < P.count && block >= P.first_block[t + 1]) ++t;
    return t;
}

__global__ void __launch_bounds__(kThreads)
sum_abs_batch_kernel(const __grid_constant__ BatchParams P, double factor, void *ws_raw)
{
    const int t = batch_tensor_of(P, blockIdx.x);
    const BatchItem &it = P.item[t];
    sum_abs_body(it.W, it.rows * it.cols, factor, carve_batch(ws_raw, t, P.count), it.stats,
                 blockIdx.x - P.first_block[t], P.first_block[t + 1] - P.first_block[t]);
}

__global__ void __launch_bounds__(kThreads)
code_pack_batch_kernel(const __grid_constant__ BatchParams P, void *ws_raw)
{
    const int t = batch_tensor_of(P, blockIdx.x);
    const BatchItem &it = P.item[t];
    code_pack_body(it.W, it.rows, it.cols, it.ld_codes, it.fast_units, it.packed, it.codes_i8,
                   carve_batch(ws_raw, t, P.count), it.stats, blockIdx.x - P.first_block[t],
                   P.first_block[t + 1] - P.first_block[t]);
}

struct SgdItem {
    float *W;
    const float *dW;
    float *V;
    long long n;
    twn_stats_t *stats;
};
struct SgdBatch {
    int count;
    unsigned int first_block[kMaxBatch + 1];
    SgdItem item[kMaxBatch];
};

__global__ void __launch_bounds__(kThreads)
sgd_update_batch_kernel(const __grid_constant__ SgdBatch P, float lr, float mu, float wd, double factor, void *ws_raw)
{
    int t = 0;
    while (t + 1 < P.count && blockIdx.x >= P.first_block[t + 1]) ++t;
    const SgdItem &it = P.item[t];
    sgd_update_body(it.W, it.dW, it.V, it.n, lr, mu, wd, factor, carve_batch(ws_raw, t, P.count), it.stats,
                    blockIdx.x - P.first_block[t], P.first_block[t + 1] - P.first_block[t]);
}

// ---- standalone pack / unpack / re-layout ----------------------------------
__device__ __forceinline__ uint32_t i8x4_to_fields(uint32_t x, uint32_t &bad)
{
    // a byte is valid iff (byte + 1) mod 256 <= 2
    const uint32_t inval = __vcmpgtu4(__vadd4(x, 0x01010101u), 0x02020202u);
    bad |= inval;
    x &= ~inval;
    // low two bits of bytes 0..3 -> fields in code8 order (low nibble e0, e2; high nibble e1, e3)
    const uint32_t y = x & 0x03030303u;
    return ((y & 3u) << 2) | ((y >> 16) & 3u) | ((y >> 2) & 0xC0u) | ((y >> 20) & 0x30u);
}

__global__ void __launch_bounds__(kThreads)
pack_kernel(const int8_t *__restrict__ codes, long long rows, long long cols, long long ld_codes,
            int vec_ok, uint32_t *__restrict__ packed, twn_stats_t *__restrict__ counts)
{
    __shared__ unsigned long long redu[kWarps];
    const long long wpr = ld_codes >> 4;
    const long long total_words = rows * wpr;
    unsigned long long npos = 0, nneg = 0;
    uint32_t bad = 0;
    for (long long w = (long long)blockIdx.x * kThreads + threadIdx.x; w < total_words;
         w += (long long)gridDim.x * kThreads) {
        const long long r = w / wpr;
        const long long j0 = (w - r * wpr) << 4;
        uint32_t word = 0;
        if (vec_ok && j0 + 16 <= cols) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(codes + r * cols + j0));
            word = bytes_to_word(i8x4_to_fields(v.x, bad) | (i8x4_to_fields(v.y, bad) << 8) |
                                 (i8x4_to_fields(v.z, bad) << 16) | (i8x4_to_fields(v.w, bad) << 24));
        } else {
            for (int e = 0; e < 16; ++e) {
                const long long j = j0 + e;
                if (j < cols) {
                    const uint32_t b = (uint8_t)codes[r * cols + j];
                    word |= ((i8x4_to_fields(b, bad) >> 2) & 3u) << field_pos(e);   // byte 0 -> bits 3:2
                }
            }
        }
        const uint32_t neg = __popc((word >> 1) & 0x55555555u);
        nneg += neg;
        npos += __popc(word & 0x55555555u) - neg;
        packed[w] = word;
    }
    if (counts) {
        const unsigned long long bp = block_sum(npos, redu);
        const unsigned long long bn = block_sum(nneg, redu);
        const int any_bad = __syncthreads_or(bad != 0);
        if (threadIdx.x == 0) {
            // integer atomics: order-independent, hence still deterministic
            atomicAdd(reinterpret_cast<unsigned long long *>(&counts->n_pos), bp);
            atomicAdd(reinterpret_cast<unsigned long long *>(&counts->n_neg), bn);
            if (any_bad) atomicMin(&counts->status, (int)TWN_ERR_BAD_CODE);
        }
    }
}

__global__ void finish_counts_kernel(twn_stats_t *counts, unsigned long long n)
{
    counts->n_zero = n - counts->n_pos - counts->n_neg;
}

__global__ void __launch_bounds__(kThreads)
unpack_kernel(const uint32_t *__restrict__ packed, long long rows, long long cols, long long ld_codes,
              int vec_ok, int8_t *__restrict__ codes, int32_t *__restrict__ dev_status)
{
    const long long wpr = ld_codes >> 4;
    const long long wpr_used = (cols + 15) >> 4;
    const long long total = rows * wpr_used;
    bool bad = false;
    for (long long t = (long long)blockIdx.x * kThreads + threadIdx.x; t < total;
         t += (long long)gridDim.x * kThreads) {
        const long long r = t / wpr_used;
        const long long wi = t - r * wpr_used;
        const uint32_t word = __ldg(packed + r * wpr + wi);
        // field 10: bit 1 set while bit 0 is clear
        const uint32_t inval = (word >> 1) & ~word & 0x55555555u;
        const long long j0 = wi << 4;
        const long long valid = cols - j0 >= 16 ? 16 : cols - j0;
        // fields of elements < valid: the top ceil(valid/2) of the low half, the top floor(valid/2) of the high half
        const uint32_t vmask = valid >= 16 ? 0xFFFFFFFFu
                                           : (((0xFFFFu << (16 - 2 * ((valid + 1) >> 1))) & 0xFFFFu) |
                                              (((0xFFFFu << (16 - 2 * (valid >> 1))) & 0xFFFFu) << 16));
        if (inval & vmask) bad = true;
        const uint32_t clean = word & ~(inval << 1);
        if (vec_ok && valid == 16) {
            const uint32_t by = word_to_bytes(clean);
            uint4 o;
            o.x = fields_to_i8x4(by & 0xFFu);
            o.y = fields_to_i8x4((by >> 8) & 0xFFu);
            o.z = fields_to_i8x4((by >> 16) & 0xFFu);
            o.w = fields_to_i8x4(by >> 24);
            *reinterpret_cast<uint4 *>(codes + r * cols + j0) = o;
        } else {
            for (int e = 0; e < valid; ++e) {
                const uint32_t f = (clean >> field_pos(e)) & 3u;
                codes[r * cols + j0 + e] = (int8_t)((f & 1u) ? ((f & 2u) ? -1 : 1) : 0);
            }
        }
    }
    if (dev_status && __syncthreads_or(bad) && threadIdx.x == 0) atomicMin(dev_status, (int)TWN_ERR_BAD_CODE);
}

// out row c, column t*Cout + o  <-  in row o, column t*Cin + c   (t = tap index)
// (32-bit index arithmetic: a filter bank has far fewer than 2^31 codes)
// `vb` of `vg`: this block's index among the blocks that work on this filter bank.
__device__ __forceinline__ void transpose_codes_body(const uint32_t *__restrict__ in, int ld_in, int Cout, int Cin,
                                                     int taps, uint32_t *__restrict__ out, int ld_out,
                                                     unsigned int vb, unsigned int vg)
{
    const int wpr_out = ld_out >> 4, wpr_in = ld_in >> 4;
    const int total = Cin * wpr_out;
    const int cols_out = taps * Cout;
    for (int w = vb * kThreads + threadIdx.x; w < total; w += vg * kThreads) {
        const int c = w / wpr_out;
        const int j0 = (w - c * wpr_out) << 4;
        int t = j0 / Cout, o = j0 - t * Cout;
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if (j0 + e < cols_out) {
                const int src = t * Cin + c;
                const uint32_t f = (__ldg(in + (size_t)o * wpr_in + (src >> 4)) >> field_pos(src & 15)) & 3u;
                word |= f << field_pos(e);
            }
            if (++o == Cout) { o = 0; ++t; }
        }
        out[w] = word;
    }
}

// The same re-layout for filter banks whose taps start on word boundaries on both sides (Cin % 16 == 0, and
// Cout % 16 == 0 or a single tap): a thread takes one tap, 64 output channels and 16 input channels, i.e. 64 input words (word
// column (t*Cin + c0)/16 of rows o0 .. o0+63, read coalesced across the threads of a warp, which take consecutive
// c0) and transposes four 16 x 16 blocks of codes in registers into the 16 runs of four output words
// (rows c0 .. c0+15, word columns (t*Cout + o0)/16 ..).  One load per output word instead of sixteen.
constexpr int kFastRows = 64;
__host__ __device__ __forceinline__ bool transpose_fast_ok(int Cout, int Cin, int taps)
{
    return Cin % 16 == 0 && (Cout % 16 == 0 || taps == 1);
}
__host__ __device__ __forceinline__ int transpose_fast_groups(int Cout) { return (Cout + kFastRows - 1) / kFastRows; }
__device__ __forceinline__ void transpose_codes_fast_body(const uint32_t *__restrict__ in, int ld_in, int Cout, int Cin,
                                                          int taps, uint32_t *__restrict__ out, int ld_out,
                                                          unsigned int vb, unsigned int vg)
{
    const int wpr_out = ld_out >> 4, wpr_in = ld_in >> 4;
    const int cgs = Cin >> 4, ogs = transpose_fast_groups(Cout);
    const int units = taps * ogs * cgs;
    for (int u = vb * kThreads + threadIdx.x; u < units; u += vg * kThreads) {
        const int cg = u % cgs;
        const int og = (u / cgs) % ogs;
        const int t = u / (cgs * ogs);
        const int o0 = og * kFastRows, c0 = cg << 4;
        const uint32_t *src = in + (size_t)o0 * wpr_in + ((t * Cin + c0) >> 4);
        uint32_t *dst = out + (size_t)c0 * wpr_out + ((t * Cout + o0) >> 4);
#pragma unroll 1
        for (int q = 0; q < kFastRows / 16 && o0 + q * 16 < Cout; ++q) {
            // rows past Cout (the last group of a bank whose Cout is no multiple of 16) read as zero codes
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = o0 + q * 16 + i < Cout ? __ldg(src + (size_t)(q * 16 + i) * wpr_in) : 0u;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                uint32_t word = 0;
#pragma unroll
                for (int i = 0; i < 16; ++i) word |= ((w[i] >> field_pos(j)) & 3u) << field_pos(i);
                dst[(size_t)j * wpr_out + q] = word;
            }
        }
    }
    // columns past the last tap (a row pitch larger than taps * Cout) read as zero codes
    const int used = (taps * Cout + 15) >> 4;
    if (used < wpr_out) {
        const int pad = wpr_out - used;
        for (int i = vb * kThreads + threadIdx.x; i < Cin * pad; i += vg * kThreads)
            out[(size_t)(i / pad) * wpr_out + used + i % pad] = 0u;
    }
}

__global__ void __launch_bounds__(kThreads)
transpose_codes_kernel(const uint32_t *__restrict__ in, int ld_in, int Cout, int Cin,
                       int taps, uint32_t *__restrict__ out, int ld_out)
{
    if (transpose_fast_ok(Cout, Cin, taps)) transpose_codes_fast_body(in, ld_in, Cout, Cin, taps, out, ld_out, blockIdx.x, gridDim.x);
    else transpose_codes_body(in, ld_in, Cout, Cin, taps, out, ld_out, blockIdx.x, gridDim.x);
}

// The filter banks of a whole network in one launch (the backward pass of a step needs them all).
struct TransposeItem {
    const uint32_t *in;
    uint32_t *out;
    int ld_in, ld_out, Cout, Cin, taps;
};
struct TransposeBatch {
    int count;
    unsigned int first_block[kMaxBatch + 1];
    TransposeItem item[kMaxBatch];
};

__global__ void __launch_bounds__(kThreads)
transpose_codes_batch_kernel(const __grid_constant__ TransposeBatch P)
{
    int t = 0;
    while (t + 1 < P.count && blockIdx.x >= P.first_block[t + 1]) ++t;
    const TransposeItem &it = P.item[t];
    if (transpose_fast_ok(it.Cout, it.Cin, it.taps))
        transpose_codes_fast_body(it.in, it.ld_in, it.Cout, it.Cin, it.taps, it.out, it.ld_out,
                                  blockIdx.x - P.first_block[t], P.first_block[t + 1] - P.first_block[t]);
    else
        transpose_codes_body(it.in, it.ld_in, it.Cout, it.Cin, it.taps, it.out, it.ld_out,
                             blockIdx.x - P.first_block[t], P.first_block[t + 1] - P.first_block[t]);
}

// Codes of a stride-2 layer re-ordered for the folded input: folded row r' holds 64 columns,
// column s'*16 + (dy*2 + dx)*Cin + c  <-  tap (2r' + dy, 2s' + dx), channel c; columns without a
// tap (past kh or kw, or past 4*Cin inside a 16-group) are 0.
__global__ void __launch_bounds__(kThreads)
fold_codes_kernel(const uint32_t *__restrict__ in, int ld_in, int Cout, int Cin, int kh, int kw,
                  uint32_t *__restrict__ out, int ld_out)
{
    const int wpr_out = ld_out >> 4, wpr_in = ld_in >> 4;
    const int total = Cout * wpr_out;
    for (int w = blockIdx.x * kThreads + threadIdx.x; w < total; w += gridDim.x * kThreads) {
        const int o = w / wpr_out;
        const int j0 = (w - o * wpr_out) << 4;      // a word is one (r', s') group of 16 columns
        const int rf = j0 >> 6, sf = (j0 >> 4) & 3;
        uint32_t word = 0;
        for (int e = 0; e < 4 * Cin; ++e) {
            const int blk = e / Cin, c = e - blk * Cin;
            const int r = 2 * rf + (blk >> 1), sx = 2 * sf + (blk & 1);
            if (r < kh && sx < kw) {
                const int src = (r * kw + sx) * Cin + c;
                const uint32_t f = (__ldg(in + (size_t)o * wpr_in + (src >> 4)) >> field_pos(src & 15)) & 3u;
                word |= f << field_pos(e);
            }
        }
        out[w] = word;
    }
}

int grid_for(long long items_per_thread_units, int sm_count)
{
    long long blocks = (items_per_thread_units + kThreads - 1) / kThreads;
    const long long cap = (long long)sm_count * 8 < kMaxBlocks ? (long long)sm_count * 8 : kMaxBlocks;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace

extern "C" size_t twn_ternarize_workspace_bytes(void) { return kWorkspaceBytes; }

extern "C" int twn_ternarize(const float *W, int64_t rows, int64_t cols, double delta_factor,
                             twn_stats_t *stats, uint32_t *packed, int64_t ld_codes,
                             int8_t *codes_i8, void *workspace, size_t workspace_bytes,
                             twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(stats != nullptr && workspace != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(delta_factor >= 0.0 && delta_factor == delta_factor, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
    const long long n = (long long)rows * cols;
    TWN_REQUIRE(n == 0 || (W != nullptr && packed != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace_bytes >= kWorkspaceBytes, TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(W, 16) && twn_aligned(packed, 16) && twn_aligned(stats, 8) &&
                    twn_aligned(workspace, 256) && twn_aligned(codes_i8, 16), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    cudaStream_t s = twn_cu(stream);

    // the two tickets must start at zero
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, 128, s));

    const int g1 = grid_for((n / 4 + 3) / 4, dev.sm_count);
    sum_abs_kernel<<<g1, kThreads, 0, s>>>(W, n, delta_factor, workspace, stats);

    // a flat run of whole 512-weight units exists when rows are stored back to back
    const bool flat = (rows <= 1) || (ld_codes == cols);
    const long long fast_units = flat ? n / 512 : 0;
    const long long rest_words = (long long)rows * (ld_codes / 16) - fast_units * 32;
    long long work = fast_units * 32 / 4;  // threads: each warp-iteration covers one unit
    if (rest_words > work) work = rest_words;
    const int g2 = grid_for(work, dev.sm_count);
    code_pack_kernel<<<g2, kThreads, 0, s>>>(W, rows, cols, ld_codes, fast_units, packed, codes_i8,
                                             workspace, stats);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_sgd_update(float *W, const float *dW, float *V, int64_t n, float lr, float momentum,
                              float weight_decay, double delta_factor, twn_stats_t *stats_next, void *workspace,
                              size_t workspace_bytes, twn_stream_t stream)
{
    TWN_REQUIRE(n >= 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(n == 0 || (W != nullptr && dW != nullptr && V != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(lr == lr && momentum == momentum && weight_decay == weight_decay, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(delta_factor >= 0.0 && delta_factor == delta_factor, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace_bytes >= kWorkspaceBytes, TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(W, 16) && twn_aligned(dW, 16) && twn_aligned(V, 16) && twn_aligned(stats_next, 8) &&
                    twn_aligned(workspace, 256), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    cudaStream_t s = twn_cu(stream);
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, 128, s));
    const int g = grid_for((n / 4 + 1) / 2, dev.sm_count);
    sgd_update_kernel<<<g, kThreads, 0, s>>>(W, dW, V, n, lr, momentum, weight_decay, delta_factor, workspace, stats_next);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_sgd_update_batch(const twn_sgd_item_t *items, int count, float lr, float momentum,
                                    float weight_decay, double delta_factor, void *workspace, size_t workspace_bytes,
                                    twn_stream_t stream)
{
    TWN_REQUIRE(count >= 0 && count <= kMaxBatch, TWN_ERR_INVALID_ARG);
    if (count == 0) return TWN_OK;
    TWN_REQUIRE(items != nullptr && workspace != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(lr == lr && momentum == momentum && weight_decay == weight_decay, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(delta_factor >= 0.0 && delta_factor == delta_factor, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace_bytes >= twn_ternarize_batch_workspace_bytes(count), TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(workspace, 256), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    SgdBatch P;
    P.count = count;
    unsigned int g = 0;
    for (int t = 0; t < count; ++t) {
        const twn_sgd_item_t &it = items[t];
        TWN_REQUIRE(it.n >= 0 && (it.n == 0 || (it.W && it.dW && it.V)), TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(twn_aligned(it.W, 16) && twn_aligned(it.dW, 16) && twn_aligned(it.V, 16) &&
                        twn_aligned(it.stats_next, 8), TWN_ERR_MISALIGNED);
        SgdItem si;
        si.W = it.W; si.dW = it.dW; si.V = it.V; si.n = it.n; si.stats = it.stats_next;
        P.item[t] = si;
        P.first_block[t] = g;
        g += (unsigned int)grid_for((it.n / 4 + 1) / 2, dev.sm_count);     // the grid of a call of its own
    }
    P.first_block[count] = g;
    cudaStream_t s = twn_cu(stream);
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, (size_t)count * 256, s));
    sgd_update_batch_kernel<<<g, kThreads, 0, s>>>(P, lr, momentum, weight_decay, delta_factor, workspace);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_ternarize_codes_batch(const twn_ternarize_item_t *items, int count, void *workspace,
                                         size_t workspace_bytes, twn_stream_t stream)
{
    TWN_REQUIRE(count >= 0 && count <= kMaxBatch, TWN_ERR_INVALID_ARG);
    if (count == 0) return TWN_OK;
    TWN_REQUIRE(items != nullptr && workspace != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace_bytes >= twn_ternarize_batch_workspace_bytes(count), TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(workspace, 256), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    BatchParams B;
    B.count = count;
    unsigned int gb = 0;
    for (int t = 0; t < count; ++t) {
        const twn_ternarize_item_t &it = items[t];
        TWN_REQUIRE(it.rows >= 0 && it.cols >= 0 && it.stats != nullptr, TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(it.ld_codes >= it.cols && it.ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
        const long long n = (long long)it.rows * it.cols;
        TWN_REQUIRE(n == 0 || (it.W != nullptr && it.packed != nullptr), TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(twn_aligned(it.W, 16) && twn_aligned(it.packed, 16) && twn_aligned(it.stats, 8) &&
                        twn_aligned(it.codes_i8, 16), TWN_ERR_MISALIGNED);
        const bool flat = (it.rows <= 1) || (it.ld_codes == it.cols);
        const long long fast_units = flat ? n / 512 : 0;
        const long long rest_words = (long long)it.rows * (it.ld_codes / 16) - fast_units * 32;
        long long work = fast_units * 32 / 4;
        if (rest_words > work) work = rest_words;
        BatchItem bi;
        bi.W = it.W; bi.rows = it.rows; bi.cols = it.cols; bi.ld_codes = it.ld_codes; bi.fast_units = fast_units;
        bi.packed = it.packed; bi.codes_i8 = it.codes_i8; bi.stats = it.stats;
        B.item[t] = bi;
        B.first_block[t] = gb;
        gb += (unsigned int)grid_for(work, dev.sm_count);
    }
    B.first_block[count] = gb;
    cudaStream_t s = twn_cu(stream);
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, (size_t)count * 256, s));
    code_pack_batch_kernel<<<gb, kThreads, 0, s>>>(B, workspace);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_ternarize_codes(const float *W, int64_t rows, int64_t cols, twn_stats_t *stats, uint32_t *packed,
                                   int64_t ld_codes, int8_t *codes_i8, void *workspace, size_t workspace_bytes,
                                   twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(stats != nullptr && workspace != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
    const long long n = (long long)rows * cols;
    TWN_REQUIRE(n == 0 || (W != nullptr && packed != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace_bytes >= kWorkspaceBytes, TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(W, 16) && twn_aligned(packed, 16) && twn_aligned(stats, 8) &&
                    twn_aligned(workspace, 256) && twn_aligned(codes_i8, 16), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    cudaStream_t s = twn_cu(stream);
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, 128, s));
    const bool flat = (rows <= 1) || (ld_codes == cols);
    const long long fast_units = flat ? n / 512 : 0;
    const long long rest_words = (long long)rows * (ld_codes / 16) - fast_units * 32;
    long long work = fast_units * 32 / 4;
    if (rest_words > work) work = rest_words;
    code_pack_kernel<<<grid_for(work, dev.sm_count), kThreads, 0, s>>>(W, rows, cols, ld_codes, fast_units, packed,
                                                                       codes_i8, workspace, stats);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" size_t twn_ternarize_batch_workspace_bytes(int count)
{
    return count > 0 ? (size_t)count * (256 + 4 * size_t(kMaxBlocks) * 8) : 0;
}

extern "C" int twn_ternarize_batch(const twn_ternarize_item_t *items, int count, double delta_factor,
                                   void *workspace, size_t workspace_bytes, twn_stream_t stream)
{
    TWN_REQUIRE(count >= 0 && count <= kMaxBatch, TWN_ERR_INVALID_ARG);
    if (count == 0) return TWN_OK;
    TWN_REQUIRE(items != nullptr && workspace != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(delta_factor >= 0.0 && delta_factor == delta_factor, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace_bytes >= twn_ternarize_batch_workspace_bytes(count), TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(workspace, 256), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;

    BatchParams A, B;
    A.count = B.count = count;
    unsigned int ga = 0, gb = 0;
    for (int t = 0; t < count; ++t) {
        const twn_ternarize_item_t &it = items[t];
        TWN_REQUIRE(it.rows >= 0 && it.cols >= 0 && it.stats != nullptr, TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(it.ld_codes >= it.cols && it.ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
        const long long n = (long long)it.rows * it.cols;
        TWN_REQUIRE(n == 0 || (it.W != nullptr && it.packed != nullptr), TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(twn_aligned(it.W, 16) && twn_aligned(it.packed, 16) && twn_aligned(it.stats, 8) &&
                        twn_aligned(it.codes_i8, 16), TWN_ERR_MISALIGNED);
        // the same grids and the same split into fast units and rest as a call of its own
        const bool flat = (it.rows <= 1) || (it.ld_codes == it.cols);
        const long long fast_units = flat ? n / 512 : 0;
        const long long rest_words = (long long)it.rows * (it.ld_codes / 16) - fast_units * 32;
        long long work = fast_units * 32 / 4;
        if (rest_words > work) work = rest_words;
        BatchItem bi;
        bi.W = it.W; bi.rows = it.rows; bi.cols = it.cols; bi.ld_codes = it.ld_codes; bi.fast_units = fast_units;
        bi.packed = it.packed; bi.codes_i8 = it.codes_i8; bi.stats = it.stats;
        A.item[t] = B.item[t] = bi;
        A.first_block[t] = ga;
        B.first_block[t] = gb;
        ga += (unsigned int)grid_for((n / 4 + 3) / 4, dev.sm_count);
        gb += (unsigned int)grid_for(work, dev.sm_count);
    }
    A.first_block[count] = ga;
    B.first_block[count] = gb;
    cudaStream_t s = twn_cu(stream);
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, (size_t)count * 256, s));     // the tickets start at zero
    sum_abs_batch_kernel<<<ga, kThreads, 0, s>>>(A, delta_factor, workspace);
    code_pack_batch_kernel<<<gb, kThreads, 0, s>>>(B, workspace);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

// ---- the variant that allocates nothing ------------------------------------------------
// Scratch for twn_ternarize_static: tickets and per-block partials, same layout as a caller's
// workspace.  File-scope device storage, one copy per GPU that loads the library.  In host
// code the name `g_static_scratch` is only a handle for cudaGetSymbolAddress, never a pointer
// a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[TWN_TERNARIZE_STATIC_SCRATCH_BYTES];
static_assert(TWN_TERNARIZE_STATIC_SCRATCH_BYTES >= kWorkspaceBytes, "static scratch too small");

// Device address of g_static_scratch on the current device, looked up once per device.
static int static_scratch_ptr(int ordinal, void **out)
{
    static void *cached[64] = {nullptr};
    if (ordinal < 0 || ordinal >= 64) return TWN_ERR_CUDA;
    if (cached[ordinal] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return TWN_ERR_CUDA;
        cached[ordinal] = p;
    }
    *out = cached[ordinal];
    return TWN_OK;
}

extern "C" int twn_ternarize_static(const float *W, int64_t rows, int64_t cols, double delta_factor,
                                    twn_stats_t *stats, uint32_t *packed, int64_t ld_codes,
                                    int8_t *codes_i8, twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(stats != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(delta_factor >= 0.0 && delta_factor == delta_factor, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(cols == 0 || rows <= TWN_TERNARIZE_STATIC_MAX_WEIGHTS / cols, TWN_ERR_TOO_LARGE);
    const long long n = (long long)rows * cols;
    TWN_REQUIRE(n <= TWN_TERNARIZE_STATIC_MAX_WEIGHTS, TWN_ERR_TOO_LARGE);
    TWN_REQUIRE(n == 0 || (W != nullptr && packed != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(W, 16) && twn_aligned(packed, 16) && twn_aligned(stats, 8) &&
                    twn_aligned(codes_i8, 16), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    void *scratch = nullptr;
    rc = static_scratch_ptr(dev.ordinal, &scratch);
    if (rc != TWN_OK) return rc;
    cudaStream_t s = twn_cu(stream);

    // the array still holds the previous call's partials; only the two tickets must start at zero
    TWN_CUDA_OK(cudaMemsetAsync(scratch, 0, 128, s));

    const int g1 = grid_for((n / 4 + 3) / 4, dev.sm_count);
    sum_abs_kernel<<<g1, kThreads, 0, s>>>(W, n, delta_factor, scratch, stats);

    const bool flat = (rows <= 1) || (ld_codes == cols);
    const long long fast_units = flat ? n / 512 : 0;
    const long long rest_words = (long long)rows * (ld_codes / 16) - fast_units * 32;
    long long work = fast_units * 32 / 4;
    if (rest_words > work) work = rest_words;
    const int g2 = grid_for(work, dev.sm_count);
    code_pack_kernel<<<g2, kThreads, 0, s>>>(W, rows, cols, ld_codes, fast_units, packed, codes_i8,
                                             scratch, stats);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_pack(const int8_t *codes, int64_t rows, int64_t cols, uint32_t *packed,
                        int64_t ld_codes, twn_stats_t *counts, twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
    const long long n = (long long)rows * cols;
    TWN_REQUIRE(n == 0 || (codes != nullptr && packed != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(packed, 16) && twn_aligned(counts, 8), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long words = (long long)rows * (ld_codes / 16);
    if (words == 0) {
        if (counts) TWN_CUDA_OK(cudaMemsetAsync(counts, 0, sizeof(twn_stats_t), twn_cu(stream)));
        return TWN_OK;
    }
    const int vec_ok = twn_aligned(codes, 16) && (cols % 16 == 0);
    if (counts) TWN_CUDA_OK(cudaMemsetAsync(counts, 0, sizeof(twn_stats_t), twn_cu(stream)));
    pack_kernel<<<grid_for(words, dev.sm_count), kThreads, 0, twn_cu(stream)>>>(
        codes, rows, cols, ld_codes, vec_ok, packed, counts);
    if (counts) finish_counts_kernel<<<1, 1, 0, twn_cu(stream)>>>(counts, (unsigned long long)n);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int64_t ld_codes,
                          int8_t *codes, int32_t *dev_status, twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
    const long long n = (long long)rows * cols;
    TWN_REQUIRE(n == 0 || (codes != nullptr && packed != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(packed, 16) && twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    if (n == 0) return TWN_OK;
    const int vec_ok = twn_aligned(codes, 16) && (cols % 16 == 0);
    const long long items = (long long)rows * ((cols + 15) / 16);
    unpack_kernel<<<grid_for(items, dev.sm_count), kThreads, 0, twn_cu(stream)>>>(
        packed, rows, cols, ld_codes, vec_ok, codes, dev_status);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_transpose_codes(const uint32_t *packed_fwd, int64_t ld_fwd,
                                   const twn_conv_desc_t *d, uint32_t *packed_bwd, int64_t ld_bwd,
                                   twn_stream_t stream)
{
    TWN_REQUIRE(d != nullptr && packed_fwd != nullptr && packed_bwd != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->Cin > 0 && d->Cout > 0 && d->kh > 0 && d->kw > 0, TWN_ERR_INVALID_ARG);
    const long long taps = (long long)d->kh * d->kw;
    TWN_REQUIRE(ld_fwd % 64 == 0 && ld_fwd >= taps * d->Cin, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_bwd % 64 == 0 && ld_bwd >= taps * d->Cout, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(packed_fwd, 16) && twn_aligned(packed_bwd, 16), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long words = d->Cin * (ld_bwd / 16);
    TWN_REQUIRE(words < 0x7fffffffLL && d->Cout * (ld_fwd / 16) < 0x7fffffffLL && ld_fwd < 0x7fffffffLL &&
                    ld_bwd < 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    // threads' worth of work: one output word each, or one tap x 64 x 16 block of codes each
    const long long work = transpose_fast_ok((int)d->Cout, (int)d->Cin, (int)taps) ? taps * transpose_fast_groups((int)d->Cout) * (d->Cin / 16) : words;
    transpose_codes_kernel<<<grid_for(work, dev.sm_count), kThreads, 0, twn_cu(stream)>>>(
        packed_fwd, (int)ld_fwd, (int)d->Cout, (int)d->Cin, (int)taps, packed_bwd, (int)ld_bwd);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_transpose_codes_batch(const twn_transpose_item_t *items, int count, twn_stream_t stream)
{
    TWN_REQUIRE(count >= 0 && count <= kMaxBatch, TWN_ERR_INVALID_ARG);
    if (count == 0) return TWN_OK;
    TWN_REQUIRE(items != nullptr, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    TransposeBatch P;
    P.count = count;
    unsigned int g = 0;
    for (int t = 0; t < count; ++t) {
        const twn_transpose_item_t &it = items[t];
        const twn_conv_desc_t *d = &it.desc;
        TWN_REQUIRE(it.packed_fwd && it.packed_bwd, TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(d->Cin > 0 && d->Cout > 0 && d->kh > 0 && d->kw > 0, TWN_ERR_INVALID_ARG);
        const long long taps = (long long)d->kh * d->kw;
        TWN_REQUIRE(it.ld_fwd % 64 == 0 && it.ld_bwd % 64 == 0 && it.ld_fwd >= taps * d->Cin && it.ld_bwd >= taps * d->Cout,
                    TWN_ERR_INVALID_ARG);
        TWN_REQUIRE(twn_aligned(it.packed_fwd, 16) && twn_aligned(it.packed_bwd, 16), TWN_ERR_MISALIGNED);
        const long long words = d->Cin * (it.ld_bwd / 16);
        TWN_REQUIRE(words < 0x7fffffffLL && d->Cout * (it.ld_fwd / 16) < 0x7fffffffLL && it.ld_fwd < 0x7fffffffLL &&
                        it.ld_bwd < 0x7fffffffLL, TWN_ERR_INVALID_ARG);
        TransposeItem ti;
        ti.in = it.packed_fwd; ti.out = it.packed_bwd; ti.ld_in = (int)it.ld_fwd; ti.ld_out = (int)it.ld_bwd;
        ti.Cout = (int)d->Cout; ti.Cin = (int)d->Cin; ti.taps = (int)taps;
        P.item[t] = ti;
        P.first_block[t] = g;
        const long long work = transpose_fast_ok(ti.Cout, ti.Cin, ti.taps) ? taps * transpose_fast_groups(ti.Cout) * (d->Cin / 16) : words;
        g += (unsigned int)grid_for(work, dev.sm_count);
    }
    P.first_block[count] = g;
    transpose_codes_batch_kernel<<<g, kThreads, 0, twn_cu(stream)>>>(P);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_fold_codes(const twn_conv_desc_t *d, const uint32_t *packed, int64_t ld_codes,
                              uint32_t *packed_folded, int64_t ld_folded, twn_stream_t stream)
{
    int64_t ldf = 0;
    int rc = twn_fold_dims(d, nullptr, nullptr, &ldf);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(packed && packed_folded, TWN_ERR_INVALID_ARG);
    const long long K = (long long)d->kh * d->kw * d->Cin;
    TWN_REQUIRE(ld_codes % 64 == 0 && ld_codes >= K && ld_folded == ldf, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(packed, 16) && twn_aligned(packed_folded, 16), TWN_ERR_MISALIGNED);
    TWN_REQUIRE(d->Cout * (ldf / 16) < 0x7fffffffLL && d->Cout * (ld_codes / 16) < 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    fold_codes_kernel<<<grid_for(d->Cout * (ldf / 16), dev.sm_count), kThreads, 0, twn_cu(stream)>>>(
        packed, (int)ld_codes, (int)d->Cout, (int)d->Cin, d->kh, d->kw, packed_folded, (int)ldf);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}
