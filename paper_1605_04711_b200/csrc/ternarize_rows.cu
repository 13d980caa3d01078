// Per-filter threshold ternarization fused with 2-bit packing: Algorithm 1 as printed, whose
// first loop runs over the filters of a layer.  Filter r (row r of the fp32 master weights)
// gets its own threshold delta_r = factor * mean |W_r| (Sec. 2.3), its own codes (Eq. 3) and
// its own scale alpha_r = mean of |W_r,i| over |W_r,i| > delta_r (Eq. 5).
//
// One thread block per filter.  The threshold needs the whole filter before any code can be
// written, but a filter is small (25 ... 8192 weights in the networks of the paper), so the
// block keeps it in shared memory between the two steps: each weight crosses HBM once
// (4 bytes read, 0.25 bytes written), against two reads for the per-layer rule.  Several
// blocks share an SM, so the loads of one filter overlap the coding of another.  Filters
// longer than the shared-memory budget, or whose rows are not 16-byte aligned, are read a
// second time (from L2, as a rule).  Both sums are fp64 with a fixed order (per-thread
// partials, shuffle tree, shared-memory tree): same inputs, same bits.  No scratch memory.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr long long kSmemCols = 16384;                      // longest filter kept in shared memory (64 KB)

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

// Block-wide sums with a fixed order: a shuffle tree per warp, one partial per warp in shared
// memory, and after a single barrier every thread adds the kWarps partials in index order.
__device__ __forceinline__ double block_sum_all(double v, double *part /* kWarps entries, not in use by a slower warp */)
{
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) r += part[w];
    return r;
}
// The same for a floating-point and an integer quantity at once (one barrier for both).
__device__ __forceinline__ void block_sum_all2(double &a, unsigned long long &b, double *part_a, unsigned long long *part_b)
{
    a = warp_sum(a);
    b = warp_sum(b);
    if ((threadIdx.x & 31) == 0) { part_a[threadIdx.x >> 5] = a; part_b[threadIdx.x >> 5] = b; }
    __syncthreads();
    double ra = 0.0;
    unsigned long long rb = 0ull;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { ra += part_a[w]; rb += part_b[w]; }
    a = ra;
    b = rb;
}

// Bit position of element e (0..15) inside its packed word (the layout of twn_ternarize): even
// elements fill the low half-word, odd elements the high one, each from its top bits down.
__device__ __forceinline__ int field_pos(int e) { return 14 - 2 * (e >> 1) + 16 * (e & 1); }

// 2-bit field of one weight against the threshold: 00 = 0, 01 = +1, 11 = -1 (Eq. 3; a weight
// equal to the threshold is 0).  Kept magnitudes are summed in fp64.  Branch-free and short: the
// coding sweep is bound by instruction issue, not by memory.
__device__ __forceinline__ uint32_t field_of(float w, float thr, double &kept)
{
    const bool keep = fabsf(w) > thr;
    kept += (double)(keep ? fabsf(w) : 0.0f);
    return keep ? ((__float_as_uint(w) >> 31) * 2u + 1u) : 0u;
}

__device__ __forceinline__ int8_t code_of(uint32_t f) { return (f & 1u) ? ((f & 2u) ? (int8_t)-1 : (int8_t)1) : (int8_t)0; }

// MODE 0: any alignment, scalar loads, the filter is read twice.
// MODE 1: rows 16-byte aligned and cols % 4 == 0, filter longer than the shared-memory budget: read twice.
// MODE 2: as 1, and the filter (cols * 4 bytes of dynamic shared memory) stays on chip between the steps.
template <int MODE>
__global__ void __launch_bounds__(kThreads, 6)      // six blocks of 32 KB filters per SM: at most 40 registers
ternarize_rows_kernel(const float *__restrict__ W, long long rows, long long cols, double factor,
                      twn_stats_t *__restrict__ stats, uint32_t *__restrict__ packed, long long wpr,
                      int8_t *__restrict__ codes_i8)
{
    extern __shared__ float4 rowbuf[];
    __shared__ double red_s[kWarps], red_k[kWarps];      // partials of the two sweeps: separate, so that a warp
    __shared__ unsigned long long red_u[kWarps];         // ahead of the others never overwrites what they still read
    const int tid = threadIdx.x, lane = tid & 31;
    const long long words = (cols + 15) >> 4;         // words that hold codes; the rest of a row is padding
    const int n4 = (int)(cols >> 2);

    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const float *Wr = W + row * cols;
        uint32_t *Pr = packed + row * wpr;
        int8_t *Cr = codes_i8 ? codes_i8 + row * cols : nullptr;

        // ---- step 1: S = sum |W_r,i|  ->  delta_r
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
        if (MODE >= 1) {
            const float4 *W4 = reinterpret_cast<const float4 *>(Wr);
#pragma unroll 8
            for (int i = tid; i < n4; i += kThreads) {
                const float4 x = __ldg(W4 + i);
                if (MODE == 2) rowbuf[i] = x;
                a0 += (double)fabsf(x.x); a1 += (double)fabsf(x.y); a2 += (double)fabsf(x.z); a3 += (double)fabsf(x.w);
            }
        } else {
            for (long long i = tid; i < cols; i += kThreads) a0 += (double)fabsf(__ldg(Wr + i));
        }
        const double S = block_sum_all((a0 + a1) + (a2 + a3), red_s);
        const double delta = cols > 0 ? factor * (S / (double)cols) : 0.0;
        // a float w satisfies |w| > delta exactly when |w| > the largest float <= delta
        const float thr = __double2float_rd(delta);

        // ---- step 2: codes, packed 16 per word; sum and counts of the kept set
        double k0 = 0.0, k1 = 0.0;
        unsigned int nz = 0u, ng = 0u;             // kept, negative (a filter has fewer than 2^31 weights)
        if (MODE == 2) {
            // float4 i holds elements 4i..4i+3: a quarter of word i/4, whose other quarters sit in
            // the neighbouring lanes of the same group of four; every thread reads back what it wrote.
            // Elements 0 and 2 of the quarter go to the low half-word, 1 and 3 to the high one, the
            // first of each pair two bits above the second.
            const int sh = 12 - 4 * (lane & 3);    // field_pos of element 2 of this lane's quarter
            auto quarter = [&](const int i, const float4 x, const bool in_row) {
                const uint32_t f0 = field_of(x.x, thr, k0), f1 = field_of(x.y, thr, k1);
                const uint32_t f2 = field_of(x.z, thr, k0), f3 = field_of(x.w, thr, k1);
                uint32_t part = ((f0 * 4u + f2) | ((f1 * 4u + f3) << 16)) << sh;
                nz += __popc(part & 0x55555555u);
                ng += __popc(part & 0xAAAAAAAAu);
                if (Cr && in_row) {
                    // cols % 4 == 0 and the matrix is aligned: the four codes are one aligned word
                    const uint32_t c4 = (uint32_t)(uint8_t)code_of(f0) | ((uint32_t)(uint8_t)code_of(f1) << 8) |
                                        ((uint32_t)(uint8_t)code_of(f2) << 16) | ((uint32_t)(uint8_t)code_of(f3) << 24);
                    *reinterpret_cast<uint32_t *>(Cr + 4 * (long long)i) = c4;
                }
                part |= __shfl_xor_sync(0xffffffffu, part, 1);
                part |= __shfl_xor_sync(0xffffffffu, part, 2);
                if ((lane & 3) == 0 && in_row) Pr[i >> 2] = part;
            };
            // whole sweeps of the block first (no bounds to check), then one ragged sweep
            const int full = n4 / kThreads;
#pragma unroll 4
            for (int it = 0; it < full; ++it) {
                const int i = it * kThreads + tid;
                quarter(i, rowbuf[i], true);
            }
            if (full * kThreads < n4) {
                const int i = full * kThreads + tid;
                quarter(i, i < n4 ? rowbuf[i] : make_float4(0.0f, 0.0f, 0.0f, 0.0f), i < n4);
            }
        } else {
            for (long long j = tid; j < words; j += kThreads) {
                uint32_t word = 0u;
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const long long c = 16 * j + e;
                    if (c < cols) {
                        const uint32_t f = field_of(__ldg(Wr + c), thr, k0);
                        word |= f << field_pos(e);
                        if (Cr) Cr[c] = code_of(f);
                    }
                }
                nz += __popc(word & 0x55555555u);
                ng += __popc(word & 0xAAAAAAAAu);
                Pr[j] = word;
            }
        }
        // padding words of the row
        for (long long j = words + tid; j < wpr; j += kThreads) Pr[j] = 0u;

        double K = k0 + k1;
        // positives in the low, negatives in the high half
        unsigned long long c2 = (unsigned long long)(nz - ng) + ((unsigned long long)ng << 32);
        block_sum_all2(K, c2, red_k, red_u);
        if (tid == 0) {
            const unsigned long long n_pos = c2 & 0xFFFFFFFFull, n_neg = c2 >> 32;
            twn_stats_t st;
            st.delta = delta;
            st.alpha = (n_pos + n_neg) > 0 ? K / (double)(n_pos + n_neg) : 0.0;
            st.sum_abs = S;
            st.sum_abs_kept = K;
            st.n_neg = n_neg;
            st.n_pos = n_pos;
            st.n_zero = (unsigned long long)cols - n_pos - n_neg;
            st.status = isfinite(S) ? TWN_OK : TWN_ERR_NONFINITE;
            st.reserved = 0;
            stats[row] = st;
        }
        __syncthreads();       // the partials are free for the next filter of this block
    }
}

// scale_out[r] = alpha_r * scale_in[r]; the worst status of the filters goes to *dev_status.
__global__ void __launch_bounds__(kThreads)
rows_scale_kernel(const twn_stats_t *__restrict__ stats, long long rows, const float *__restrict__ scale_in,
                  float *__restrict__ scale_out, int32_t *dev_status)
{
    const long long r = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (r >= rows) return;
    const float a = (float)stats[r].alpha;
    scale_out[r] = scale_in ? a * scale_in[r] : a;
    if (dev_status && stats[r].status != TWN_OK) atomicMin(dev_status, stats[r].status);
}

}  // namespace

extern "C" int twn_ternarize_rows(const float *W, int64_t rows, int64_t cols, double delta_factor,
                                  twn_stats_t *stats, uint32_t *packed, int64_t ld_codes,
                                  int8_t *codes_i8, twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0 && cols <= 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(delta_factor >= 0.0 && delta_factor == delta_factor, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 64 == 0, TWN_ERR_INVALID_ARG);
    if (rows == 0) return TWN_OK;
    TWN_REQUIRE(stats != nullptr && packed != nullptr && (cols == 0 || W != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(W, 4) && twn_aligned(packed, 16) && twn_aligned(stats, 8), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    // one block per filter: blocks are scheduled as others retire, so filters of any number spread
    // evenly over the SMs (the row loop of the kernel only serves more than 2^31 - 1 filters)
    const int grid = (int)(rows < 0x7fffffffLL ? rows : 0x7fffffffLL);
    const bool vec = twn_aligned(W, 16) && cols % 4 == 0 && twn_aligned(codes_i8, 4);
    if (vec && cols <= kSmemCols) {
        static bool attr_set[64] = {false};
        if (!attr_set[dev.ordinal]) {
            TWN_CUDA_OK(cudaFuncSetAttribute(ternarize_rows_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(kSmemCols * 4)));
            attr_set[dev.ordinal] = true;
        }
        ternarize_rows_kernel<2><<<grid, kThreads, (size_t)cols * 4, twn_cu(stream)>>>(
            W, rows, cols, delta_factor, stats, packed, ld_codes / 16, codes_i8);
    } else if (vec) {
        ternarize_rows_kernel<1><<<grid, kThreads, 0, twn_cu(stream)>>>(W, rows, cols, delta_factor, stats, packed,
                                                                      ld_codes / 16, codes_i8);
    } else {
        ternarize_rows_kernel<0><<<grid, kThreads, 0, twn_cu(stream)>>>(W, rows, cols, delta_factor, stats, packed,
                                                                      ld_codes / 16, codes_i8);
    }
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_rows_scale(const twn_stats_t *stats, int64_t rows, const float *scale_in, float *scale_out,
                              int32_t *dev_status, twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0, TWN_ERR_INVALID_ARG);
    if (rows == 0) return TWN_OK;
    TWN_REQUIRE(stats != nullptr && scale_out != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(stats, 8) && twn_aligned(scale_in, 4) && twn_aligned(scale_out, 4) &&
                    twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const int grid = (int)((rows + kThreads - 1) / kThreads);
    rows_scale_kernel<<<grid, kThreads, 0, twn_cu(stream)>>>(stats, rows, scale_in, scale_out, dev_status);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}
