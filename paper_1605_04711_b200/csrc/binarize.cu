// Binary precision weights (Sec. 3: the BPWN baseline binarizes the weights with the sign function;
// like the ternary weights they carry one scale per layer) fused with 1-bit packing, and the helpers
// for the 1-bit format (unpack, re-layout for the backward-for-data pass).
//
//   B_i = +1 if W_i >= 0, -1 if W_i < 0;      alpha = (1/n) sum |W_i|
//
// Neither needs a threshold, so one sweep over the fp32 master weights does both: 4 bytes read and
// 1/32 byte written per weight, bound by HBM bandwidth.  A warp works on one word of 32 codes at a
// time: lane l loads the element whose bit it owns in the packed word (a permutation inside one
// 128-byte line, so the load is fully coalesced), and a warp vote on "negative" IS the packed word.
// sum |W| has a fixed order: per-lane fp64 partial sums, shuffle tree, block tree, one partial per
// block, folded in index order by the block that finishes last.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxBlocks = 2048;
// workspace: [0,256) ticket, then kMaxBlocks fp64 partial sums and kMaxBlocks 8-byte negative counts
constexpr size_t kBinWorkspaceBytes = 256 + 2 * size_t(kMaxBlocks) * 8;

// element of a 32-code group whose bit is bit l of the word: even elements fill the low half-word from
// bit 15 down, odd elements the high half-word from bit 31 down
__device__ __forceinline__ int element_of_bit(int l) { return l < 16 ? 2 * (15 - l) : 2 * (31 - l) + 1; }
__host__ __device__ inline int bit_of_element(int e) { return 15 - (e >> 1) + 16 * (e & 1); }

__device__ __forceinline__ double warp_sum_d(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u(unsigned long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kThreads)
binarize_kernel(const float *__restrict__ W, long long rows, long long cols, long long ld_codes,
                uint32_t *__restrict__ packed, void *ws_raw, twn_stats_t *__restrict__ stats)
{
    __shared__ double red_s[kWarps];
    __shared__ unsigned long long red_n[kWarps];
    __shared__ bool is_last;
    unsigned int *ticket = reinterpret_cast<unsigned int *>(ws_raw);
    double *part_sum = reinterpret_cast<double *>(static_cast<char *>(ws_raw) + 256);
    unsigned long long *part_neg = reinterpret_cast<unsigned long long *>(part_sum + kMaxBlocks);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int e = element_of_bit(lane);
    const long long wpr = ld_codes >> 5;                       // words per packed row
    const long long total_words = rows * wpr;
    const long long warp_id = (long long)blockIdx.x * kWarps + warp, n_warps = (long long)gridDim.x * kWarps;
    // a contiguous matrix whose rows are whole words is one long row
    const bool flat = (ld_codes == cols);
    const long long n = rows * cols;

    double acc = 0.0;
    unsigned long long negs = 0;
    if (flat) {
        // sixteen words per warp and iteration, their loads issued before any is used: the sweep is bound by the
        // bytes a warp keeps in flight
        constexpr int kU = 16;
        double a1 = 0.0;
        for (long long w0 = warp_id * kU; w0 < total_words; w0 += n_warps * kU) {
            float x[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) x[u] = (w0 + u < total_words) ? __ldg(W + ((w0 + u) << 5) + e) : 0.0f;
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                if (u & 1) a1 += (double)fabsf(x[u]); else acc += (double)fabsf(x[u]);
                const unsigned int word = __ballot_sync(0xffffffffu, x[u] < 0.0f);     // -0.0 and NaN vote "not negative"
                if (lane == u && w0 + u < total_words) {
                    packed[w0 + u] = word;
                    negs += (unsigned long long)__popc(word);
                }
            }
        }
        acc += a1;
    } else {
        for (long long w = warp_id; w < total_words; w += n_warps) {
            const long long r = w / wpr, c = ((w - r * wpr) << 5) + e;
            const bool valid = c < cols;
            const float x = valid ? __ldg(W + r * cols + c) : 0.0f;
            acc += (double)fabsf(x);
            const unsigned int word = __ballot_sync(0xffffffffu, x < 0.0f);
            if (lane == 0) {
                packed[w] = word;
                negs += (unsigned long long)__popc(word);
            }
        }
    }
    // block partials
    acc = warp_sum_d(acc);
    negs = warp_sum_u(negs);
    if (lane == 0) { red_s[warp] = acc; red_n[warp] = negs; }
    __syncthreads();
    if (warp == 0) {
        double s = lane < kWarps ? red_s[lane] : 0.0;
        unsigned long long c = lane < kWarps ? red_n[lane] : 0ull;
        s = warp_sum_d(s);
        c = warp_sum_u(c);
        if (lane == 0) { part_sum[blockIdx.x] = s; part_neg[blockIdx.x] = c; }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    // the last block folds the partials in index order
    double s = 0.0;
    unsigned long long c = 0;
    for (int b = threadIdx.x; b < (int)gridDim.x; b += kThreads) { s += __ldcg(part_sum + b); c += __ldcg(part_neg + b); }
    s = warp_sum_d(s);
    c = warp_sum_u(c);
    __syncthreads();
    if (lane == 0) { red_s[warp] = s; red_n[warp] = c; }
    __syncthreads();
    if (warp == 0) {
        s = lane < kWarps ? red_s[lane] : 0.0;
        c = lane < kWarps ? red_n[lane] : 0ull;
        s = warp_sum_d(s);
        c = warp_sum_u(c);
        if (lane == 0) {
            stats->delta = 0.0;
            stats->alpha = n > 0 ? s / (double)n : 0.0;
            stats->sum_abs = s;
            stats->sum_abs_kept = s;
            stats->n_neg = c;
            stats->n_zero = 0;
            stats->n_pos = (unsigned long long)n - c;
            stats->status = isfinite(s) ? TWN_OK : TWN_ERR_NONFINITE;
            stats->reserved = 0;
            *ticket = 0u;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
unpack_b1_kernel(const uint32_t *__restrict__ packed, long long rows, long long cols, long long ld_codes,
                 int8_t *__restrict__ codes)
{
    const long long wpr = ld_codes >> 5, total = rows * cols;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < total; i += (long long)gridDim.x * kThreads) {
        const long long r = i / cols, c = i - r * cols;
        const uint32_t w = __ldg(packed + r * wpr + (c >> 5));
        codes[i] = ((w >> bit_of_element((int)(c & 31))) & 1u) ? -1 : 1;
    }
}

// [Cout][taps][Cin] -> [Cin][taps][Cout]: a thread builds one word of the output
__global__ void __launch_bounds__(kThreads)
transpose_b1_kernel(const uint32_t *__restrict__ in, long long ld_in, int Cout, int Cin, int taps,
                    uint32_t *__restrict__ out, long long ld_out)
{
    const long long wpr_in = ld_in >> 5, wpr_out = ld_out >> 5, total = (long long)Cin * wpr_out;
    for (long long w = (long long)blockIdx.x * kThreads + threadIdx.x; w < total; w += (long long)gridDim.x * kThreads) {
        const long long c = w / wpr_out, j0 = (w - c * wpr_out) << 5;
        uint32_t word = 0u;
        for (int e = 0; e < 32; ++e) {
            const long long j = j0 + e;                       // column of the output row: tap * Cout + o
            if (j >= (long long)taps * Cout) break;
            const long long t = j / Cout, o = j - t * Cout;
            const long long src = t * Cin + c;                // column of input row o
            const uint32_t bit = (__ldg(in + o * wpr_in + (src >> 5)) >> bit_of_element((int)(src & 31))) & 1u;
            word |= bit << bit_of_element(e);
        }
        out[w] = word;
    }
}

int grid_for_words(long long work, int sms)
{
    long long g = (work + kThreads - 1) / kThreads;
    const long long cap = (long long)sms * 8 < kMaxBlocks ? (long long)sms * 8 : kMaxBlocks;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

}  // namespace

extern "C" size_t twn_binarize_workspace_bytes(void) { return kBinWorkspaceBytes; }

extern "C" int twn_binarize(const float *W, int64_t rows, int64_t cols, twn_stats_t *stats, uint32_t *packed,
                            int64_t ld_codes, void *workspace, size_t workspace_bytes, twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0 && stats != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ld_codes >= cols && ld_codes % 128 == 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(cols == 0 || rows <= (int64_t)0x3fffffffffffLL / (cols > ld_codes ? cols : ld_codes), TWN_ERR_INVALID_ARG);
    const long long n = (long long)rows * cols;
    TWN_REQUIRE(n == 0 || (W != nullptr && packed != nullptr), TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(workspace != nullptr && workspace_bytes >= kBinWorkspaceBytes, TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(W, 4) && twn_aligned(packed, 16) && twn_aligned(stats, 8) && twn_aligned(workspace, 256),
                TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    cudaStream_t s = twn_cu(stream);
    TWN_CUDA_OK(cudaMemsetAsync(workspace, 0, 64, s));           // the ticket
    const long long words = (long long)rows * (ld_codes / 32);
    // a warp takes one word per iteration
    const int grid = grid_for_words(words * 32, dev.sm_count);
    binarize_kernel<<<grid, kThreads, 0, s>>>(W, rows, cols, ld_codes, packed, workspace, stats);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_unpack_b1(const uint32_t *packed, int64_t rows, int64_t cols, int64_t ld_codes, int8_t *codes,
                             twn_stream_t stream)
{
    TWN_REQUIRE(rows >= 0 && cols >= 0 && ld_codes >= cols && ld_codes % 128 == 0, TWN_ERR_INVALID_ARG);
    if (rows == 0 || cols == 0) return TWN_OK;
    TWN_REQUIRE(packed && codes, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(packed, 16), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    unpack_b1_kernel<<<grid_for_words((long long)rows * cols, dev.sm_count), kThreads, 0, twn_cu(stream)>>>(
        packed, rows, cols, ld_codes, codes);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

extern "C" int twn_transpose_codes_b1(const uint32_t *packed_fwd, int64_t ld_fwd, const twn_conv_desc_t *d,
                                      uint32_t *packed_bwd, int64_t ld_bwd, twn_stream_t stream)
{
    TWN_REQUIRE(d != nullptr && packed_fwd && packed_bwd, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->Cin > 0 && d->Cout > 0 && d->kh > 0 && d->kw > 0, TWN_ERR_INVALID_ARG);
    const long long taps = (long long)d->kh * d->kw;
    TWN_REQUIRE(ld_fwd % 128 == 0 && ld_bwd % 128 == 0 && ld_fwd >= taps * d->Cin && ld_bwd >= taps * d->Cout,
                TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->Cin <= 0x7fffffffLL && d->Cout <= 0x7fffffffLL && taps <= 4096, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(packed_fwd, 16) && twn_aligned(packed_bwd, 16), TWN_ERR_MISALIGNED);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    const long long words = d->Cin * (ld_bwd / 32);
    transpose_b1_kernel<<<grid_for_words(words, dev.sm_count), kThreads, 0, twn_cu(stream)>>>(
        packed_fwd, ld_fwd, (int)d->Cout, (int)d->Cin, (int)taps, packed_bwd, ld_bwd);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}
