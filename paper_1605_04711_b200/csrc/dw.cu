// Straight-through weight gradient (Algorithm 1, UpdateParameters; Fig. 1 caption): the
// gradient with respect to T = alpha * W~ computed by ordinary back-propagation and applied
// to the fp32 master weights unchanged,
//     dW[o, r, s, c] = sum_{b,ho,wo} dZ[b,ho,wo,o] * X[b, ho*stride - pad + r, wo*stride - pad + s, c].
// A dense bf16 x bf16 -> fp32 contraction whose reduction runs over the pixels, i.e. over the
// slow dimension of both NHWC operands.  tcgen05 takes such operands directly ("MN-major"
// shared-memory descriptors), so the dZ tile and the tap-shifted X tile go from TMA straight
// into the MMA: D[o, c] += dZ_tile^T * X_tile, 64 or 128 pixels per k-block (a tensor copy of 128 rows
// moves its bytes almost twice as fast as one of 64, so the larger k-block is taken wherever its padding
// and the ring depth allow).
//
// One MMA covers up to four 64-channel column blocks of dW, taken in (tap, channel block)
// order, so narrow layers (Cin = 64) process four taps per pass over the dZ tile.
// The output has few tiles (Cout/128 x taps*Cin/256) but a long reduction (up to 8e5 pixels),
// so the pixels are split across CTAs; each CTA writes its fp32 partial tile to the workspace
// and a second kernel adds the partials in split order (deterministic, no atomics).
//
//   warp 0     TMA producer: lane j issues copy j of a k-block (gradient blocks, activation blocks)
//   warps 1, 6 one MMA-issuing thread each, alternate k-blocks, an accumulator each
//   warps 2-5, 7-10  epilogue (two per tensor-memory lane quadrant, alternate 32-column chunks): sum of the
//              two accumulators -> workspace
#include <cstddef>

#include "common.cuh"
#include "tc_ptx.cuh"


namespace {

constexpr int kDwMaxStages = 12;
constexpr int kDwPoolBytes = 208 * 1024;         // operand ring: stages of one or two blocks of dZ plus the X blocks
constexpr int kDwMaxMma = 8;                     // K = 16 pixels per MMA: 4 or 8 MMAs per k-block of 64 or 128 pixels
constexpr int kDwMaxCb = 4;                      // up to 256 input channels per tile
constexpr int kDwThreads = 352;                  // warp 0 producer, 1 and 6 MMA issuers, 2-5 and 7-10 epilogue
constexpr int kDwIssuerB = 6;                    // the warp of the second MMA-issuing thread
constexpr int kDwEpiWarps = 8;                   // two per tensor-memory lane quadrant; they take alternate 32-column chunks
constexpr int kDwMaxTaps = 64;
constexpr int kDwAccCols = 256;

struct DwTap { int16_t dh, dw; int32_t koff; };

struct DwParams {
    int n_otiles, n_taps, n_groups, splits, total_units;
    int cblocks, n_colblocks;    // 64-channel blocks per tap; column blocks = taps * cblocks, 4 per group
    int lgBW, lgBH, tw, th, tb, pix_tiles, tiles_per_split;
    int sw, sh;
    int Cout, Cin;
    long long K;                 // row length of dW and of a partial
    long long split_stride;      // elements between partials of consecutive splits
    float *partial;
    int vec_ok;
    int32_t *status;
    // row mode (stride-1 layers, 2..4 taps per filter row): a group is one filter row of one
    // 64-channel block.  Its kw column blocks read ONE activation tile with kw - 1 extra pixel
    // columns: tap s is the tile one pixel (128 bytes) further, so a single MMA of N = 64 kw
    // covers the row and the tile is loaded once instead of kw times.
    // Column mode (row_mode = 2) is the same with the roles of rows and columns swapped, for stride-1 layers with
    // one tap per filter row and 2..4 filter rows (the folded first layer of ResNet-18): the tile has kh - 1 extra
    // rows per image and tap r is the tile one row further; `kw` then holds kh.
    int row_mode, kw, x_bytes, k_group_bytes;
    int tap_stride_bytes;        // row / column mode: bytes between the tiles of consecutive taps (a pixel, or a row of the tile)
    int x_off;                   // byte offset of the activation blocks inside a stage (after the blocks of dZ)
    int kpix, n_mma, blk_bytes;  // pixels per k-block (64 or 128), its MMAs (K = 16 pixels each), bytes of one 64-channel block of it
    int mma_off[kDwMaxMma];      // byte offset of the 16 pixels of MMA i inside the activation tile
    int stages, stage_bytes;
    DwTap taps[kDwMaxTaps];
};

struct __align__(1024) DwSmem {
    // a stage: dZ as two 64-channel blocks (16 KB), then X: up to four 64-channel blocks, or one
    // tile with its extra columns in row mode
    uint8_t pool[kDwPoolBytes];
    // per epilogue warp: 32 rows x 16 fp32 of the accumulator (half a chunk), 16-byte pieces XOR-swizzled
    // by the row so that row-wise writes and the transposed reads are both free of bank conflicts
    float4 stg[kDwEpiWarps][32][4];
    unsigned long long full[kDwMaxStages], empty[kDwMaxStages], acc_full, acc_empty;
    uint32_t tmem_base;
    volatile int abort_flag;
};

// D[tmem] (+)= A[smem] * B[smem]^T issued by the calling thread alone, accumulate flag in a register.
__device__ __forceinline__ void dw_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void dw_commit(void *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(kDwThreads, 1)
dw_kernel(const __grid_constant__ CUtensorMap map_dz, const __grid_constant__ CUtensorMap map_x,
          const __grid_constant__ DwParams P)
{
    extern __shared__ uint8_t smem_raw[];
    DwSmem *sm = reinterpret_cast<DwSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    volatile int *abort_flag = &sm->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDwMaxStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        mbar_init(&sm->acc_full, 2);
        mbar_init(&sm->acc_empty, kDwEpiWarps);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm->tmem_base;

    // unit -> (o tile, group of column blocks, split); the split covers pixel tiles [p0, p1)
    auto unit_range = [&](int u, int &ot, int &gi, int &nb, int &sp, int &p0, int &p1) {
        sp = u % P.splits; u /= P.splits;
        gi = u % P.n_groups;
        ot = u / P.n_groups;
        if (P.row_mode) {
            nb = P.kw;
        } else {
            nb = P.n_colblocks - gi * kDwMaxCb;
            if (nb > kDwMaxCb) nb = kDwMaxCb;
        }
        p0 = sp * P.tiles_per_split;
        p1 = p0 + P.tiles_per_split;
        if (p1 > P.pix_tiles) p1 = P.pix_tiles;
        if (p0 > p1) p0 = p1;
    };
    // row mode: filter row and 64-channel block of group gi
    auto row_group = [&](int gi, int &r, int &cb0) {
        r = gi / P.cblocks;
        cb0 = gi - r * P.cblocks;
    };
    const int x_slot = (P.x_bytes + 1023) & ~1023;     // row mode: one activation tile

    if (warp == 0) {
        // ------------------------------------------------ TMA producer: the whole warp
        // Issuing a tensor copy holds its thread for roughly a hundred cycles, and a k-block needs up to six
        // of them (two gradient blocks, up to four activation blocks); here lane j issues copy j, all in the
        // same instruction.
        uint32_t it = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < P.total_units && ok; u += gridDim.x) {
            int ot, gi, nb, sp, p0, p1;
            unit_range(u, ot, gi, nb, sp, p0, p1);
            // the second 64-channel block of dZ is not loaded when it lies past Cout: what the MMA
            // then reads there lands in accumulator rows that are never stored
            const bool a1 = ot * 128 + 64 < P.Cout;
            const int nx = P.row_mode ? 1 : nb;
            const uint32_t bytes = (a1 ? 2 : 1) * P.blk_bytes + (P.row_mode ? P.x_bytes : nb * P.blk_bytes);
            // this lane's copy: lanes 0, 1 the two gradient blocks, lanes 2.. the activation blocks.
            // Everything that does not change along the pixel tiles is worked out here.
            bool active;
            const CUtensorMap *my_map;
            int my_c0, my_dw = 0, my_dh = 0, my_sw = 1, my_sh = 1;
            uint32_t my_off;
            if (lane < 2) {
                active = lane == 0 || a1;
                my_map = &map_dz;
                my_c0 = ot * 128 + lane * 64;
                my_off = (uint32_t)(lane * P.blk_bytes);
            } else {
                const int j = lane - 2;
                active = j < nx;
                my_map = &map_x;
                my_sw = P.sw; my_sh = P.sh;
                int t = 0, cb = 0;
                if (P.row_mode) {
                    // one box per 64-channel block, kw - 1 pixels wider than the tile
                    int r, cb0;
                    row_group(gi, r, cb0);
                    t = r * P.kw; cb = cb0 + j;
                    my_off = (uint32_t)(P.x_off + j * x_slot);
                } else {
                    const int i = gi * kDwMaxCb + (active ? j : 0);
                    t = i / P.cblocks; cb = i - t * P.cblocks;
                    my_off = (uint32_t)(P.x_off + j * P.blk_bytes);
                }
                const DwTap tap = P.taps[active ? t : 0];
                my_c0 = cb * 64; my_dw = tap.dw; my_dh = tap.dh;
            }
            // pixel tile p0 as (column tile, row tile, image tile), stepped without divisions
            int twi = p0 % P.tw, thi = (p0 / P.tw) % P.th, tbi = p0 / (P.tw * P.th);
            const int bstep = P.kpix >> (P.lgBW + P.lgBH);
            int s = it % P.stages;
            uint32_t ph = (it / P.stages) & 1u;
            for (int p = p0; p < p1; ++p, ++it) {
                uint8_t *const st = sm->pool + s * P.stage_bytes;
                const int w0 = twi << P.lgBW, h0 = thi << P.lgBH, b0 = tbi * bstep;
                if (!mbar_wait_warp(&sm->empty[s], ph ^ 1u, abort_flag, P.status, 32)) { ok = false; break; }
                if (lane == 0) mbar_expect_tx(&sm->full[s], bytes);
                __syncwarp();
                if (active) tma_load_4d(st + my_off, my_map, &sm->full[s], my_c0, w0 * my_sw + my_dw, h0 * my_sh + my_dh, b0);
                if (++twi == P.tw) { twi = 0; if (++thi == P.th) { thi = 0; ++tbi; } }
                if (++s == P.stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1 || warp == kDwIssuerB) {
        // Two MMA-issuing threads, each with an accumulator of its own (256 tensor-memory columns).
        // tcgen05.mma holds its issuing thread until the tensor core accepts the instruction, so whatever one
        // thread executes between two MMAs (waits, descriptor arithmetic, commits) is time the tensor core
        // idles unless another thread has work queued.  The threads take alternate k-blocks and the epilogue
        // adds the two accumulators; the ring has an even number of stages, so a stage always belongs to the
        // same thread and each full barrier has one waiter that sees every phase in turn.
        if (lane == 0) {
            const uint32_t me = warp == 1 ? 0u : 1u;
            uint32_t it = 0, lu = 0;     // lu counts the units that accumulate something
            bool ok = true;
            const uint32_t pool = smem_u32(sm->pool);
            const uint32_t st_step = (uint32_t)P.stage_bytes >> 4;
            for (int u = blockIdx.x; u < P.total_units && ok; u += gridDim.x) {
                int ot, gi, nb, sp, p0, p1;
                unit_range(u, ot, gi, nb, sp, p0, p1);
                if (p1 <= p0) continue;                      // the epilogue writes zeros for an empty split
                const uint32_t idesc = make_idesc_mn(128, 64 * nb);
                if (!mbar_wait(&sm->acc_empty, (lu & 1u) ^ 1u, abort_flag, P.status, 0)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem + me * kDwAccCols;
                // descriptors of stage 0; a stage further is st_step more in the address field.
                // 16 pixels per MMA = 16 rows of 128 bytes = 2048 bytes
                const uint64_t adesc0 = smem_desc_mn_sw128(pool, (uint32_t)P.blk_bytes);
                uint64_t bd[kDwMaxMma];
                if (P.row_mode) {
                    const uint32_t xt = pool + (uint32_t)P.x_off;
#pragma unroll
                    for (int j = 0; j < kDwMaxMma; ++j) bd[j] = smem_desc_mn_sw128_groups(xt + P.mma_off[j], (uint32_t)P.tap_stride_bytes, P.k_group_bytes);
                } else {
                    const uint64_t b0 = smem_desc_mn_sw128(pool + (uint32_t)P.x_off, (uint32_t)P.blk_bytes);
#pragma unroll
                    for (int j = 0; j < kDwMaxMma; ++j) bd[j] = b0 + 128 * j;
                }
                uint32_t s = it % P.stages;
                uint32_t ph = (it / P.stages) & 1u;
                uint32_t acc = 0;
                for (int p = p0; p < p1; ++p, ++it) {
                    if ((it & 1u) == me) {
                        if (!mbar_wait(&sm->full[s], ph, abort_flag, P.status, 0)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t so = (uint64_t)(s * st_step);
                        dw_mma(d_tmem, adesc0 + so, bd[0] + so, idesc, acc);
                        dw_mma(d_tmem, adesc0 + so + 128, bd[1] + so, idesc, 1u);
                        dw_mma(d_tmem, adesc0 + so + 256, bd[2] + so, idesc, 1u);
                        dw_mma(d_tmem, adesc0 + so + 384, bd[3] + so, idesc, 1u);
                        if (P.n_mma > 4) {
                            dw_mma(d_tmem, adesc0 + so + 512, bd[4] + so, idesc, 1u);
                            dw_mma(d_tmem, adesc0 + so + 640, bd[5] + so, idesc, 1u);
                            dw_mma(d_tmem, adesc0 + so + 768, bd[6] + so, idesc, 1u);
                            dw_mma(d_tmem, adesc0 + so + 896, bd[7] + so, idesc, 1u);
                        }
                        acc = 1u;
                        dw_commit(&sm->empty[s]);
                    }
                    if (++s == (uint32_t)P.stages) { s = 0; ph ^= 1u; }
                }
                if (ok) dw_commit(&sm->acc_full);
                ++lu;
            }
        }
    } else {
        // The accumulator of a unit is exposed time (a block mostly has one unit), so eight warps drain it: the
        // two warps of a lane quadrant take alternate 32-column chunks.
        const int q = warp & 3;
        const int set = warp > kDwIssuerB ? 1 : 0;
        uint32_t lu = 0, it = 0;
        for (int u = blockIdx.x; u < P.total_units; u += gridDim.x) {
            int ot, gi, nb, sp, p0, p1;
            unit_range(u, ot, gi, nb, sp, p0, p1);
            const bool have = p1 > p0;
            // which of the two accumulators hold something: the threads took the k-blocks in turn, starting
            // with the one whose number is the parity of `it`
            const uint32_t len = (uint32_t)(p1 - p0);
            const bool have0 = have && ((len + ((it & 1u) == 0u ? 1u : 0u)) >> 1) > 0u;
            const bool have1 = have && ((len + ((it & 1u) == 1u ? 1u : 0u)) >> 1) > 0u;
            it += len;
            if (have && !mbar_wait_warp(&sm->acc_full, lu & 1u, abort_flag, P.status, 32)) break;
            tc_fence_after();
            const int o = ot * 128 + q * 32 + lane;
            float *row = P.partial + (long long)sp * P.split_stride + (long long)o * P.K;
            int rr_ = 0, cb0 = 0;
            if (P.row_mode) row_group(gi, rr_, cb0);
            const int n_chunks = nb * 2;
#pragma unroll 1
            for (int c = set; c < n_chunks; c += 2) {
                // columns [32cc, 32cc+32) of an accumulator: half of column block cc/2
                const int cc = c;
                int t, cb;
                if (P.row_mode) {
                    cb = cb0;
                    t = rr_ * P.kw + (cc >> 1);
                } else {
                    const int i = gi * kDwMaxCb + (cc >> 1);
                    t = i / P.cblocks;
                    cb = i - t * P.cblocks;
                }
                const int ch0 = cb * 64 + (cc & 1) * 32;          // first input channel of this chunk
                float *dst = row + P.taps[t].koff + ch0;
                uint32_t v[32];
                const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16) + cc * 32;
                {
                    // the sum of the two threads' accumulators (fixed order: deterministic)
                    uint32_t w[32];
                    if (have0) tmem_ld32(t_lane, v);
                    if (have1) tmem_ld32(t_lane + kDwAccCols, w);
                    if (have0) tmem_wait_ld(v);
                    if (have1) tmem_wait_ld(w);
                    if (!have0) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = 0u;
                    }
                    if (have1) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
                    }
                }
                if (P.vec_ok && ch0 + 32 <= P.Cin) {
                    // through shared memory, half a chunk at a time, so that a store instruction writes eight
                    // 64-byte runs (8 rows x 4 lanes x 16 bytes) instead of 16 bytes in each of 32 rows
                    float4 (*stg)[4] = sm->stg[set * 4 + q];
                    const int rr = lane >> 2, ch = lane & 3;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            stg[lane][j ^ ((lane >> 1) & 3)] =
                                make_float4(__uint_as_float(v[16 * h + 4 * j]), __uint_as_float(v[16 * h + 4 * j + 1]),
                                            __uint_as_float(v[16 * h + 4 * j + 2]), __uint_as_float(v[16 * h + 4 * j + 3]));
                        __syncwarp();
                        float *const base = P.partial + (long long)sp * P.split_stride + P.taps[t].koff + ch0 + 16 * h + ch * 4;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int r = i * 8 + rr;
                            const int orow = ot * 128 + q * 32 + r;
                            if (orow < P.Cout)
                                *reinterpret_cast<float4 *>(base + (long long)orow * P.K) = stg[r][ch ^ ((r >> 1) & 3)];
                        }
                        __syncwarp();
                    }
                } else if (o < P.Cout) {
                    {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (ch0 + j < P.Cin) dst[j] = __uint_as_float(v[j]);
                    }
                }
            }
            if (have) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->acc_empty);
                ++lu;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (sm->abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// dW = sum over the splits of their partial tiles, added in split order (deterministic).  A thread owns one
// output; the loads of eight splits are in flight before the first is added.
__global__ void __launch_bounds__(256)
dw_reduce_kernel(const float *__restrict__ partial, long long n, int splits, float *__restrict__ dW)
{
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        float s = 0.0f;
        int k = 0;
        for (; k + 8 <= splits; k += 8) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __ldg(partial + (long long)(k + j) * n + i);
#pragma unroll
            for (int j = 0; j < 8; ++j) s += v[j];
        }
        for (; k < splits; ++k) s += __ldg(partial + (long long)k * n + i);
        dW[i] = s;
    }
}

// The same sum for many splits of a small tile.  A warp owns 32 consecutive outputs; the eight warps of a
// block take the splits k = g, g + 8, g + 16, ... (each warp in increasing k, up to eight loads in flight) and
// warp 0 adds the eight sums in warp order: a fixed order of additions, the same on every run.  (One thread per
// output is bound by the latency of its chain of loads when the splits are many and the outputs few; with few
// splits and many outputs it is the faster form.)
__global__ void __launch_bounds__(256)
dw_reduce_many_kernel(const float *__restrict__ partial, long long n, int splits, float *__restrict__ dW)
{
    __shared__ float sums[8][32];
    const int ix = threadIdx.x & 31, g = threadIdx.x >> 5;
    for (long long base = (long long)blockIdx.x * 32; base < n; base += (long long)gridDim.x * 32) {
        const long long i = base + ix;
        float s = 0.0f;
        if (i < n) {
            for (int k = g; k < splits; k += 64) {
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int kk = k + 8 * j;
                    v[j] = kk < splits ? __ldg(partial + (long long)kk * n + i) : 0.0f;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) s += v[j];
            }
        }
        sums[g][ix] = s;
        __syncthreads();
        if (g == 0 && i < n) {
            float t = sums[0][ix];
#pragma unroll
            for (int w = 1; w < 8; ++w) t += sums[w][ix];
            dW[i] = t;
        }
        __syncthreads();
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn dw_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

struct DwPlan {
    DwParams P;
    long long Ho, Wo;
    size_t ws_bytes;
};

int dw_plan(const twn_conv_desc_t *d, int sm_count, DwPlan *plan)
{
    TWN_REQUIRE(d != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->B > 0 && d->H > 0 && d->W > 0 && d->Cin > 0 && d->Cout > 0 && d->kh > 0 && d->kw > 0 &&
                    d->stride_h > 0 && d->stride_w > 0 && d->stride_h <= 8 && d->stride_w <= 8 && d->pad_h >= 0 &&
                    d->pad_w >= 0 && d->kh * d->kw <= kDwMaxTaps, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->Cin % 8 == 0 && d->Cout % 8 == 0, TWN_ERR_MISALIGNED);
    DwParams &P = plan->P;
    memset(&P, 0, sizeof P);
    plan->Ho = (d->H + 2 * d->pad_h - d->kh) / d->stride_h + 1;
    plan->Wo = (d->W + 2 * d->pad_w - d->kw) / d->stride_w + 1;
    TWN_REQUIRE(plan->Ho > 0 && plan->Wo > 0, TWN_ERR_INVALID_ARG);
    P.n_otiles = (int)((d->Cout + 127) / 128);
    P.n_taps = d->kh * d->kw;
    P.cblocks = (int)((d->Cin + 63) / 64);
    P.n_colblocks = P.n_taps * P.cblocks;
    P.kw = d->kw;
    memset(P.mma_off, 0, sizeof P.mma_off);
    const bool row_ok = d->stride_h == 1 && d->stride_w == 1 && d->kw >= 2 && d->kw <= kDwMaxCb;
    const bool col_ok = d->stride_h == 1 && d->stride_w == 1 && d->kw == 1 && d->kh >= 2 && d->kh <= kDwMaxCb;
    // Pixel box of a k-block: kpix = BB x BH x BW, fewest tiles.  Row mode (see DwParams) needs a box at least 8
    // pixels wide (its extra columns are a halo in w only, so the box may span several images).  Two sizes: a copy of 128 rows moves its bytes almost twice as fast as one
    // of 64 (measured: 1.75 against 3.25 cycles per 128-byte row), so 128-pixel k-blocks are taken unless their
    // padding costs more than a fifth (small images).
    struct Box { long long tiles; int lgBW, lgBH; bool row; };
    auto best_box = [&](int kpix) {
        Box best = {-1, 0, 0, false};
        int lg = 0;
        while ((1 << lg) < kpix) ++lg;
        for (int pass = 0; pass < 2; ++pass) {          // first among the boxes row mode can use, then among all
            for (int a = 0; a <= lg; ++a)
                for (int b = 0; a + b <= lg; ++b) {
                    const int BW = 1 << a, BH = 1 << b, BB = kpix >> (a + b);
                    if (BW * d->stride_w > 256 || BH * d->stride_h > 256 || BB > 256) continue;
                    // column mode also wants the 16 pixels of an MMA inside one image of the box
                    const bool row = (row_ok && BW >= 8 && BW + d->kw - 1 <= 256) ||
                                     (col_ok && BW >= 8 && BW * BH >= 16 && BH + d->kh - 1 <= 256);
                    if (pass == 0 && !row) continue;
                    const long long tiles = ((plan->Wo + BW - 1) / BW) * ((plan->Ho + BH - 1) / BH) * ((d->B + BB - 1) / BB);
                    // among equally many tiles: wider rows, or in column mode taller boxes (fewer extra rows per pixel)
                    const bool nicer = (col_ok && row) ? b > best.lgBH : a > best.lgBW;
                    if (best.tiles < 0 || tiles < best.tiles || (tiles == best.tiles && nicer)) best = {tiles, a, b, row};
                }
            if (best.tiles >= 0) break;
        }
        return best;
    };
    const Box b64 = best_box(64), b128 = best_box(128);
    TWN_REQUIRE(b64.tiles > 0 && b64.tiles <= 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    // a box that row mode can use beats one it cannot (three copies per k-block instead of up to six)
    bool use128 = b128.tiles > 0 && b128.tiles * 2 * 5 <= b64.tiles * 6 && (b128.row || !b64.row);
    int BW = 0, BH = 0, BB = 0;
    for (int attempt = 0; attempt < 2; ++attempt) {
        const Box bx = use128 ? b128 : b64;
        P.kpix = use128 ? 128 : 64;
        P.n_mma = P.kpix / 16;
        P.blk_bytes = P.kpix * 128;
        P.lgBW = bx.lgBW; P.lgBH = bx.lgBH;
        BW = 1 << P.lgBW; BH = 1 << P.lgBH; BB = P.kpix >> (P.lgBW + P.lgBH);
        P.tw = (int)((plan->Wo + BW - 1) / BW);
        P.th = (int)((plan->Ho + BH - 1) / BH);
        P.tb = (int)((d->B + BB - 1) / BB);
        P.pix_tiles = (int)bx.tiles;
        P.n_groups = (P.n_colblocks + kDwMaxCb - 1) / kDwMaxCb;
        // a layer of at most 64 output channels has one block of dZ per stage: rows 64..127 of the MMA then read
        // whatever follows in the stage, into accumulator rows that are never stored
        P.x_off = (d->Cout > 64 ? 2 : 1) * P.blk_bytes;
        {
            const int nb_max = P.n_colblocks < kDwMaxCb ? P.n_colblocks : kDwMaxCb;
            P.stage_bytes = P.x_off + nb_max * P.blk_bytes;
        }
        P.row_mode = 0;
        P.kw = d->kw;
        P.tap_stride_bytes = 0;
        // row mode: stride 1, 2..4 taps per filter row, the tile at least 8 pixels wide
        if (bx.row && row_ok) {
            P.row_mode = 1;
            P.n_groups = d->kh * P.cblocks;
            const int pitch = BW + d->kw - 1;                 // pixels per row of the widened tile
            P.x_bytes = pitch * BH * BB * 128;       // rows of consecutive images follow each other: no halo in h
            P.k_group_bytes = BW == 8 ? pitch * 128 : 1024;   // second 8-pixel run of an MMA: next row, or same row
            P.tap_stride_bytes = 128;
            for (int i = 0; i < P.n_mma; ++i) {
                const int h = (16 * i) / BW, w = (16 * i) % BW;
                P.mma_off[i] = (h * pitch + w) * 128;
            }
            P.stage_bytes = P.x_off + ((P.x_bytes + 1023) & ~1023);
        } else if (bx.row) {
            P.row_mode = 2;
            P.kw = d->kh;                                     // taps of a unit
            P.n_groups = P.cblocks;
            const int rows = BH + d->kh - 1;                  // rows per image of the heightened tile
            P.x_bytes = BW * rows * BB * 128;
            P.k_group_bytes = 1024;                           // second 8-pixel run: same row, or the next row of the image
            P.tap_stride_bytes = BW * 128;
            for (int i = 0; i < P.n_mma; ++i) {
                const int w = (16 * i) % BW, h = ((16 * i) / BW) % BH, b = (16 * i) / (BW * BH);
                P.mma_off[i] = ((b * rows + h) * BW + w) * 128;
            }
            P.stage_bytes = P.x_off + ((P.x_bytes + 1023) & ~1023);
        }
        // the MMA reads two blocks of dZ whatever Cout is: the stage must hold that many bytes
        if (P.stage_bytes < 2 * P.blk_bytes) P.stage_bytes = 2 * P.blk_bytes;
        P.stages = kDwPoolBytes / P.stage_bytes;
        if (P.stages > kDwMaxStages) P.stages = kDwMaxStages;
        // the two issuing threads take alternate stages of the ring: an even count
        P.stages &= ~1;
        // large k-blocks only with a ring of at least four of them
        if (!use128 || P.stages >= 4) break;
        use128 = false;
    }
    TWN_REQUIRE(P.stages >= 2, TWN_ERR_INVALID_ARG);
    const long long units = (long long)P.n_otiles * P.n_groups;
    // as many splits as keep the unit count within two full rounds of the grid (never a third,
    // nearly empty round)
    long long splits = (1LL * sm_count) / units;
    if (splits > P.pix_tiles) splits = P.pix_tiles;
    if (splits < 1) splits = 1;
    P.tiles_per_split = (int)((P.pix_tiles + splits - 1) / splits);
    splits = (P.pix_tiles + P.tiles_per_split - 1) / P.tiles_per_split;
    P.splits = (int)splits;
    TWN_REQUIRE(units * splits <= 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    P.total_units = (int)(units * splits);
    P.sw = d->stride_w; P.sh = d->stride_h;
    P.Cout = (int)d->Cout; P.Cin = (int)d->Cin;
    P.K = (long long)P.n_taps * d->Cin;
    P.split_stride = d->Cout * P.K;
    P.vec_ok = (d->Cin % 4 == 0) ? 1 : 0;
    for (int r = 0; r < d->kh; ++r)
        for (int s = 0; s < d->kw; ++s) {
            DwTap &t = P.taps[r * d->kw + s];
            t.dh = (int16_t)(r - d->pad_h);
            t.dw = (int16_t)(s - d->pad_w);
            t.koff = (int32_t)((r * d->kw + s) * d->Cin);
        }
    plan->ws_bytes = (size_t)P.splits * (size_t)P.split_stride * sizeof(float);
    return TWN_OK;
}

}  // namespace

extern "C" size_t twn_conv2d_bwd_weight_workspace_bytes(const twn_conv_desc_t *d)
{
    DwPlan plan;
    // the split count depends on the SM count; size for the largest part in use (148 SMs)
    int sms = 148;
    twn_device_info dev;
    if (twn_current_device(&dev) == TWN_OK) sms = dev.sm_count;
    if (dw_plan(d, sms, &plan) != TWN_OK) return 0;
    return plan.ws_bytes;
}

namespace {

// dW of layer `d`.  The activation tensor may be laid out with its own pitches (elements between
// pixels, rows and images; 0 = dense NHWC), which is how the folded first layer presents windows
// of four 16-channel pixels as 64-channel pixels.
int dw_run(const twn_conv_desc_t *d, const void *X, long long x_pix, long long x_row, long long x_img,
           const void *dZ, float *dW, void *workspace, size_t workspace_bytes, int32_t *dev_status,
           twn_stream_t stream)
{
    TWN_REQUIRE(X && dZ && dW && workspace, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    DwPlan plan;
    rc = dw_plan(d, dev.sm_count, &plan);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(workspace_bytes >= plan.ws_bytes, TWN_ERR_WORKSPACE);
    TWN_REQUIRE(twn_aligned(X, 16) && twn_aligned(dZ, 16) && twn_aligned(dW, 16) && twn_aligned(workspace, 16) &&
                    twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    EncodeTiledFn enc = dw_encode_fn();
    if (!enc) return TWN_ERR_CUDA;
    DwParams &P = plan.P;
    // a single split needs no reduction: its tile is the result
    P.partial = P.splits == 1 ? dW : static_cast<float *>(workspace);
    P.status = dev_status;
    const int BW = 1 << P.lgBW, BH = 1 << P.lgBH, BB = P.kpix >> (P.lgBW + P.lgBH);

    CUtensorMap map_dz, map_x;
    {
        cuuint64_t dims[4] = {(cuuint64_t)d->Cout, (cuuint64_t)plan.Wo, (cuuint64_t)plan.Ho, (cuuint64_t)d->B};
        cuuint64_t strides[3] = {(cuuint64_t)d->Cout * 2, (cuuint64_t)plan.Wo * d->Cout * 2,
                                 (cuuint64_t)plan.Ho * plan.Wo * d->Cout * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)BW, (cuuint32_t)BH, (cuuint32_t)BB};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(&map_dz, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(dZ), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TWN_ERR_INVALID_ARG;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)d->Cin, (cuuint64_t)d->W, (cuuint64_t)d->H, (cuuint64_t)d->B};
        const long long pixp = x_pix ? x_pix : d->Cin, rowp = x_row ? x_row : d->W * pixp, imgp = x_img ? x_img : d->H * rowp;
        cuuint64_t strides[3] = {(cuuint64_t)pixp * 2, (cuuint64_t)rowp * 2, (cuuint64_t)imgp * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)(BW * d->stride_w), (cuuint32_t)(BH * d->stride_h), (cuuint32_t)BB};
        if (P.row_mode == 1) box[1] = (cuuint32_t)(BW + d->kw - 1);
        if (P.row_mode == 2) box[2] = (cuuint32_t)(BH + d->kh - 1);
        cuuint32_t estr[4] = {1, (cuuint32_t)d->stride_w, (cuuint32_t)d->stride_h, 1};
        if (enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(X), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TWN_ERR_INVALID_ARG;
    }
    static bool attr_set[64] = {false};
    const int smem_bytes = (int)sizeof(DwSmem) + 1024;
    if (!attr_set[dev.ordinal]) {
        TWN_CUDA_OK(cudaFuncSetAttribute(dw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        attr_set[dev.ordinal] = true;
    }
    cudaStream_t s = twn_cu(stream);
    const int grid = dev.sm_count < P.total_units ? dev.sm_count : P.total_units;
    dw_kernel<<<grid, kDwThreads, smem_bytes, s>>>(map_dz, map_x, P);
    const long long n = P.split_stride;
    if (P.splits >= 40) {
        long long rb = (n + 31) / 32;
        if (rb > dev.sm_count * 8) rb = dev.sm_count * 8;
        dw_reduce_many_kernel<<<(int)rb, 256, 0, s>>>(P.partial, n, P.splits, dW);
    } else if (P.splits > 1) {
        long long rb = (n + 255) / 256;
        if (rb > dev.sm_count * 8) rb = dev.sm_count * 8;
        dw_reduce_kernel<<<(int)rb, 256, 0, s>>>(P.partial, n, P.splits, dW);
    }
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

// dW[o][r][s][c]  <-  folded gradient dWf[o][(r/2)*64 + (s/2)*16 + ((r%2)*2 + s%2)*Cin + c]
__global__ void __launch_bounds__(256)
dw_unfold_kernel(const float *__restrict__ dWf, int Cout, int kh, int kw, int Cin, int ldf, float *__restrict__ dW)
{
    const int K = kh * kw * Cin, total = Cout * K;
    for (int i = blockIdx.x * 256 + threadIdx.x; i < total; i += gridDim.x * 256) {
        const int o = i / K, k = i - o * K;
        const int t = k / Cin, c = k - t * Cin, r = t / kw, sx = t - r * kw;
        dW[i] = dWf[(size_t)o * ldf + (r >> 1) * 64 + (sx >> 1) * 16 + ((r & 1) * 2 + (sx & 1)) * Cin + c];
    }
}

// the stride-1 layer that the folded tensors describe: ceil(kh/2) x 1 taps on 64 "channels"
int folded_desc(const twn_conv_desc_t *d, twn_conv_desc_t *f, int64_t *Hf, int64_t *Wf, int64_t *ldf)
{
    const int rc = twn_fold_dims(d, Hf, Wf, ldf);
    if (rc != TWN_OK) return rc;
    *f = *d;
    f->H = *Hf; f->W = *Wf - 3; f->Cin = 64;
    f->kh = (int)(*ldf / 64); f->kw = 1;
    f->stride_h = f->stride_w = 1;
    f->pad_h = f->pad_w = 0;
    return TWN_OK;
}

}  // namespace

extern "C" int twn_conv2d_bwd_weight(const twn_conv_desc_t *d, const void *X, const void *dZ, float *dW,
                                     void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                     twn_stream_t stream)
{
    return dw_run(d, X, 0, 0, 0, dZ, dW, workspace, workspace_bytes, dev_status, stream);
}

extern "C" size_t twn_conv2d_bwd_weight_folded_workspace_bytes(const twn_conv_desc_t *d)
{
    twn_conv_desc_t f;
    int64_t Hf, Wf, ldf;
    if (folded_desc(d, &f, &Hf, &Wf, &ldf) != TWN_OK) return 0;
    const size_t inner = twn_conv2d_bwd_weight_workspace_bytes(&f);
    if (inner == 0) return 0;
    // the folded gradient [Cout][ldf] first (256-byte multiple), then the partial sums
    return (((size_t)d->Cout * (size_t)ldf * sizeof(float) + 255) & ~(size_t)255) + inner;
}

extern "C" int twn_conv2d_bwd_weight_folded(const twn_conv_desc_t *d, const void *Xf, const void *dZ, float *dW,
                                            void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                            twn_stream_t stream)
{
    twn_conv_desc_t f;
    int64_t Hf, Wf, ldf;
    int rc = folded_desc(d, &f, &Hf, &Wf, &ldf);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(Xf && dZ && dW && workspace, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(workspace, 16) && twn_aligned(dW, 4), TWN_ERR_MISALIGNED);
    const size_t head = ((size_t)d->Cout * (size_t)ldf * sizeof(float) + 255) & ~(size_t)255;
    TWN_REQUIRE(workspace_bytes >= twn_conv2d_bwd_weight_folded_workspace_bytes(d) && workspace_bytes > head,
                TWN_ERR_WORKSPACE);
    TWN_REQUIRE(d->Cout * (long long)d->kh * d->kw * d->Cin < 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    float *dWf = static_cast<float *>(workspace);
    rc = dw_run(&f, Xf, 16, Wf * 16, Hf * Wf * 16, dZ, dWf, static_cast<char *>(workspace) + head,
                workspace_bytes - head, dev_status, stream);
    if (rc != TWN_OK) return rc;
    const int total = (int)(d->Cout * d->kh * d->kw * d->Cin);
    dw_unfold_kernel<<<(total + 255) / 256, 256, 0, twn_cu(stream)>>>(dWf, (int)d->Cout, d->kh, d->kw, (int)d->Cin,
                                                                     (int)ldf, dW);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

