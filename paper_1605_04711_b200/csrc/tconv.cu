// Ternary-weight contraction on the 5th-generation tensor cores (Eq. 2 forward block;
// Algorithm 1 TernaryForward / TernaryBackward):  Y = epilogue(alpha * X (*) T).
//
// One persistent, warp-specialised kernel serves the inner product, the convolution
// forward pass and the backward-for-data pass.  All three are written as a sum over
// "taps": for output pixel p and output channel n
//     acc[n, p] = sum_t sum_c  T[n, koff_t + c] * X[pixel(p) * stride + (dh_t, dw_t), c]
// with X an NHWC bf16 tensor addressed through a 4-D TMA tensor map (out-of-range
// pixels and channels read as zero) and T the packed 2-bit codes, one row per n.
//
// The weights are the A operand of tcgen05.mma and live in tensor memory: decode
// warps turn the packed codes into exact bf16 {-1, 0, +1} in registers and write them
// with tcgen05.st.  The activations are the B operand, staged by TMA into 128-byte
// swizzled shared memory.  The accumulator (fp32, tensor memory) therefore holds
// D[n, p]: a lane is an output channel, a column a pixel.  In the epilogue each thread
// owns one channel, so alpha, the per-channel affine and ReLU cost one register each,
// and a warp's store of one pixel covers 32 consecutive channels (128 contiguous bytes).
//
//   warp 0            TMA producer: one activation tile per k-block
//   warp 1            allocates tensor memory, issues tcgen05.mma, commits to mbarriers
//   warps 2-5 (2-9)   decode: packed codes (global, L2) -> bf16 pairs -> tensor memory; one group
//                     of four warps (one per lane quadrant), or two groups that take the stages
//                     in turn (template parameter DS)
//   last eight warps  epilogue, two per lane quadrant: tensor memory -> registers -> per-warp
//                     staging buffer -> TMA store
//
// Three tile shapes (template parameter PIX = pixels per tile; the channel tile is always 128).
// Measured on B200: one thread can issue a tcgen05.mma about every 50-90 cycles whatever its
// size, and waits or commits between MMAs are not hidden unless the MMA itself is long.  A
// 128x256x16 MMA (128 cycles) hides that; a 128x128x16 one (64 cycles) does not.
//   PIX = 256: one accumulator (256 of the 512 tensor-memory columns, the rest holds decoded
//              weights), five stages; the epilogue of a tile is not overlapped with the next
//              tile's MMAs.  Long reductions with many tiles.
//   PIX = 192: two accumulators and four stages fill the tensor memory exactly; the epilogue
//              overlaps the next tile.
//   PIX = 128: two accumulators, four stages of two k-blocks each.  Small problems.
// The host picks the shape and the number of decode groups per launch with a cost model.
//
// Every wait on an mbarrier is bounded (about a second); on expiry the kernel records
// TWN_ERR_TIMEOUT, all roles leave their loops, tensor memory is freed and the grid exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstddef>

#include <mutex>

#include "common.cuh"
#include "tc_ptx.cuh"
#include "tconv_host.cuh"

using namespace twn_detail;


namespace {

constexpr int kChan = 128;          // output channels per tile (UMMA M)
constexpr int kBlockK = 64;         // reduction elements per k-block (128 bytes of bf16)
// Groups of 4 decode warps in a block (template parameter DS): one, or two that take the stages in turn.
// Two pay where decoding paces an overlapped tile shape on a long reduction; elsewhere the four extra
// warps cost speed (they cap the block at 112 registers), so each variant is a kernel of its own.
__host__ __device__ constexpr int first_epi_warp(int ds) { return 2 + 4 * ds; }
constexpr int kEpiSets = 2;         // epilogue warps per lane quadrant; each drains every other 32-pixel chunk
__host__ __device__ constexpr int threads_conv(int ds) { return 32 * (first_epi_warp(ds) + 4 * kEpiSets); }
constexpr int kEpiWarps = 4 * kEpiSets;
constexpr int kStageBytes = 2048;   // one output staging buffer of a warp: 32 channels x 32 pixels of bf16 or 16 pixels of fp32
constexpr int kWordTab = 128;       // k-blocks per tile whose code offsets are tabulated in shared memory
constexpr int kAColsPerBlock = kBlockK / 2;    // 32 columns of bf16 pairs per k-block
constexpr uint32_t kTmemCols = 512;

template <int PIX> struct Cfg;
template <> struct Cfg<128> {
    static constexpr int kStages = 4;   // operand ring depth (shared and tensor memory)
    static constexpr int kSub = 2;      // k-blocks per stage: one wait and one commit per 8 MMAs
    static constexpr int kAccBufs = 2;  // the epilogue of a tile overlaps the MMAs of the next
    static constexpr int kOutBufs = 4;  // output staging buffers per epilogue warp
};
template <> struct Cfg<256> {
    static constexpr int kStages = 5;
    static constexpr int kSub = 1;
    static constexpr int kAccBufs = 1;
    static constexpr int kOutBufs = 2;
};
// 192 pixels: the largest tile that leaves room for two accumulators beside four stages of
// decoded weights (2 x 192 + 4 x 32 = 512 columns); the pixel tile is 3 * 2^k images deep.
template <> struct Cfg<192> {
    static constexpr int kStages = 4;
    static constexpr int kSub = 1;
    static constexpr int kAccBufs = 2;
    static constexpr int kOutBufs = 4;
};

struct ConvParams {
    // tiles
    int n_tiles, tw, th, tb, total_tiles;
    int lgBW, lgBH;               // pixel tile = BB x BH x BW, powers of two, product PIX
    // reduction
    int n_taps, n_cblk;           // k-blocks per tile = n_taps * n_cblk
    int codes_aligned;            // 1: every k-block starts on a 16-byte boundary of the packed row
    const uint32_t *T;            // packed codes, one row of `wpr` words per output channel
    long long wpr;
    int sw, sh;                   // input pixel = output pixel * (sh, sw) + (dh, dw)
    // virtual output grid and its embedding in the output tensor
    int Bv, Hv, Wv;
    int OH, OW, osh, osw, ooh, oow;
    long long ldy;                // output pixel pitch in elements
    int Cout;
    // epilogue
    const double *alpha;          // device scalar (twn_stats_t::alpha) or nullptr for 1
    const float *scale, *shift;
    const void *residual;
    int res_dtype, relu, out_dtype;
    int res_gate;                 // 0: the residual is added; 1: it gates the result (kept where residual > 0)
    int dsets;                    // host only: decode groups of the kernel variant to launch
    void *Y;
    int32_t *status;
    // optional batch statistics: [tile][epilogue warp of the quadrant][128 channels][sum, sum of squares]
    float *bn_partial;
    // output path: 1 = each epilogue warp stages its 32 channels x 32 pixels in shared memory and
    // writes them with a TMA store (box = 32 channels x sbw x sbh x sbb pixels); 0 = per-thread stores
    int tma_store, lg_sbw, lg_sbh;
    int res_tma;                  // 1: the residual (bf16) is staged by per-warp TMA loads, two chunks deep
    Tap taps[kMaxTaps];
};

template <int PIX>
struct __align__(1024) SmemLayout {
    static constexpr int kStages = Cfg<PIX>::kStages, kSub = Cfg<PIX>::kSub;
    static constexpr int kXBytes = PIX * kBlockK * 2;
    uint8_t x[kStages][kSub][kXBytes];           // swizzled activation tiles
    // TMA and decode -> MMA: the activation tile has landed (one arrival with its byte count) and the
    // four decode warps have put the stage's weights into tensor memory (one arrival each).  One
    // barrier for both: every wait of the issuing warp is latency that the tensor core may sit out.
    unsigned long long full[kStages];
    unsigned long long empty[kStages];     // MMA commit -> TMA and decode: both operand slots are free
    unsigned long long acc_full[2];        // MMA commit -> epilogue
    unsigned long long acc_empty[2];       // epilogue -> MMA
    // per-warp output staging for TMA stores: [pixels][32 channels].  The stores of the epilogue
    // queue behind the producer's tile loads in the copy engine, so while the main loop of the next
    // tile runs a store takes long to release its buffer: the overlapped tile shapes keep four.
    alignas(128) uint8_t stage_out[kEpiWarps][Cfg<PIX>::kOutBufs][kStageBytes];
    alignas(128) __nv_bfloat16 stage_res[kEpiWarps][2][32 * 32];  // per-warp residual staging: [32 pixels][32 channels]
    unsigned long long res_full[kEpiWarps][2];
    uint32_t kword[kWordTab];              // first code word of k-block u in a packed row, u < kWordTab
    uint32_t tmem_base;
    volatile int abort_flag;
};

static_assert(offsetof(SmemLayout<128>, stage_res) % 128 == 0 && offsetof(SmemLayout<256>, stage_res) % 128 == 0 &&
                  offsetof(SmemLayout<192>, stage_res) % 128 == 0 && offsetof(SmemLayout<192>, stage_out) % 128 == 0 &&
                  sizeof(SmemLayout<256>) + 1024 <= 232448 && sizeof(SmemLayout<128>) + 1024 <= 232448 &&
                  sizeof(SmemLayout<192>) + 1024 <= 232448 &&
                  offsetof(SmemLayout<128>, stage_out) % 128 == 0 && offsetof(SmemLayout<256>, stage_out) % 128 == 0,
              "TMA and vector accesses need aligned shared-memory regions");

template <int PIX, int DS, int BITS>
__global__ void __launch_bounds__(threads_conv(DS), 1)
tconv_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
             const __grid_constant__ CUtensorMap map_r, const __grid_constant__ ConvParams P)
{
    using L = SmemLayout<PIX>;
    constexpr int kStages = Cfg<PIX>::kStages, kSub = Cfg<PIX>::kSub, kAccBufs = Cfg<PIX>::kAccBufs;
    constexpr int kOutBufs = Cfg<PIX>::kOutBufs;
    constexpr int kXBytes = L::kXBytes;
    constexpr int kAColsPerStage = kSub * kAColsPerBlock;
    constexpr int kCodesPerWord = 32 / BITS, kWordsPerBlock = kBlockK / kCodesPerWord;   // 16 and 4, or 32 and 2
    static_assert(kAccBufs * PIX + kStages * kAColsPerStage <= (int)kTmemCols, "tensor memory budget");
    

    pdl_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    L *sm = reinterpret_cast<L *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    volatile int *abort_flag = &sm->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kbpt = P.n_taps * P.n_cblk;               // k-blocks per tile
    const int spt = (kbpt + kSub - 1) / kSub;           // stages per tile (the last may hold fewer k-blocks)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm->full[s], 1 + 4);
            mbar_init(&sm->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm->acc_full[b], 1);
            mbar_init(&sm->acc_empty[b], kEpiWarps);
        }
        for (int b = 0; b < 2 * kEpiWarps; ++b) mbar_init(&sm->res_full[0][0] + b, 1);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // code-word offset of every k-block, in the order the k-blocks are consumed: taps outer,
    // channel blocks inner
    constexpr int kFirstEpiWarp = first_epi_warp(DS), kThreadsConv = threads_conv(DS);
    for (int u = threadIdx.x; u < kbpt && u < kWordTab; u += kThreadsConv) {
        const int t = u / P.n_cblk, cb = u - t * P.n_cblk;
        sm->kword[u] = (uint32_t)(P.taps[t].koff / kCodesPerWord) + cb * kWordsPerBlock;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // the set-up above touched no global memory; everything below may read what the previous kernel wrote
    pdl_wait();
    const uint32_t tmem = sm->tmem_base;
    const uint32_t tmem_acc = tmem;                       // kAccBufs x PIX columns
    const uint32_t tmem_a = tmem + kAccBufs * PIX;        // kStages x kAColsPerStage columns

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t block_bytes = kXBytes;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x) {
                int pt = tile / P.n_tiles;
                const int twi = pt % P.tw; pt /= P.tw;
                const int thi = pt % P.th;
                const int tbi = pt / P.th;
                const int w0 = (twi << P.lgBW) * P.sw;
                const int h0 = (thi << P.lgBH) * P.sh;
                const int b0 = tbi * (PIX >> (P.lgBW + P.lgBH));
                int t = 0, cb = 0;
                for (int st = 0; st < spt; ++st, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    const int nsb = (kbpt - st * kSub) < kSub ? (kbpt - st * kSub) : kSub;
                    if (!mbar_wait(&sm->empty[s], ph ^ 1u, abort_flag, P.status)) { ok = false; break; }
                    mbar_expect_tx(&sm->full[s], nsb * block_bytes);
                    for (int sb = 0; sb < nsb; ++sb) {
                        const Tap tap = P.taps[t];
                        tma_load_4d(sm->x[s][sb], &map_x, &sm->full[s], cb * kBlockK, w0 + tap.dw, h0 + tap.dh, b0);
                        if (++cb == P.n_cblk) { cb = 0; ++t; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (whole warp, converged)
        // One wait and one commit per stage, constant accumulate flags.  With no taps at all
        // (kbpt == 0) nothing is accumulated and the epilogue does not wait.
        if (kbpt > 0) {
            constexpr uint32_t idesc = make_idesc(kChan, PIX);
            const uint64_t bdesc0 = smem_desc_sw128(smem_u32(sm->x[0][0]));
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x, ++lt) {
                const int buf = lt % kAccBufs;
                const uint32_t aph = (lt / kAccBufs) & 1u;
                if (!mbar_wait_warp(&sm->acc_empty[buf], aph ^ 1u, abort_flag, P.status, 0)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_acc + buf * PIX;
                for (int st = 0; st < spt; ++st, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!mbar_wait_warp(&sm->full[s], ph, abort_flag, P.status, 0)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t bdesc = bdesc0 + (uint64_t)(s * ((kSub * kXBytes) >> 4));
                    const uint32_t a_tmem = tmem_a + s * kAColsPerStage;
                    if (st == 0) tc_mma_block<true>(d_tmem, a_tmem, bdesc, idesc);
                    else tc_mma_block<false>(d_tmem, a_tmem, bdesc, idesc);
                    if (kSub > 1 && kbpt - st * kSub > 1)
                        tc_mma_block<false>(d_tmem, a_tmem + kAColsPerBlock, bdesc + (kXBytes >> 4), idesc);
                    tc_commit(&sm->empty[s]);
                }
                if (ok) tc_commit(&sm->acc_full[buf]);
            }
        }
    } else if (warp < kFirstEpiWarp) {
        // ------------------------------------------------ decode: codes -> bf16 -> tensor memory
        // Two groups of four warps; a group handles every other stage.  Each thread owns one
        // channel row: it reads the row's 16 bytes of codes per k-block straight from global
        // memory (L2-resident, fetched two of its stages ahead), so decoding depends only on a
        // free tensor-memory slot, not on the activation pipeline.
        const int q = warp & 3;                 // tensor-memory lane quadrant of this warp
        const int set = (warp - 2) >> 2;
        constexpr int dsets = DS;               // groups of this kernel; the loops below are stepped by it
        const int row = q * 32 + lane;          // channel row inside the tile
        const uint32_t lane_base = tmem_a + ((uint32_t)(q * 32) << 16);

        // Code words are fetched with explicit non-coherent loads straight into the registers that
        // hold them until they are decoded, from addresses clamped into the packed matrix: no
        // branch and no register copy stands between a load and its use, so its latency stays
        // hidden.  What a clamped fetch returns is either never decoded (no such stage) or feeds
        // channels that are never stored, or multiplies activations that the TMA zero-fills.
        struct Codes { uint4 v[kSub]; };
        auto fetch = [&](Codes &c, const uint32_t *rowp, int st) {
#pragma unroll
            for (int sb = 0; sb < kSub; ++sb) {
                int u = st * kSub + sb;
                u = u < kbpt ? u : kbpt - 1;
                long long word;
                if (kbpt <= kWordTab) {
                    word = sm->kword[u];
                } else {
                    const int t = u / P.n_cblk, cb = u - t * P.n_cblk;
                    word = (P.taps[t].koff / kCodesPerWord) + cb * kWordsPerBlock;
                }
                if (BITS == 2) {
                    if (P.codes_aligned) {
                        ld_nc_v4(c.v[sb], rowp + word);
                    } else {
                        const long long last = P.wpr - 1;
                        ld_nc_u32(c.v[sb].x, rowp + (word + 0 < last ? word + 0 : last));
                        ld_nc_u32(c.v[sb].y, rowp + (word + 1 < last ? word + 1 : last));
                        ld_nc_u32(c.v[sb].z, rowp + (word + 2 < last ? word + 2 : last));
                        ld_nc_u32(c.v[sb].w, rowp + (word + 3 < last ? word + 3 : last));
                    }
                } else {
                    if (P.codes_aligned) {
                        ld_nc_v2(c.v[sb].x, c.v[sb].y, rowp + word);
                    } else {
                        const long long last = P.wpr - 1;
                        ld_nc_u32(c.v[sb].x, rowp + (word + 0 < last ? word + 0 : last));
                        ld_nc_u32(c.v[sb].y, rowp + (word + 1 < last ? word + 1 : last));
                    }
                }
            }
        };
        // position of this group's next stages: (tile, st), advanced dsets stages at a time
        auto advance = [&](int &tile, int &st, int steps) {
            for (int i = 0; i < steps; ++i)
                if (++st >= spt) { st = 0; tile += gridDim.x; }
        };
        // the fetch position also carries its row of the packed matrix: the channel tile of
        // `tile` is tile mod n_tiles, stepped without a division (one sits in the way of every
        // stage otherwise); rows past Cout read the last row and are never stored
        const int nt_step = (int)(gridDim.x % (unsigned)P.n_tiles);
        auto row_ptr = [&](int nt) -> const uint32_t * {
            long long n = (long long)nt * kChan + row;
            n = n < P.Cout ? n : P.Cout - 1;
            return P.T + n * P.wpr;
        };
        auto advance_f = [&](int &tile, int &st, int &nt, const uint32_t *&rowp, int steps) {
            for (int i = 0; i < steps; ++i)
                if (++st >= spt) {
                    st = 0; tile += gridDim.x;
                    nt += nt_step; if (nt >= P.n_tiles) nt -= P.n_tiles;
                    rowp = row_ptr(nt);
                }
        };
        if (spt > 0) {
            // 256-pixel tiles: three code buffers in rotation, each refilled right after use for the
            // stage three of this group's stages ahead: no register is copied while its load is still
            // in flight.  The other shapes: two buffers, see below.
            int tile_c = blockIdx.x, st_c = 0;               // the stage being decoded
            advance(tile_c, st_c, set);
            int tile_f = tile_c, st_f = st_c;                // the stage being fetched
            int nt_f = tile_f % P.n_tiles;
            const uint32_t *rowp_f = row_ptr(nt_f);
            Codes c0, c1, c2;
            fetch(c0, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets);
            fetch(c1, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets);
            if (PIX == 256) { fetch(c2, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets); }
            uint32_t it = set;
            auto decode_stage = [&](const Codes &cur) -> bool {
                const int s = it % kStages;
                const uint32_t ph = (it / kStages) & 1u;
                const int nsb = (kbpt - st_c * kSub) < kSub ? (kbpt - st_c * kSub) : kSub;
                // the MMAs that read this slot's previous contents have completed
                if (!mbar_wait_warp(&sm->empty[s], ph ^ 1u, abort_flag, P.status, 32)) return false;
                tc_fence_after();
#pragma unroll
                for (int sb = 0; sb < kSub; ++sb) {
                    if (sb < nsb) {
                        const uint32_t wv[4] = {cur.v[sb].x, cur.v[sb].y, cur.v[sb].z, cur.v[sb].w};
                        uint32_t out[32];
                        decode_kblock<BITS>(wv, out);
                        tmem_st32(lane_base + s * kAColsPerStage + sb * kAColsPerBlock, out);
                    }
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->full[s]);
                advance(tile_c, st_c, dsets);
                it += dsets;
                return true;
            };
            if (PIX == 256) {
                // long reductions, no slack for a late code word: three buffers in rotation
                while (true) {
                    if (tile_c >= P.total_tiles || !decode_stage(c0)) break;
                    { fetch(c0, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets); }
                    if (tile_c >= P.total_tiles || !decode_stage(c1)) break;
                    { fetch(c1, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets); }
                    if (tile_c >= P.total_tiles || !decode_stage(c2)) break;
                    { fetch(c2, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets); }
                }
            } else {
                // The overlapped tile shapes are paced by this loop, and a loop that is a third as long
                // gains more than it loses by fetching only two stages ahead and moving the code words
                // one buffer down per stage (measured: 128-pixel tiles 6-20 % faster, 192-pixel tiles
                // unchanged).
#pragma unroll 1
                while (true) {
                    if (tile_c >= P.total_tiles || !decode_stage(c0)) break;
                    c0 = c1;
                    { fetch(c1, rowp_f, st_f); advance_f(tile_f, st_f, nt_f, rowp_f, dsets); }
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue
        // Eight warps, two per tensor-memory lane quadrant; the two warps of a quadrant take
        // alternate 32-pixel chunks of the accumulator.  Every warp works on its own: it drains
        // its 32 channels x 32 pixels with tcgen05.ld (the load of its next chunk is in flight
        // while the current one is processed), applies scale / shift / residual / ReLU, stages
        // the chunk in its own shared-memory buffer and writes it with its own TMA store
        // (box = 32 channels x 32 pixels).  No barrier joins the epilogue warps, so a warp never
        // waits for a slower one, and the accumulator goes back to the MMA warp as soon as the
        // last tensor-memory load of every warp has completed.
        const int q = warp & 3;
        const int es = (warp - kFirstEpiWarp) >> 2;          // which of the two warps of the quadrant
        const int ewi = warp - kFirstEpiWarp;                // buffer set of this warp
        // decoded ternary weights are +-2, so half of alpha scales the accumulators
        const float alpha = (P.alpha ? (float)(*P.alpha) : 1.0f) * (1.0f / decoded_unit<BITS>());
        const int BWm = (1 << P.lgBW) - 1, BHm = (1 << P.lgBH) - 1;
        const bool out_bf16 = P.out_dtype == TWN_BF16, res_bf16 = P.res_dtype == TWN_BF16;
        const bool need_off = !P.tma_store || (P.residual && !P.res_tma);
        // the ReLU of a bf16 output rides on the conversion (a NaN stays a NaN); every other path clamps explicitly
        const bool relu_in_cvt = P.relu && out_bf16 && P.tma_store;
        const bool relu_here = P.relu && !relu_in_cvt;
        constexpr int kChunks = PIX / 32;
        constexpr int kMine = kChunks / kEpiSets;            // chunks of a tile this warp drains
        static_assert(kChunks % kEpiSets == 0, "the chunks of a tile are split evenly over the warps of a quadrant");
        uint8_t *const my_out = sm->stage_out[ewi][0];
        __nv_bfloat16 *const my_res = sm->stage_res[ewi][0];
        unsigned long long *const my_res_full = sm->res_full[ewi];
        uint32_t lt = 0;
        uint32_t nst = 0;      // staging buffers this warp has filled so far (selects the buffer)
        uint32_t nres = 0;     // residual chunks this warp has consumed so far (buffer and phase)
        bool alive = true;
        for (int tile = blockIdx.x; tile < P.total_tiles && alive; tile += gridDim.x, ++lt) {
            const int nt = tile % P.n_tiles;
            int pt = tile / P.n_tiles;
            const int twi = pt % P.tw; pt /= P.tw;
            const int thi = pt % P.th;
            const int tbi = pt / P.th;
            const int n = nt * kChan + q * 32 + lane;
            const bool n_ok = n < P.Cout;
            // a warp whose 32 channels all lie past Cout hands the accumulator back but loads,
            // computes and stores nothing
            const bool warp_on = nt * kChan + q * 32 < P.Cout;
            const float sc = ((P.scale && n_ok) ? __ldg(P.scale + n) : 1.0f) * alpha;
            const float sf = (P.shift && n_ok) ? __ldg(P.shift + n) : 0.0f;
            const int p_w0 = twi << P.lgBW, p_h0 = thi << P.lgBH, p_b0 = tbi * (PIX >> (P.lgBW + P.lgBH));
            const int c_n0 = nt * kChan + q * 32;            // first channel of this warp
            // residual chunk `c` of this tile -> buffer `slot` of this warp (one lane)
            auto res_load = [&](int c, uint32_t slot) {
                const int p0 = c * 32;
                mbar_expect_tx(&my_res_full[slot], 32 * 32 * 2);
                tma_load_4d(my_res + slot * (32 * 32), &map_r, &my_res_full[slot], c_n0,
                            (p_w0 + (p0 & BWm)) * P.osw, (p_h0 + ((p0 >> P.lgBW) & BHm)) * P.osh,
                            p_b0 + (p0 >> (P.lgBW + P.lgBH)));
            };
            // both buffers are free here: the warp has read the last chunk of its previous tile
            const bool use_res_tma = P.res_tma && warp_on;
            if (use_res_tma && lane == 0) {
                res_load(es, nres & 1u);
                if (kMine > 1) res_load(es + kEpiSets, (nres + 1) & 1u);
            }
            const int buf = lt % kAccBufs;
            if (kbpt > 0 && !mbar_wait_warp(&sm->acc_full[buf], (lt / kAccBufs) & 1u, abort_flag, P.status, 32)) break;
            tc_fence_after();
            float *const y32 = reinterpret_cast<float *>(P.Y) + n;
            __nv_bfloat16 *const y16 = reinterpret_cast<__nv_bfloat16 *>(P.Y) + n;
            const uint32_t t_acc = tmem_acc + ((uint32_t)(q * 32) << 16) + buf * PIX;
            uint32_t v[32];
            float bn_s1 = 0.0f, bn_s2 = 0.0f;      // this thread's channel: sum and sum of squares over its pixels of the tile
            // the chunk loop stays rolled: the epilogue is straight-line code that every warp walks
            // once per chunk, so its size is instruction-fetch time
#pragma unroll 1
            for (int i = 0; i < kMine; ++i) {
                const int c = es + i * kEpiSets;
                if (kbpt > 0) {
                    if (warp_on) {
                        tmem_ld32(t_acc + c * 32, v);
                        tmem_wait_ld(v);
                    }
                    if (i + 1 == kMine) {
                        // this warp's share of the accumulator is in registers: hand it back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&sm->acc_empty[buf]);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (!warp_on) continue;
                // output offset of pixel `lane` of this chunk (per-thread stores and residual loads
                // exchange them by shuffle), ~0 = outside the output
                uint32_t my_off = 0xFFFFFFFFu;
                if (need_off) {
                    const int p = c * 32 + lane;
                    const int wv = p_w0 + (p & BWm);
                    const int hv = p_h0 + ((p >> P.lgBW) & BHm);
                    const int bv = p_b0 + (p >> (P.lgBW + P.lgBH));
                    if (wv < P.Wv && hv < P.Hv && bv < P.Bv)
                        my_off = (uint32_t)((((long long)bv * P.OH + (hv * P.osh + P.ooh)) * P.OW + (wv * P.osw + P.oow)) * P.ldy);
                }
                if (use_res_tma) {
                    if (!mbar_wait_warp(&my_res_full[nres & 1u], (nres >> 1) & 1u, abort_flag, P.status, 32)) { alive = false; break; }
                }
                if (P.bn_partial) {
                    // Batch statistics of z = acc * scale' + shift, the value before the residual and the ReLU,
                    // over the pixels that exist (a ragged tile computes on zero-filled pixels too).  Lane j
                    // decides for pixel j of the chunk, a vote makes the mask warp-wide.
                    const int p = c * 32 + lane;
                    const bool in_range = (p_w0 + (p & BWm)) < P.Wv && (p_h0 + ((p >> P.lgBW) & BHm)) < P.Hv &&
                                          (p_b0 + (p >> (P.lgBW + P.lgBH))) < P.Bv;
                    const uint32_t live = __ballot_sync(0xffffffffu, in_range);
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float z = fmaf(__uint_as_float(v[j]), sc, sf);
                        if ((live >> j) & 1u) { bn_s1 += z; bn_s2 = fmaf(z, z, bn_s2); }
                    }
                }
                // The inner loops are kept free of conditionals: every instruction issued here is
                // exposed latency of this warp's chunk.
                if (use_res_tma) {
                    const __nv_bfloat16 *rs = my_res + (nres & 1u) * (32 * 32) + lane;
                    if (P.res_gate) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float y = fmaf(__uint_as_float(v[j]), sc, sf);
                            v[j] = __float_as_uint(__bfloat162float(rs[j * 32]) > 0.0f ? y : 0.0f);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            v[j] = __float_as_uint(fmaf(__uint_as_float(v[j]), sc, sf) + __bfloat162float(rs[j * 32]));
                    }
                    // the buffer is free again: fetch the residual of the chunk after the next
                    __syncwarp();
                    if (lane == 0 && i + 2 < kMine) res_load(c + 2 * kEpiSets, nres & 1u);
                    ++nres;
                } else if (P.residual) {
                    // y = acc * scale' + shift + residual (residual fetched with the per-pixel offsets)
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const uint32_t o = __shfl_sync(0xffffffffu, my_off, j);
                        float r = 0.0f;
                        if (o != 0xFFFFFFFFu && n_ok)
                            r = res_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(P.residual)[(size_t)o + n])
                                         : reinterpret_cast<const float *>(P.residual)[(size_t)o + n];
                        const float y = fmaf(__uint_as_float(v[j]), sc, sf);
                        v[j] = __float_as_uint(P.res_gate ? (r > 0.0f ? y : 0.0f) : y + r);
                    }
                } else {
                    // two pixels per instruction
#pragma unroll
                    for (int j = 0; j < 32; j += 2) fma_f32x2(v[j], v[j + 1], sc, sc, sf, sf);
                }
                if (relu_here) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(fmaxf(__uint_as_float(v[j]), 0.0f));
                }
                if (P.tma_store) {
                    // a staging buffer holds 32 pixels of bf16 or 16 of fp32: one or two rounds per chunk
                    const int rounds = out_bf16 ? 1 : 2;
                    for (int h = 0; h < rounds; ++h) {
                        // the buffer was last read by the store this warp issued kOutBufs rounds ago
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kOutBufs - 1) : "memory");
                        __syncwarp();
                        uint8_t *const sbuf = my_out + (nst % kOutBufs) * kStageBytes;
                        if (out_bf16) {
                            uint16_t *const st16 = reinterpret_cast<uint16_t *>(sbuf) + lane;
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                // one packed conversion per two pixels
                                const uint32_t pk = relu_in_cvt ? pack_bf16x2_relu(__uint_as_float(v[j]), __uint_as_float(v[j + 1]))
                                                                : pack_bf16x2(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                                st16[j * 32] = (uint16_t)pk;
                                st16[(j + 1) * 32] = (uint16_t)(pk >> 16);
                            }
                        } else {
                            uint32_t *const st32 = reinterpret_cast<uint32_t *>(sbuf) + lane;
                            if (h == 0) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) st32[j * 32] = v[j];
                            } else {
#pragma unroll
                                for (int j = 0; j < 16; ++j) st32[j * 32] = v[16 + j];
                            }
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) {
                            const int p0 = c * 32 + h * 16;
                            tma_store_4d(&map_y, sbuf, c_n0, (p_w0 + (p0 & BWm)) * P.osw,
                                         (p_h0 + ((p0 >> P.lgBW) & BHm)) * P.osh, p_b0 + (p0 >> (P.lgBW + P.lgBH)));
                        }
                        ++nst;
                    }
                } else {
                    if (out_bf16) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const uint32_t o = __shfl_sync(0xffffffffu, my_off, j);
                            if (o != 0xFFFFFFFFu && n_ok) y16[o] = __float2bfloat16_rn(__uint_as_float(v[j]));
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const uint32_t o = __shfl_sync(0xffffffffu, my_off, j);
                            if (o != 0xFFFFFFFFu && n_ok) y32[o] = __uint_as_float(v[j]);
                        }
                    }
                }
            }
            if (P.bn_partial && warp_on)
                *reinterpret_cast<float2 *>(P.bn_partial + ((size_t)tile * kEpiSets + es) * (2 * kChan) + (q * 32 + lane) * 2) =
                    make_float2(bn_s1, bn_s2);
            __syncwarp();
        }
        // all bulk stores of this thread have been written before the block may exit
        if (P.tma_store && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (sm->abort_flag) {
        // give copies and MMAs still in flight time to land before the memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Totals of the per-tile statistics: one warp per channel, the lanes take the tiles in turn and a shuffle tree
// adds the 32 partial totals: a fixed order, so the result is the same bits on every run.
__global__ void __launch_bounds__(256)
bn_reduce_kernel(const float *__restrict__ partial, int total_tiles, int n_tiles, int Cout,
                 double *__restrict__ sum, double *__restrict__ sumsq)
{
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (c >= Cout) return;
    const int nt = c / kChan, within = c - nt * kChan;
    double s1 = 0.0, s2 = 0.0;
    for (int tile = nt + lane * n_tiles; tile < total_tiles; tile += 32 * n_tiles)
#pragma unroll
        for (int es = 0; es < kEpiSets; ++es) {
            const float2 v = __ldg(reinterpret_cast<const float2 *>(partial + ((size_t)tile * kEpiSets + es) * (2 * kChan) + within * 2));
            s1 += (double)v.x; s2 += (double)v.y;
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_down_sync(0xffffffffu, s1, o);
        s2 += __shfl_down_sync(0xffffffffu, s2, o);
    }
    if (lane == 0) { sum[c] = s1; sumsq[c] = s2; }
}

// ---------------------------------------------------------------- host side
template <int PIX, int DS, int BITS>
int launch_conv_t(const Geometry &g, ConvParams &P, const void *X, const twn_device_info &dev,
                  EncodeTiledFn enc, cudaStream_t s)
{
    static bool attr_set[64] = {false};
    const int smem_bytes = (int)sizeof(SmemLayout<PIX>) + 1024;
    if (!attr_set[dev.ordinal]) {
        TWN_CUDA_OK(cudaFuncSetAttribute(tconv_kernel<PIX, DS, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        attr_set[dev.ordinal] = true;
    }
    pick_tile(g, PIX, &P.lgBW, &P.lgBH);
    const int BW = 1 << P.lgBW, BH = 1 << P.lgBH, BB = PIX >> (P.lgBW + P.lgBH);
    P.tw = (g.Wv + BW - 1) / BW;
    P.th = (g.Hv + BH - 1) / BH;
    P.tb = (g.Bv + BB - 1) / BB;
    const long long total = (long long)P.n_tiles * P.tw * P.th * P.tb;
    if (total <= 0 || total > 0x7fffffffLL) return TWN_ERR_INVALID_ARG;
    P.total_tiles = (int)total;

    // activations: (C, W, H, B), 64-channel boxes with 128-byte swizzle, zero fill outside
    CUtensorMap map_x;
    {
        cuuint64_t dims[4] = {(cuuint64_t)g.XC, (cuuint64_t)g.XW, (cuuint64_t)g.XH, (cuuint64_t)g.XB};
        const long long rowp = g.x_row_pitch ? g.x_row_pitch : g.XW * g.ldx;
        const long long imgp = g.x_img_pitch ? g.x_img_pitch : g.XH * rowp;
        cuuint64_t strides[3] = {(cuuint64_t)g.ldx * 2, (cuuint64_t)rowp * 2, (cuuint64_t)imgp * 2};
        // with a traversal stride the box counts traversed elements: N loaded elements need N * stride
        cuuint32_t box[4] = {(cuuint32_t)kBlockK, (cuuint32_t)(BW * g.sw), (cuuint32_t)(BH * g.sh), (cuuint32_t)BB};
        cuuint32_t estr[4] = {1, (cuuint32_t)g.sw, (cuuint32_t)g.sh, 1};
        if (enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(X), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TWN_ERR_INVALID_ARG;
    }
    // output: TMA stores when the pitch allows it.  The virtual output grid may be embedded in
    // the tensor with a stride and an offset (backward for data of a strided layer): the map
    // then starts at the offset pixel and traverses with that stride.
    // (the channel extent must be a whole number of 16-byte units: the store clips at that granularity)
    CUtensorMap map_y = map_x, map_r = map_x;
    const int es = P.out_dtype == TWN_BF16 ? 2 : 4;
    P.tma_store = 0;
    P.res_tma = 0;
    const long long base_pix = (long long)g.ooh * g.OW + g.oow;
    if ((g.ldy * es) % 16 == 0 && ((long long)g.Cout * es) % 16 == 0 && (reinterpret_cast<uintptr_t>(P.Y) % 16) == 0 &&
        g.OW > g.oow && g.OH > g.ooh) {
        // 2^lg consecutive tile pixels are a sub-box sbw x sbh x sbb of the tile box, 32 channels wide
        // (one epilogue warp): a staging buffer holds 32 pixels of bf16 or 16 of fp32, a residual
        // buffer 32 pixels
        auto sub_box = [&](int lg, cuuint32_t *bx) {
            const int lg_sbw = P.lgBW < lg ? P.lgBW : lg;
            const int lg_sbh = P.lgBH < lg - lg_sbw ? P.lgBH : lg - lg_sbw;
            const int lg_sbb = lg - lg_sbw - lg_sbh;
            bx[0] = 32u; bx[1] = (cuuint32_t)((1 << lg_sbw) * g.osw);
            bx[2] = (cuuint32_t)((1 << lg_sbh) * g.osh); bx[3] = 1u << lg_sbb;
        };
        cuuint64_t dims[4] = {(cuuint64_t)g.Cout, (cuuint64_t)(g.OW - g.oow), (cuuint64_t)(g.OH - g.ooh), (cuuint64_t)g.Bv};
        cuuint32_t box[4], rbox[4];
        sub_box(es == 2 ? 5 : 4, box);
        sub_box(5, rbox);
        cuuint32_t estr[4] = {1, (cuuint32_t)g.osw, (cuuint32_t)g.osh, 1};
        if (box[1] <= 256 && box[2] <= 256 && rbox[1] <= 256 && rbox[2] <= 256) {
            cuuint64_t strides[3] = {(cuuint64_t)g.ldy * es, (cuuint64_t)g.OW * g.ldy * es, (cuuint64_t)g.OH * g.OW * g.ldy * es};
            void *ybase = static_cast<char *>(P.Y) + base_pix * g.ldy * es;
            if (enc(&map_y, es == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ybase, dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
                P.tma_store = 1;
            // a bf16 residual of the same geometry is staged the same way
            if (P.tma_store && P.residual && P.res_dtype == TWN_BF16 && (g.ldy * 2) % 16 == 0 &&
                ((long long)g.Cout * 2) % 16 == 0 && (reinterpret_cast<uintptr_t>(P.residual) % 16) == 0) {
                cuuint64_t rstrides[3] = {(cuuint64_t)g.ldy * 2, (cuuint64_t)g.OW * g.ldy * 2, (cuuint64_t)g.OH * g.OW * g.ldy * 2};
                void *rbase = const_cast<char *>(static_cast<const char *>(P.residual)) + base_pix * g.ldy * 2;
                if (enc(&map_r, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, rbase, dims, rstrides, rbox, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
                    P.res_tma = 1;
            }
        }
    }
    const int grid = dev.sm_count < P.total_tiles ? dev.sm_count : P.total_tiles;
    // Programmatic dependent launch pays when the blocks cover the GPU (set-up and launch latency hide behind the
    // previous kernel's last tiles); a launch of a few blocks measured slower with it (an inner product of 8 blocks
    // after a convolution: 21 us instead of 12), so those launch the plain way.
    const bool kPdlConv = grid * 2 >= dev.sm_count;
    if (P.bn_partial && (size_t)P.total_tiles * kEpiSets * 2 * kChan * sizeof(float) > g.bn_partial_bytes) return TWN_ERR_WORKSPACE;
    TWN_CUDA_OK(twn_launch_pdl(kPdlConv, tconv_kernel<PIX, DS, BITS>, grid, threads_conv(DS), (size_t)smem_bytes, s, map_x, map_y, map_r, P));
    if (P.bn_partial)
        bn_reduce_kernel<<<(g.Cout + 7) / 8, 256, 0, s>>>(P.bn_partial, P.total_tiles, P.n_tiles, g.Cout, g.bn_sum, g.bn_sumsq);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}

int launch_conv(const Geometry &g, const void *X, const uint32_t *T, const twn_stats_t *stats,
                const twn_epilogue_t *epi, void *Y, int out_dtype_default, int32_t *dev_status, cudaStream_t s)
{
    twn_device_info dev;
    int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TWN_ERR_CUDA;

    // the epilogue keeps output offsets in 32 bits
    if ((long long)g.Bv * g.OH * g.OW * g.ldy >= 0xFFFFFFFFLL) return TWN_ERR_INVALID_ARG;
    {
        // narrow layers: the kernel that decodes the layer's codes once per block
        EpilogueArgs ea;
        ea.alpha = stats ? &stats->alpha : nullptr;
        ea.scale = epi ? epi->scale : nullptr;
        ea.shift = epi ? epi->shift : nullptr;
        ea.residual = epi ? epi->residual : nullptr;
        ea.res_dtype = epi ? epi->residual_dtype : TWN_F32;
        ea.res_gate = (epi && epi->residual) ? epi->residual_op : 0;
        ea.relu = epi ? epi->relu : 0;
        ea.out_dtype = epi ? epi->out_dtype : out_dtype_default;
        bool handled = false;
        rc = launch_conv_resident(g, X, T, ea, Y, dev_status, dev, s, &handled);
        if (rc != TWN_OK || handled) return rc;
    }
    ConvParams P;
    memset(&P, 0, sizeof P);
    P.n_tiles = (g.Cout + kChan - 1) / kChan;
    P.n_taps = g.n_taps;
    P.n_cblk = (int)((g.Cin + kBlockK - 1) / kBlockK);
    P.codes_aligned = 1;
    for (int t = 0; t < g.n_taps; ++t)
        if (g.taps[t].koff % kBlockK != 0) P.codes_aligned = 0;
    P.T = T;
    P.wpr = g.ld_codes / (g.code_bits == 1 ? 32 : 16);
    P.sw = g.sw; P.sh = g.sh;
    P.Bv = g.Bv; P.Hv = g.Hv; P.Wv = g.Wv;
    P.OH = g.OH; P.OW = g.OW; P.osh = g.osh; P.osw = g.osw; P.ooh = g.ooh; P.oow = g.oow;
    P.ldy = g.ldy;
    P.Cout = g.Cout;
    P.alpha = stats ? &stats->alpha : nullptr;
    P.scale = epi ? epi->scale : nullptr;
    P.shift = epi ? epi->shift : nullptr;
    P.residual = epi ? epi->residual : nullptr;
    P.res_dtype = epi ? epi->residual_dtype : TWN_F32;
    P.res_gate = (epi && epi->residual) ? epi->residual_op : 0;
    P.relu = epi ? epi->relu : 0;
    P.out_dtype = epi ? epi->out_dtype : out_dtype_default;
    P.Y = Y;
    P.status = dev_status;
    P.bn_partial = g.bn_partial;
    for (int t = 0; t < g.n_taps; ++t) P.taps[t] = g.taps[t];

    // Tile shape by a cost model fitted to measured launches (cycles per round of tiles, kb = k-blocks
    // per tile):
    //   128 pixels: max(2000 + 680 kb, 6500), 540 kb with both decode groups: the epilogue overlaps
    //               the next tile and bounds short reductions
    //   192 pixels: max(2500 + 700 kb, 10500), 630 kb with both decode groups; floor 7600 when only the lower half of the channel
    //               tile exists: overlapped as well, fewer rounds than 128
    //   256 pixels: 8000 + 700 kb: one accumulator, so the epilogue is exposed; 7000 when only the
    //               lower half of the channel tile exists (half of the epilogue warps idle)
    int a, b;
    const long long kb = (long long)P.n_taps * P.n_cblk;
    const long long sms = dev.sm_count;
    const bool half = g.Cout <= kChan / 2;
    const long long t128 = pick_tile(g, 128, &a, &b) * P.n_tiles, t256 = pick_tile(g, 256, &a, &b) * P.n_tiles;
    const long long t192 = pick_tile(g, 192, &a, &b) * P.n_tiles;
    // a second decode group pays where decoding paces the overlapped shapes: long reductions
    const bool two = kb >= 18;
    const long long lin128 = two ? 2000 + 540 * kb : 2000 + 680 * kb;
    const long long per128 = lin128 > 6500 ? lin128 : 6500;
    const long long floor192 = half ? 7600 : 10500;
    const long long lin192 = two ? 2500 + 630 * kb : 2500 + 700 * kb;
    const long long per192 = lin192 > floor192 ? lin192 : floor192;
    const long long per256 = (half ? 7000 : 8000) + 700 * kb;
    const long long c128 = ((t128 + sms - 1) / sms) * per128, c192 = ((t192 + sms - 1) / sms) * per192,
                    c256 = ((t256 + sms - 1) / sms) * per256;
    int choice = c256 < c128 ? 1 : 0;
    if (c192 < (choice ? c256 : c128)) choice = 2;
    P.dsets = (choice != 1 && two) ? 2 : 1;
    if (g.code_bits == 1) {
        if (choice == 1) return launch_conv_t<256, 1, 1>(g, P, X, dev, enc, s);
        if (choice == 2) return P.dsets == 2 ? launch_conv_t<192, 2, 1>(g, P, X, dev, enc, s) : launch_conv_t<192, 1, 1>(g, P, X, dev, enc, s);
        return P.dsets == 2 ? launch_conv_t<128, 2, 1>(g, P, X, dev, enc, s) : launch_conv_t<128, 1, 1>(g, P, X, dev, enc, s);
    }
    if (choice == 1) return launch_conv_t<256, 1, 2>(g, P, X, dev, enc, s);
    if (choice == 2) return P.dsets == 2 ? launch_conv_t<192, 2, 2>(g, P, X, dev, enc, s) : launch_conv_t<192, 1, 2>(g, P, X, dev, enc, s);
    return P.dsets == 2 ? launch_conv_t<128, 2, 2>(g, P, X, dev, enc, s) : launch_conv_t<128, 1, 2>(g, P, X, dev, enc, s);
}

// Helper streams for launches that are independent of one another (the residue classes of a
// strided backward-for-data pass write disjoint pixels).  They fork from the caller's stream
// through an event and join it again the same way, so the caller sees one stream-ordered
// operation; under stream capture the fork and the join become graph edges.  Created once per
// device; a mutex keeps two host threads from interleaving their use of the shared events.
struct ForkPool {
    cudaStream_t side[3];
    cudaEvent_t fork, join[3];
    bool ready = false, failed = false;
};
std::mutex g_fork_mutex;

ForkPool *fork_pool(int ordinal)
{
    static ForkPool pools[64];
    ForkPool &p = pools[ordinal];
    if (p.failed) return nullptr;
    if (!p.ready) {
        bool ok = cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < 3 && ok; ++i)
            ok = cudaStreamCreateWithFlags(&p.side[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.join[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { p.failed = true; return nullptr; }
        p.ready = true;
    }
    return &p;
}

int check_epilogue(const twn_epilogue_t *e)
{
    if (!e) return TWN_OK;
    TWN_REQUIRE(e->out_dtype == TWN_F32 || e->out_dtype == TWN_BF16, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(e->residual_dtype == TWN_F32 || e->residual_dtype == TWN_BF16, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(e->relu == 0 || e->relu == 1, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(e->residual_op == TWN_RESIDUAL_ADD || e->residual_op == TWN_RESIDUAL_GATE, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(e->scale, 4) && twn_aligned(e->shift, 4) && twn_aligned(e->residual, 4), TWN_ERR_MISALIGNED);
    return TWN_OK;
}

}  // namespace

namespace {

// Shared by the ternary (bits = 2) and binary (bits = 1) entry points.
int gemm_impl(const void *X, int64_t ldx, const uint32_t *T_packed, int64_t ld_codes,
              const twn_stats_t *stats, int64_t M, int64_t N, int64_t K,
              const twn_epilogue_t *epi, void *Y, int64_t ldy, int32_t *dev_status,
              twn_stream_t stream, int bits)
{
    TWN_REQUIRE(M >= 0 && N >= 0 && K >= 0, TWN_ERR_INVALID_ARG);
    if (M == 0 || N == 0) return TWN_OK;
    TWN_REQUIRE(X && T_packed && Y && K > 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ldx >= K && ldy >= N && ld_codes >= K && ld_codes % (bits == 1 ? 128 : 64) == 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(M <= 0x7fffffffLL && N <= 0x7fffffffLL && K <= 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(ldx % 8 == 0, TWN_ERR_MISALIGNED);
    TWN_REQUIRE(twn_aligned(X, 16) && twn_aligned(T_packed, 16) && twn_aligned(Y, 4) && twn_aligned(stats, 8) &&
                    twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    int rc = check_epilogue(epi);
    if (rc != TWN_OK) return rc;
    Geometry g;
    memset(&g, 0, sizeof g);
    g.XB = 1; g.XH = 1; g.XW = M; g.XC = K; g.ldx = ldx;
    g.Bv = 1; g.Hv = 1; g.Wv = (int)M; g.OH = 1; g.OW = (int)M;
    g.osh = g.osw = 1; g.ooh = g.oow = 0; g.ldy = ldy;
    g.sh = g.sw = 1;
    g.Cout = (int)N; g.ld_codes = ld_codes; g.code_cols = K;
    g.n_taps = 1; g.taps[0] = Tap{0, 0, 0};
    g.Cin = K;
    g.code_bits = bits;
    return launch_conv(g, X, T_packed, stats, epi, Y, TWN_F32, dev_status, twn_cu(stream));
}

}  // namespace

extern "C" int twn_gemm(const void *X, int64_t ldx, const uint32_t *T_packed, int64_t ld_codes,
                        const twn_stats_t *stats, int64_t M, int64_t N, int64_t K,
                        const twn_epilogue_t *epi, void *Y, int64_t ldy, int32_t *dev_status,
                        twn_stream_t stream)
{
    return gemm_impl(X, ldx, T_packed, ld_codes, stats, M, N, K, epi, Y, ldy, dev_status, stream, 2);
}

extern "C" int twn_gemm_b1(const void *X, int64_t ldx, const uint32_t *B_packed, int64_t ld_codes,
                           const twn_stats_t *stats, int64_t M, int64_t N, int64_t K,
                           const twn_epilogue_t *epi, void *Y, int64_t ldy, int32_t *dev_status,
                           twn_stream_t stream)
{
    return gemm_impl(X, ldx, B_packed, ld_codes, stats, M, N, K, epi, Y, ldy, dev_status, stream, 1);
}

namespace {

int conv_common_checks(const twn_conv_desc_t *d)
{
    TWN_REQUIRE(d != nullptr, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->B > 0 && d->H > 0 && d->W > 0 && d->Cin > 0 && d->Cout > 0, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->kh > 0 && d->kw > 0 && d->stride_h > 0 && d->stride_w > 0 && d->pad_h >= 0 && d->pad_w >= 0,
                TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->stride_h <= 8 && d->stride_w <= 8, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->kh * d->kw <= kMaxTaps, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->H + 2 * d->pad_h >= d->kh && d->W + 2 * d->pad_w >= d->kw, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->B <= 0x7fffffffLL && d->H <= 0x7fffffffLL && d->W <= 0x7fffffffLL && d->Cin <= 0x7fffffffLL &&
                    d->Cout <= 0x7fffffffLL, TWN_ERR_INVALID_ARG);
    return TWN_OK;
}

}  // namespace

namespace {

struct BnArgs { double *sum, *sumsq; void *ws; size_t ws_bytes; };

int conv_fwd_impl(const twn_conv_desc_t *d, const void *X, const uint32_t *T_fwd, int64_t ld_codes,
                  const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                  int32_t *dev_status, twn_stream_t stream, int bits, const BnArgs *bn = nullptr)
{
    int rc = conv_common_checks(d);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(X && T_fwd && Y, TWN_ERR_INVALID_ARG);
    const long long taps = (long long)d->kh * d->kw;
    TWN_REQUIRE(ld_codes % (bits == 1 ? 128 : 64) == 0 && ld_codes >= taps * d->Cin, TWN_ERR_INVALID_ARG);
    // channel runs must start on 16-byte boundaries for TMA, tap columns on word boundaries
    TWN_REQUIRE(d->Cin % 8 == 0 && (taps == 1 || d->Cin % (bits == 1 ? 32 : 16) == 0), TWN_ERR_MISALIGNED);
    TWN_REQUIRE(twn_aligned(X, 16) && twn_aligned(T_fwd, 16) && twn_aligned(Y, 4) && twn_aligned(stats, 8) &&
                    twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    rc = check_epilogue(epi);
    if (rc != TWN_OK) return rc;
    const long long Ho = (d->H + 2 * d->pad_h - d->kh) / d->stride_h + 1;
    const long long Wo = (d->W + 2 * d->pad_w - d->kw) / d->stride_w + 1;
    Geometry g;
    memset(&g, 0, sizeof g);
    g.XB = d->B; g.XH = d->H; g.XW = d->W; g.XC = d->Cin; g.ldx = d->Cin;
    g.Bv = (int)d->B; g.Hv = (int)Ho; g.Wv = (int)Wo; g.OH = (int)Ho; g.OW = (int)Wo;
    g.osh = g.osw = 1; g.ooh = g.oow = 0; g.ldy = d->Cout;
    g.sh = d->stride_h; g.sw = d->stride_w;
    g.Cout = (int)d->Cout; g.ld_codes = ld_codes; g.code_cols = taps * d->Cin;
    g.Cin = d->Cin;
    for (int r = 0; r < d->kh; ++r)
        for (int s = 0; s < d->kw; ++s) {
            Tap &t = g.taps[g.n_taps++];
            t.dh = (int16_t)(r - d->pad_h);
            t.dw = (int16_t)(s - d->pad_w);
            t.koff = (int32_t)((r * d->kw + s) * d->Cin);
        }
    g.code_bits = bits;
    if (bn) {
        g.bn_partial = static_cast<float *>(bn->ws);
        g.bn_partial_bytes = bn->ws_bytes;
        g.bn_sum = bn->sum; g.bn_sumsq = bn->sumsq;
    }
    return launch_conv(g, X, T_fwd, stats, epi, Y, TWN_F32, dev_status, twn_cu(stream));
}

}  // namespace

extern "C" size_t twn_conv2d_fwd_bn_workspace_bytes(const twn_conv_desc_t *d)
{
    if (conv_common_checks(d) != TWN_OK) return 0;
    // the smallest pixel tile gives the most tiles: 128 pixels, whatever shape the launch then picks
    Geometry g;
    memset(&g, 0, sizeof g);
    g.Bv = (int)d->B;
    g.Hv = (int)((d->H + 2 * d->pad_h - d->kh) / d->stride_h + 1);
    g.Wv = (int)((d->W + 2 * d->pad_w - d->kw) / d->stride_w + 1);
    g.sh = d->stride_h; g.sw = d->stride_w;
    int a, b;
    const long long tiles = pick_tile(g, 128, &a, &b) * ((d->Cout + kChan - 1) / kChan);
    return (size_t)tiles * kEpiSets * 2 * kChan * sizeof(float);
}

extern "C" int twn_conv2d_fwd_bn(const twn_conv_desc_t *d, const void *X, const uint32_t *T_fwd, int64_t ld_codes,
                                 const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y, double *bn_sum,
                                 double *bn_sumsq, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                 twn_stream_t stream)
{
    TWN_REQUIRE(bn_sum && bn_sumsq && workspace, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(bn_sum, 8) && twn_aligned(bn_sumsq, 8) && twn_aligned(workspace, 16), TWN_ERR_MISALIGNED);
    TWN_REQUIRE(workspace_bytes >= twn_conv2d_fwd_bn_workspace_bytes(d) && workspace_bytes > 0, TWN_ERR_WORKSPACE);
    const BnArgs bn = {bn_sum, bn_sumsq, workspace, workspace_bytes};
    return conv_fwd_impl(d, X, T_fwd, ld_codes, stats, epi, Y, dev_status, stream, 2, &bn);
}

extern "C" int twn_conv2d_fwd(const twn_conv_desc_t *d, const void *X, const uint32_t *T_fwd, int64_t ld_codes,
                              const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                              int32_t *dev_status, twn_stream_t stream)
{
    return conv_fwd_impl(d, X, T_fwd, ld_codes, stats, epi, Y, dev_status, stream, 2);
}

extern "C" int twn_conv2d_fwd_b1(const twn_conv_desc_t *d, const void *X, const uint32_t *B_fwd, int64_t ld_codes,
                                 const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                                 int32_t *dev_status, twn_stream_t stream)
{
    return conv_fwd_impl(d, X, B_fwd, ld_codes, stats, epi, Y, dev_status, stream, 1);
}

extern "C" int twn_conv2d_fwd_folded(const twn_conv_desc_t *d, const void *Xf, const uint32_t *Tf, int64_t ld_folded,
                                     const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                                     int32_t *dev_status, twn_stream_t stream)
{
    int64_t Hf, Wf, ldf;
    int rc = twn_fold_dims(d, &Hf, &Wf, &ldf);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(Xf && Tf && Y && ld_folded == ldf, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(twn_aligned(Xf, 16) && twn_aligned(Tf, 16) && twn_aligned(Y, 4) && twn_aligned(stats, 8) &&
                    twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    rc = check_epilogue(epi);
    if (rc != TWN_OK) return rc;
    const long long Ho = (d->H + 2 * d->pad_h - d->kh) / 2 + 1, Wo = (d->W + 2 * d->pad_w - d->kw) / 2 + 1;
    // A 64-"channel" tensor whose pixels are 16 elements apart: window position w reads folded
    // pixels w..w+3.  One tap per folded filter row, stride 1, no padding.
    Geometry g;
    memset(&g, 0, sizeof g);
    g.XB = d->B; g.XH = Hf; g.XW = Wo; g.XC = 64; g.ldx = 16;
    g.x_row_pitch = Wf * 16; g.x_img_pitch = Hf * Wf * 16;
    g.Bv = (int)d->B; g.Hv = (int)Ho; g.Wv = (int)Wo; g.OH = (int)Ho; g.OW = (int)Wo;
    g.osh = g.osw = 1; g.ooh = g.oow = 0; g.ldy = d->Cout;
    g.sh = g.sw = 1;
    g.Cout = (int)d->Cout; g.ld_codes = ldf; g.code_cols = ldf;
    g.Cin = 64;
    for (int r = 0; r < (int)(ldf / 64); ++r) {
        Tap &t = g.taps[g.n_taps++];
        t.dh = (int16_t)r;
        t.dw = 0;
        t.koff = (int32_t)(r * 64);
    }
    g.code_bits = 2;
    return launch_conv(g, Xf, Tf, stats, epi, Y, TWN_F32, dev_status, twn_cu(stream));
}

namespace {

int conv_bwd_data_impl(const twn_conv_desc_t *d, const void *dZ, const uint32_t *T_bwd, int64_t ld_codes,
                       const twn_stats_t *stats, const twn_epilogue_t *epi, void *dX,
                       int32_t *dev_status, twn_stream_t stream, int bits)
{
    int rc = conv_common_checks(d);
    if (rc != TWN_OK) return rc;
    TWN_REQUIRE(dZ && T_bwd && dX, TWN_ERR_INVALID_ARG);
    const long long taps = (long long)d->kh * d->kw;
    TWN_REQUIRE(ld_codes % (bits == 1 ? 128 : 64) == 0 && ld_codes >= taps * d->Cout, TWN_ERR_INVALID_ARG);
    TWN_REQUIRE(d->Cout % 8 == 0 && (taps == 1 || d->Cout % (bits == 1 ? 32 : 16) == 0), TWN_ERR_MISALIGNED);
    TWN_REQUIRE(twn_aligned(dZ, 16) && twn_aligned(T_bwd, 16) && twn_aligned(dX, 4) && twn_aligned(stats, 8) &&
                    twn_aligned(dev_status, 4), TWN_ERR_MISALIGNED);
    rc = check_epilogue(epi);
    if (rc != TWN_OK) return rc;
    const long long Ho = (d->H + 2 * d->pad_h - d->kh) / d->stride_h + 1;
    const long long Wo = (d->W + 2 * d->pad_w - d->kw) / d->stride_w + 1;
    // One launch per residue class (ph, pw) of the input pixel modulo the stride: inside a
    // class the adjoint is a stride-1 sum over the taps r with (ph + pad - r) divisible by
    // the stride, reading dZ at ho = h' + (ph + pad - r)/stride.  The classes write disjoint
    // pixels, so with more than one class they run side by side on helper streams.
    cudaStream_t user = twn_cu(stream);
    ForkPool *pool = nullptr;
    std::unique_lock<std::mutex> lock(g_fork_mutex, std::defer_lock);
    if (d->stride_h * d->stride_w > 1) {
        twn_device_info dev;
        rc = twn_current_device(&dev);
        if (rc != TWN_OK) return rc;
        lock.lock();
        pool = fork_pool(dev.ordinal);
        if (pool) {
            TWN_CUDA_OK(cudaEventRecord(pool->fork, user));
            for (int i = 0; i < 3; ++i) TWN_CUDA_OK(cudaStreamWaitEvent(pool->side[i], pool->fork, 0));
        }
    }
    int cls = 0;
    int first_error = TWN_OK;
    for (int ph = 0; ph < d->stride_h; ++ph)
        for (int pw = 0; pw < d->stride_w; ++pw) {
            if (ph >= d->H || pw >= d->W) continue;
            cudaStream_t s = (pool && cls % 4 != 0) ? pool->side[cls % 4 - 1] : user;
            ++cls;
            Geometry g;
            memset(&g, 0, sizeof g);
            g.XB = d->B; g.XH = Ho; g.XW = Wo; g.XC = d->Cout; g.ldx = d->Cout;
            g.Bv = (int)d->B;
            g.Hv = (int)((d->H - ph + d->stride_h - 1) / d->stride_h);
            g.Wv = (int)((d->W - pw + d->stride_w - 1) / d->stride_w);
            g.OH = (int)d->H; g.OW = (int)d->W;
            g.osh = d->stride_h; g.osw = d->stride_w; g.ooh = ph; g.oow = pw;
            g.ldy = d->Cin;
            g.sh = g.sw = 1;
            g.Cout = (int)d->Cin; g.ld_codes = ld_codes; g.code_cols = taps * d->Cout;
            g.Cin = d->Cout;
            for (int r = 0; r < d->kh; ++r) {
                const int xh = ph + d->pad_h - r;
                if (((xh % d->stride_h) + d->stride_h) % d->stride_h != 0) continue;
                for (int s = 0; s < d->kw; ++s) {
                    const int xw = pw + d->pad_w - s;
                    if (((xw % d->stride_w) + d->stride_w) % d->stride_w != 0) continue;
                    Tap &t = g.taps[g.n_taps++];
                    t.dh = (int16_t)(xh / d->stride_h);
                    t.dw = (int16_t)(xw / d->stride_w);
                    t.koff = (int32_t)((r * d->kw + s) * d->Cout);
                }
            }
            g.code_bits = bits;
            // A residue class no tap reaches gets epilogue(0); when the epilogue only adds a second gradient
            // branch that already lives in dX (in place), that leaves the class as it is: nothing to launch.
            if (g.n_taps == 0 && epi && epi->residual == dX && epi->residual_op == TWN_RESIDUAL_ADD && !epi->scale &&
                !epi->shift && !epi->relu && epi->residual_dtype == epi->out_dtype) {
                --cls;              // the class takes no stream slot
                continue;
            }
            rc = launch_conv(g, dZ, T_bwd, stats, epi, dX, TWN_F32, dev_status, s);
            if (rc != TWN_OK && first_error == TWN_OK) first_error = rc;
        }
    if (pool) {
        // always rejoin, also after a failed launch: the caller's stream must not be left forked
        for (int i = 0; i < 3; ++i) {
            TWN_CUDA_OK(cudaEventRecord(pool->join[i], pool->side[i]));
            TWN_CUDA_OK(cudaStreamWaitEvent(user, pool->join[i], 0));
        }
    }
    return first_error;
}

}  // namespace

extern "C" int twn_conv2d_bwd_data(const twn_conv_desc_t *d, const void *dZ, const uint32_t *T_bwd, int64_t ld_codes,
                                   const twn_stats_t *stats, const twn_epilogue_t *epi, void *dX,
                                   int32_t *dev_status, twn_stream_t stream)
{
    return conv_bwd_data_impl(d, dZ, T_bwd, ld_codes, stats, epi, dX, dev_status, stream, 2);
}

extern "C" int twn_conv2d_bwd_data_b1(const twn_conv_desc_t *d, const void *dZ, const uint32_t *B_bwd, int64_t ld_codes,
                                      const twn_stats_t *stats, const twn_epilogue_t *epi, void *dX,
                                      int32_t *dev_status, twn_stream_t stream)
{
    return conv_bwd_data_impl(d, dZ, B_bwd, ld_codes, stats, epi, dX, dev_status, stream, 1);
}

