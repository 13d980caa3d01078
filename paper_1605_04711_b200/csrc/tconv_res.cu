// Ternary-weight contraction for narrow layers (at most 64 output channels): Eq. 2 forward
// block and Algorithm 1 TernaryForward / TernaryBackward, Y = epilogue(alpha * X (*) T), with
// the layer's decoded weights RESIDENT in shared memory.
//
// tconv.cu keeps the weights as the A operand (128 channel rows) and decodes them again for
// every pixel tile; with 64 or fewer output channels half of every MMA is idle and the decode
// and the epilogue pace the kernel.  Here the roles are swapped:
//
//   D[pixel, channel] (+)= A[pixel, k] * B[channel, k]^T      M = 128 pixels, N = Cout (<= 64)
//
//   B  the whole packed code matrix of the layer is decoded ONCE per block into 128-byte
//      swizzled shared memory (exact bf16 +-2 / 0, the factor 2 leaves with alpha) and stays
//      there for every tile the persistent block processes: no decode role in the main loop.
//   A  activations, staged by TMA.  One tile WITH ITS HALO serves all taps of a stride-1
//      filter: a K-major operand may start on any 128-byte row, so tap (dh, dw) is the same
//      shared-memory tile read (dh * row pitch + dw) pixels further.  A 3x3 layer therefore
//      loads (8+2) x (16+2) pixels per 128 outputs instead of nine 128-pixel tiles.
//   D  four accumulators of 64 tensor-memory columns: the epilogue of a tile overlaps the
//      MMAs of the next three.
//
// In the epilogue a thread owns one pixel and reads its channels from tensor memory, so its
// output is one contiguous run (128 bytes of bf16): it goes through a swizzled per-warp
// staging buffer and one TMA store per 32 pixels; a bf16 residual (or gate) tensor arrives
// the same way, one tile ahead.
//
//   warp 0      TMA producer: one activation tile (with halo) per tile and 64-channel block
//   warp 1      allocates tensor memory; one thread issues the tcgen05.mma of every third tile of the block
//   warps 2-9   epilogue: two sets of four (one warp per tensor-memory lane quadrant), the sets
//               take alternate tiles
//   warps 10-11 one thread each issues the tcgen05.mma of the other tiles, in turn
// All warps but the producer decode the weights before their roles start; the producer fetches meanwhile.
//
// Every wait on an mbarrier is bounded; on expiry the kernel records TWN_ERR_TIMEOUT, all roles
// leave their loops, tensor memory is freed and the grid exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstddef>

#include "common.cuh"
#include "tc_ptx.cuh"
#include "tconv_host.cuh"

using namespace twn_detail;

namespace {

constexpr int kPix = 128;                 // pixels per tile (UMMA M)
constexpr int kBlockK = 64;               // reduction elements per k-block (128 bytes of bf16)
constexpr int kNMax = 64;                 // output channels (UMMA N)
constexpr int kAccBufs = 4;
constexpr uint32_t kTmemCols = kAccBufs * kNMax;
constexpr int kEpiWarps = 8;
constexpr int kIssuers = 3;                // MMA-issuing threads: warp 1 and the warps after the epilogue warps
constexpr int kIssuerB = 2 + kEpiWarps;    // the warp of the second MMA-issuing thread
constexpr int kThreads = 32 * (2 + kEpiWarps + (kIssuers - 1));
constexpr int kMaxStages = 8;
constexpr int kStageBuf = 4096;           // per-warp staging: 32 pixels x 128 bytes
constexpr int kSmemLimit = 232448;

struct Ctl {
    unsigned long long full[kMaxStages], empty[kMaxStages];
    unsigned long long acc_full[kAccBufs], acc_empty[kAccBufs];
    unsigned long long res_full[kEpiWarps];
    unsigned long long turn[kIssuers];           // issuer -> issuer: "every stage up to the end of my tile has landed"
    alignas(16) float sc[kNMax];          // read with 16-byte loads
    alignas(16) float sf[kNMax];          // per-channel scale (alpha and the decode factor folded in) and shift
    uint2 tap[kMaxTaps + 1];              // per tap: operand offsets of its first k-block (A inside a stage, B inside the weights), 16-byte units
    uint32_t tmem_base;
    volatile int abort_flag;
};

struct ResParams {
    int total_tiles, tw, th;
    int lgBW, lgBH;               // pixel tile = BB x BH x BW, powers of two, product 128
    int n_taps, n_cblk, kbpt;     // k-blocks per tile = n_taps * n_cblk
    int N;                        // UMMA N: Cout rounded up to 16
    int Cout;
    const uint32_t *T;            // packed codes, one row of `wpr` words per output channel
    long long wpr;
    int codes_aligned;            // 1: every k-block starts on a 64-code boundary of the packed row
    int code_bits;                // 2: ternary codes; 1: binary codes
    int w_lo, h_lo;               // smallest tap offsets: origin of the halo
    int stage_bytes, stage_tx;    // pitch of an activation stage (multiple of 1024), bytes one load delivers
    int n_stages;
    uint32_t a_sbo;               // bytes between consecutive 8-pixel groups of the A operand
    uint32_t wts_off, stg_off, res_off, ctl_off;   // regions of the dynamic shared memory
    int osw, osh;                 // output pixel = virtual pixel * (osh, osw) (+ offset, in the tensor map's base)
    const double *alpha;
    const float *scale, *shift;
    int has_res, res_gate, relu, out_bf16;
    int32_t *status;
    int a_off[kMaxTaps];          // start of tap t inside a stage, in 16-byte units
    int koff[kMaxTaps];           // first code column of tap t in a packed row
};

// K-major, 128-byte swizzled operand whose 8-row groups are `sbo_bytes` apart.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t saddr, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// D[tmem] (+)= A[smem] * B[smem]^T, issued by the calling thread alone.  The descriptors arrive as
// halves: the upper words never change and the lower ones advance by 32-bit additions, so an MMA
// costs its issuing thread two additions and the instruction itself.
template <bool ACC>
__device__ __forceinline__ void tc_mma_ss_1t(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                             uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(ACC ? 1 : 0)
        : "memory");
}
// One k-block of one tap: four K = 16 steps, 32 bytes apart in both operands.
template <bool FIRST>
__device__ __forceinline__ void tc_mma_tap(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                           uint32_t idesc)
{
    tc_mma_ss_1t<!FIRST>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc);
    tc_mma_ss_1t<true>(d_tmem, a_lo + 2, a_hi, b_lo + 2, b_hi, idesc);
    tc_mma_ss_1t<true>(d_tmem, a_lo + 4, a_hi, b_lo + 4, b_hi, idesc);
    tc_mma_ss_1t<true>(d_tmem, a_lo + 6, a_hi, b_lo + 6, b_hi, idesc);
}
__device__ __forceinline__ void tc_commit_1t(void *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// The register cap is below what one block per SM would allow (65536 / 384 = 170): the block then leaves room
// on its SM for a small block of another stream.  In a training step the reduction kernels of the weight-
// gradient stream run in that room beside this kernel; with 168 registers per thread they had to wait for it
// (ResNet-18 step, batch 64: 1.424 ms against 1.387 ms with the cap; no spills either way).
__global__ void __maxnreg__(144)
tconv_res_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                 const __grid_constant__ CUtensorMap map_r, const __grid_constant__ ResParams P)
{
    pdl_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    uint8_t *const base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctl *const ctl = reinterpret_cast<Ctl *>(base + P.ctl_off);
    volatile int *abort_flag = &ctl->abort_flag;
    const uint32_t base_u32 = smem_u32(base);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BWm = (1 << P.lgBW) - 1, BHm = (1 << P.lgBH) - 1;
    const int lgHW = P.lgBW + P.lgBH;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int b = 0; b < kAccBufs; ++b) { mbar_init(&ctl->acc_full[b], 1); mbar_init(&ctl->acc_empty[b], 4); }
        for (int w = 0; w < kEpiWarps; ++w) mbar_init(&ctl->res_full[w], 1);
        for (int i = 0; i < kIssuers; ++i) mbar_init(&ctl->turn[i], 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // The producer warp does not take part in the set-up below: it signals the barriers it has initialised
    // and starts fetching the first activation tiles at once, so that their latency (the operands come from
    // DRAM) runs beside the decoding of the weights instead of after it.
    // nothing above touched global memory; from here on every role reads what earlier kernels wrote
    pdl_wait();
    if (warp == 0) {
        asm volatile("bar.arrive 1, %0;" ::"n"(kThreads) : "memory");
    } else {
        constexpr int kWorkers = kThreads - 32;
        const int tid = threadIdx.x - 32;
        // per-channel scale and shift; the decoded weights are +-2, so half of alpha scales the accumulators
        if (tid < kNMax) {
            const int c = tid;
            const float alpha = (P.alpha ? (float)(*P.alpha) : 1.0f) * (P.code_bits == 2 ? 1.0f / kDecodedUnit : 1.0f);
            const bool c_ok = c < P.Cout;
            ctl->sc[c] = ((P.scale && c_ok) ? __ldg(P.scale + c) : 1.0f) * alpha;
            ctl->sf[c] = (P.shift && c_ok) ? __ldg(P.shift + c) : 0.0f;
        }
        for (int t = tid; t <= P.n_taps && t <= kMaxTaps; t += kWorkers)
            ctl->tap[t] = make_uint2(t < P.n_taps ? (uint32_t)P.a_off[t] : 0u, (uint32_t)(t * P.n_cblk) * ((uint32_t)(P.N * 128) >> 4));
        // Decode the layer: item (channel n, k-block u) = 64 codes = 16 bytes -> 128 bytes of bf16, written as
        // row n of k-block u in the K-major layout the MMA reads (16-byte chunk j of row n at chunk j ^ (n & 7)).
        // Code words past the end of a row are clamped into it: they only ever meet activations that the TMA
        // zero-fills.  Rows past Cout are zero.
        {
            const uint32_t wts = base_u32 + P.wts_off;
            const int items = P.N * P.kbpt;
            for (int i = tid; i < items; i += kWorkers) {
                const int u = i / P.N, n = i - u * P.N;
                const int t = u / P.n_cblk, cb = u - t * P.n_cblk;
                const uint32_t *rowp = P.T + (long long)(n < P.Cout ? n : P.Cout - 1) * P.wpr;
                uint32_t wv[4] = {0u, 0u, 0u, 0u};
                const long long last = P.wpr - 1;
                if (P.code_bits == 2) {
                    const long long word = (P.koff[t] >> 4) + cb * (kBlockK / 16);
                    if (P.codes_aligned) {
                        uint4 c;
                        ld_nc_v4(c, rowp + word);
                        wv[0] = c.x; wv[1] = c.y; wv[2] = c.z; wv[3] = c.w;
                    } else {
#pragma unroll
                        for (int g = 0; g < 4; ++g) ld_nc_u32(wv[g], rowp + (word + g < last ? word + g : last));
                    }
                } else {
                    const long long word = (P.koff[t] >> 5) + cb * (kBlockK / 32);
#pragma unroll
                    for (int g = 0; g < 2; ++g) ld_nc_u32(wv[g], rowp + (word + g < last ? word + g : last));
                }
                uint32_t out[32];
                if (P.code_bits == 2) decode_kblock<2>(wv, out);
                else decode_kblock<1>(wv, out);
                if (n >= P.Cout) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) out[j] = 0u;
                }
                const uint32_t dst = wts + (uint32_t)(u * P.N + n) * 128u;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    st_shared_v4(dst + (uint32_t)((j ^ (n & 7)) << 4), out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
            }
            // the tensor core reads shared memory through the async proxy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
        tc_fence_after();
    }
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0 && P.kbpt > 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x) {
                int pt = tile;
                const int twi = pt % P.tw; pt /= P.tw;
                const int thi = pt % P.th;
                const int tbi = pt / P.th;
                const int w0 = (twi << P.lgBW) + P.w_lo, h0 = (thi << P.lgBH) + P.h_lo, b0 = tbi * (kPix >> lgHW);
                for (int cb = 0; cb < P.n_cblk; ++cb) {
                    if (!mbar_wait(&ctl->empty[s], ph ^ 1u, abort_flag, P.status)) { ok = false; break; }
                    mbar_expect_tx(&ctl->full[s], (uint32_t)P.stage_tx);
                    tma_load_4d(base + (size_t)s * P.stage_bytes, &map_x, &ctl->full[s], cb * kBlockK, w0, h0, b0);
                    if (++s == (uint32_t)P.n_stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1 || warp >= kIssuerB) {
        // ------------------------------------------------ MMA issuers: three threads, tiles in turn
        // Measured on B200: a 128x64x16 MMA with both operands in shared memory occupies the tensor core
        // for 48 cycles, and tcgen05.mma holds its issuing thread until the tensor core accepts it, so every
        // instruction that thread runs between two MMAs (address arithmetic, waits) is time the tensor core
        // idles: one issuer reached 59 to 76 cycles per MMA, two issuers on different accumulators 48 while
        // both are issuing.  A thread also waits three times per tile (token, accumulator, stage) and commits
        // twice; with short tiles (16 MMAs in the folded first layer of ResNet-18) two threads spend so much of
        // their time there that the tensor core idles half of the time, hence three.  The threads take the tiles
        // in turn; each works on the accumulator and the activation stages of its own tile, so the instruction
        // streams never touch the same data.
        // The stages form one ring that all of them consume, and an mbarrier wait only tells a phase from
        // its neighbours: a thread may wait for "stage s, parity p" only once every earlier phase of that
        // barrier is known to be over.  So the threads pass a token: after seeing the last stage of its tile
        // land, a thread lets the next one start waiting for the stages of the next tile.
        if (lane == 0 && P.kbpt > 0) {
            const uint32_t me = warp == 1 ? 0u : (uint32_t)(warp - kIssuerB + 1);
            const uint32_t idesc = make_idesc(kPix, P.N);
            const uint64_t adesc0 = smem_desc_k_sw128(base_u32, P.a_sbo);
            const uint64_t bdesc0 = smem_desc_sw128(base_u32 + P.wts_off);
            const uint32_t a_hi = (uint32_t)(adesc0 >> 32), b_hi = (uint32_t)(bdesc0 >> 32);
            const uint32_t a_lo0 = (uint32_t)adesc0, b_lo0 = (uint32_t)bdesc0;
            const uint32_t b_step = (uint32_t)(P.N * 128) >> 4;      // one k-block of weights, 16-byte units
            const uint32_t a_step = (uint32_t)P.stage_bytes >> 4;
            const int n_taps = P.n_taps;
            uint32_t s = 0, ph = 0;
            // stage position of this thread's first tile, then of every other tile
            auto skip_tile = [&]() {
                for (int cb = 0; cb < P.n_cblk; ++cb)
                    if (++s == (uint32_t)P.n_stages) { s = 0; ph ^= 1u; }
            };
            for (uint32_t i = 0; i < me; ++i) skip_tile();
            bool ok = true;
            uint32_t lt = me;
            for (int tile = blockIdx.x + (int)me * (int)gridDim.x; tile < P.total_tiles && ok; tile += kIssuers * (int)gridDim.x, lt += kIssuers) {
                const uint32_t buf = lt & (kAccBufs - 1);
                // The token first: once it is here, the threads of all earlier tiles are past their waits for an
                // accumulator, so the accumulator barrier (shared by the issuing threads in turn) is at most one
                // phase behind the one waited for.
                if (lt > 0 && !mbar_wait(&ctl->turn[me], ((lt - 1) / kIssuers) & 1u, abort_flag, P.status, 0)) break;
                if (!mbar_wait(&ctl->acc_empty[buf], ((lt / kAccBufs) & 1u) ^ 1u, abort_flag, P.status, 0)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem + buf * kNMax;
                for (int cb = 0; cb < P.n_cblk; ++cb) {
                    if (!mbar_wait(&ctl->full[s], ph, abort_flag, P.status, 0)) { ok = false; break; }
                    if (cb == P.n_cblk - 1) mbar_arrive(&ctl->turn[me + 1 == kIssuers ? 0u : me + 1]);
                    tc_fence_after();
                    const uint32_t a_s = a_lo0 + s * a_step, b_s = b_lo0 + (uint32_t)cb * b_step;
                    uint2 cur = ctl->tap[0];
                    uint2 nxt = ctl->tap[1];
                    if (cb == 0) tc_mma_tap<true>(d_tmem, a_s + cur.x, a_hi, b_s + cur.y, b_hi, idesc);
                    else tc_mma_tap<false>(d_tmem, a_s + cur.x, a_hi, b_s + cur.y, b_hi, idesc);
#pragma unroll 1
                    for (int t = 1; t < n_taps; ++t) {
                        cur = nxt;
                        nxt = ctl->tap[t + 1];
                        tc_mma_tap<false>(d_tmem, a_s + cur.x, a_hi, b_s + cur.y, b_hi, idesc);
                    }
                    tc_commit_1t(&ctl->empty[s]);
                    if (++s == (uint32_t)P.n_stages) { s = 0; ph ^= 1u; }
                }
                if (ok) {
                    tc_commit_1t(&ctl->acc_full[buf]);
                    for (int i = 1; i < kIssuers; ++i) skip_tile();
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue
        const int ew = warp - 2;
        const int set = ew >> 2;                 // which of the two sets; a set takes every other tile
        const int q = warp & 3;                  // tensor-memory lane quadrant of this warp
        const uint32_t stg = base_u32 + P.stg_off + (uint32_t)ew * kStageBuf;
        const uint32_t res = base_u32 + P.res_off + (uint32_t)ew * kStageBuf;
        const uint32_t my_row = (uint32_t)lane * 128u;
        const uint32_t sw_x = (uint32_t)(lane & 7);
        const int chunks = (P.N + 31) >> 5;      // 32-channel chunks of the accumulator
        const bool per_channel = P.scale != nullptr || P.shift != nullptr;
        const float sc_all = ctl->sc[0];         // without a per-channel scale every entry is the same
        const int p0 = q * 32;                   // first tile pixel of this warp
        uint32_t nres = 0;

        auto tile_coords = [&](int tile, int &cw, int &ch, int &cbt) {
            int pt = tile;
            const int twi = pt % P.tw; pt /= P.tw;
            const int thi = pt % P.th;
            const int tbi = pt / P.th;
            cw = ((twi << P.lgBW) + (p0 & BWm)) * P.osw;
            ch = ((thi << P.lgBH) + ((p0 >> P.lgBW) & BHm)) * P.osh;
            cbt = tbi * (kPix >> lgHW) + (p0 >> lgHW);
        };
        auto res_load = [&](int tile) {
            int cw, ch, cbt;
            tile_coords(tile, cw, ch, cbt);
            mbar_expect_tx(&ctl->res_full[ew], kStageBuf);
            tma_load_4d(base + P.res_off + (size_t)ew * kStageBuf, &map_r, &ctl->res_full[ew], 0, cw, ch, cbt);
        };
        const int first_tile = blockIdx.x + set * (int)gridDim.x;
        if (P.has_res && lane == 0 && first_tile < P.total_tiles) res_load(first_tile);

        uint32_t lt = set;
        for (int tile = first_tile; tile < P.total_tiles; tile += 2 * (int)gridDim.x, lt += 2) {
            int cw, ch, cbt;
            tile_coords(tile, cw, ch, cbt);
            const uint32_t buf = lt & (kAccBufs - 1);
            if (P.kbpt > 0 && !mbar_wait_warp(&ctl->acc_full[buf], (lt / kAccBufs) & 1u, abort_flag, P.status, 32)) break;
            tc_fence_after();
            const uint32_t t_acc = tmem + ((uint32_t)(q * 32) << 16) + buf * kNMax;
            if (P.out_bf16) {
                // the staging buffer was last read by the store of this warp's previous tile
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
            }
            // The whole accumulator goes to registers at once (one exposed tensor-memory latency per tile
            // instead of one per 32 channels) and is handed back before any arithmetic.
            uint32_t va[32], vb[32];
            if (P.kbpt > 0) {
                tmem_ld32(t_acc, va);
                if (chunks > 1) tmem_ld32(t_acc + 32, vb);
                tmem_wait_ld(va);
                if (chunks > 1) tmem_wait_ld(vb);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->acc_empty[buf]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) va[j] = vb[j] = 0u;
            }
            if (P.has_res && !mbar_wait_warp(&ctl->res_full[ew], nres & 1u, abort_flag, P.status, 32)) break;
            // 32 channels of this thread's pixel: affine (two channels per instruction), residual or gate, ReLU,
            // conversion, staging
            auto chunk = [&](uint32_t (&v)[32], const int hf) {
                if (per_channel) {
                    // all sixteen loads of the scales and shifts are issued before the first use
                    const uint32_t sc_a = smem_u32(ctl->sc + hf * 32), sf_a = smem_u32(ctl->sf + hf * 32);
                    uint4 a[8], b[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) a[j] = ld_shared_v4(sc_a + j * 16);
#pragma unroll
                    for (int j = 0; j < 8; ++j) b[j] = ld_shared_v4(sf_a + j * 16);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        fma_f32x2(v[4 * j + 0], v[4 * j + 1], __uint_as_float(a[j].x), __uint_as_float(a[j].y),
                                  __uint_as_float(b[j].x), __uint_as_float(b[j].y));
                        fma_f32x2(v[4 * j + 2], v[4 * j + 3], __uint_as_float(a[j].z), __uint_as_float(a[j].w),
                                  __uint_as_float(b[j].z), __uint_as_float(b[j].w));
                    }
                } else {
                    // one factor for every channel (alpha and the decode factor): it lives in a register
#pragma unroll
                    for (int j = 0; j < 16; ++j) fma_f32x2(v[2 * j], v[2 * j + 1], sc_all, sc_all, 0.0f, 0.0f);
                }
                if (P.has_res) {
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const uint4 r = ld_shared_v4(res + my_row + ((((uint32_t)(hf * 4 + jj)) ^ sw_x) << 4));
                        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float r0 = __uint_as_float(rw[i] << 16), r1 = __uint_as_float(rw[i] & 0xFFFF0000u);
                            float &y0 = reinterpret_cast<float &>(v[jj * 8 + 2 * i]);
                            float &y1 = reinterpret_cast<float &>(v[jj * 8 + 2 * i + 1]);
                            if (P.res_gate) {
                                y0 = r0 > 0.0f ? y0 : 0.0f;
                                y1 = r1 > 0.0f ? y1 : 0.0f;
                            } else {
                                y0 += r0;
                                y1 += r1;
                            }
                        }
                    }
                }
                if (P.out_bf16) {
                    // the ReLU rides on the conversion
                    if (P.relu) {
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj)
                            st_shared_v4(stg + my_row + ((((uint32_t)(hf * 4 + jj)) ^ sw_x) << 4),
                                         pack_bf16x2_relu(__uint_as_float(v[jj * 8 + 0]), __uint_as_float(v[jj * 8 + 1])),
                                         pack_bf16x2_relu(__uint_as_float(v[jj * 8 + 2]), __uint_as_float(v[jj * 8 + 3])),
                                         pack_bf16x2_relu(__uint_as_float(v[jj * 8 + 4]), __uint_as_float(v[jj * 8 + 5])),
                                         pack_bf16x2_relu(__uint_as_float(v[jj * 8 + 6]), __uint_as_float(v[jj * 8 + 7])));
                    } else {
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj)
                            st_shared_v4(stg + my_row + ((((uint32_t)(hf * 4 + jj)) ^ sw_x) << 4),
                                         pack_bf16x2(__uint_as_float(v[jj * 8 + 0]), __uint_as_float(v[jj * 8 + 1])),
                                         pack_bf16x2(__uint_as_float(v[jj * 8 + 2]), __uint_as_float(v[jj * 8 + 3])),
                                         pack_bf16x2(__uint_as_float(v[jj * 8 + 4]), __uint_as_float(v[jj * 8 + 5])),
                                         pack_bf16x2(__uint_as_float(v[jj * 8 + 6]), __uint_as_float(v[jj * 8 + 7])));
                    }
                } else {
                    // fp32: 32 channels are a 128-byte row of their own box; one store per chunk
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
                    if (P.relu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(fmaxf(__uint_as_float(v[j]), 0.0f));
                    }
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj)
                        st_shared_v4(stg + my_row + ((((uint32_t)jj) ^ sw_x) << 4), v[jj * 4 + 0], v[jj * 4 + 1], v[jj * 4 + 2],
                                     v[jj * 4 + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) tma_store_4d(&map_y, base + P.stg_off + (size_t)ew * kStageBuf, hf * 32, cw, ch, cbt);
                }
            };
            chunk(va, 0);
            if (chunks > 1) chunk(vb, 1);
            if (P.out_bf16) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) tma_store_4d(&map_y, base + P.stg_off + (size_t)ew * kStageBuf, 0, cw, ch, cbt);
            }
            if (P.has_res) {
                // every lane has read its row of the residual: fetch the one of this warp's next tile
                ++nres;
                __syncwarp();
                const int next = tile + 2 * (int)gridDim.x;
                if (lane == 0 && next < P.total_tiles) res_load(next);
            }
        }
        // all bulk stores of this thread have been written before the block may exit
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (ctl->abort_flag) {
        // give copies and MMAs still in flight time to land before the memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

int twn_detail::launch_conv_resident(const Geometry &g, const void *X, const uint32_t *T, const EpilogueArgs &epi,
                                     void *Y, int32_t *dev_status, const twn_device_info &dev, cudaStream_t s,
                                     bool *handled)
{
    *handled = false;
    if (g.sw != 1 || g.sh != 1 || g.Cout > kNMax || g.Cout < 1) return TWN_OK;
    if (g.bn_partial) return TWN_OK;      // batch statistics come out of the general kernel's epilogue
    const bool out_bf16 = epi.out_dtype == TWN_BF16;
    const int es = out_bf16 ? 2 : 4;
    // the output (and a residual) must be addressable by TMA
    if ((g.ldy * es) % 16 != 0 || ((long long)g.Cout * es) % 16 != 0 || reinterpret_cast<uintptr_t>(Y) % 16 != 0 ||
        g.OW <= g.oow || g.OH <= g.ooh)
        return TWN_OK;
    if (epi.residual && (epi.res_dtype != TWN_BF16 || (g.ldy * 2) % 16 != 0 || ((long long)g.Cout * 2) % 16 != 0 ||
                         reinterpret_cast<uintptr_t>(epi.residual) % 16 != 0))
        return TWN_OK;

    ResParams P;
    memset(&P, 0, sizeof P);
    P.n_taps = g.n_taps;
    P.n_cblk = (int)((g.Cin + kBlockK - 1) / kBlockK);
    P.kbpt = P.n_taps * P.n_cblk;
    P.N = (g.Cout + 15) / 16 * 16;
    P.Cout = g.Cout;
    P.codes_aligned = 1;
    int w_lo = 0, w_hi = 0, h_lo = 0, h_hi = 0;
    for (int t = 0; t < g.n_taps; ++t) {
        if (g.taps[t].koff % (g.code_bits == 1 ? 32 : 16) != 0) return TWN_OK;   // code words must not straddle taps
        if (g.taps[t].koff % kBlockK != 0) P.codes_aligned = 0;
        P.koff[t] = g.taps[t].koff;
        if (t == 0) { w_lo = w_hi = g.taps[t].dw; h_lo = h_hi = g.taps[t].dh; }
        if (g.taps[t].dw < w_lo) w_lo = g.taps[t].dw;
        if (g.taps[t].dw > w_hi) w_hi = g.taps[t].dw;
        if (g.taps[t].dh < h_lo) h_lo = g.taps[t].dh;
        if (g.taps[t].dh > h_hi) h_hi = g.taps[t].dh;
    }
    const int hw = w_hi - w_lo, hh = h_hi - h_lo;
    // Tile shape.  With a halo in w the tile is 8 pixels wide (an 8-row group of the operand is one
    // row segment, the halo only changes the distance between groups); with a halo in h only, rows
    // follow each other densely and any width works; a halo rules out more than one image per tile.
    if (hw > 0) {
        P.lgBW = 3; P.lgBH = 4;
    } else if (hh > 0) {
        long long best = -1;
        for (int a = 0; a <= 7; ++a) {
            const int BW = 1 << a, BH = kPix >> a;
            const long long tiles = (long long)((g.Wv + BW - 1) / BW) * ((g.Hv + BH - 1) / BH) * g.Bv;
            if (best < 0 || tiles < best || (tiles == best && BW <= 16)) { best = tiles; P.lgBW = a; P.lgBH = 7 - a; }
        }
    } else {
        pick_tile(g, kPix, &P.lgBW, &P.lgBH);
    }
    const int BW = 1 << P.lgBW, BH = 1 << P.lgBH, BB = kPix >> (P.lgBW + P.lgBH);
    if (BW + hw > 256 || BH + hh > 256 || BB > 256) return TWN_OK;
    P.tw = (g.Wv + BW - 1) / BW;
    P.th = (g.Hv + BH - 1) / BH;
    const long long tb = (g.Bv + BB - 1) / BB;
    const long long total = (long long)P.tw * P.th * tb;
    if (total <= 0 || total > 0x7fffffffLL) return TWN_ERR_INVALID_ARG;
    P.total_tiles = (int)total;
    // large problems whose tiles would be mostly empty stay with the general kernel
    const long long pixels = (long long)g.Bv * g.Hv * g.Wv;
    if (pixels > 65536 && total * kPix > 3 * pixels) return TWN_OK;

    P.w_lo = w_lo; P.h_lo = h_lo;
    const int row_pix = BW + hw;
    P.a_sbo = hw > 0 ? (uint32_t)row_pix * 128u : 1024u;
    for (int t = 0; t < g.n_taps; ++t)
        P.a_off[t] = (((g.taps[t].dh - h_lo) * row_pix + (g.taps[t].dw - w_lo)) * 128) >> 4;
    P.stage_tx = 128 * row_pix * (BH + hh) * BB;
    P.stage_bytes = (P.stage_tx + 1023) / 1024 * 1024;
    const long long wts_bytes = (long long)P.kbpt * P.N * 128;
    const long long fixed = 1024 + wts_bytes + kEpiWarps * kStageBuf * (epi.residual ? 2 : 1) + 2048;
    if (fixed > kSmemLimit) return TWN_OK;
    int n_stages = P.kbpt > 0 ? (int)((kSmemLimit - fixed) / P.stage_bytes) : 0;
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    if (P.kbpt > 0 && n_stages < 2) return TWN_OK;
    P.n_stages = n_stages;
    P.wts_off = (uint32_t)(n_stages * P.stage_bytes);
    P.stg_off = P.wts_off + (uint32_t)wts_bytes;
    P.res_off = P.stg_off + kEpiWarps * kStageBuf;
    P.ctl_off = P.res_off + (epi.residual ? kEpiWarps * kStageBuf : 0);
    static_assert(sizeof(Ctl) <= 2048, "control block");
    const int smem_bytes = 1024 + (int)P.ctl_off + 2048;

    P.T = T;
    P.wpr = g.ld_codes / (g.code_bits == 1 ? 32 : 16);
    P.code_bits = g.code_bits == 1 ? 1 : 2;
    P.osw = g.osw; P.osh = g.osh;
    P.alpha = epi.alpha;
    P.scale = epi.scale; P.shift = epi.shift;
    P.has_res = epi.residual ? 1 : 0;
    P.res_gate = epi.residual ? epi.res_gate : 0;
    P.relu = epi.relu;
    P.out_bf16 = out_bf16 ? 1 : 0;
    P.status = dev_status;

    EncodeTiledFn enc = encode_fn();
    if (!enc) return TWN_ERR_CUDA;
    // activations: (C, W, H, B), one 64-channel block of a tile with its halo per load, zero fill outside
    CUtensorMap map_x;
    {
        cuuint64_t dims[4] = {(cuuint64_t)g.XC, (cuuint64_t)g.XW, (cuuint64_t)g.XH, (cuuint64_t)g.XB};
        const long long rowp = g.x_row_pitch ? g.x_row_pitch : g.XW * g.ldx;
        const long long imgp = g.x_img_pitch ? g.x_img_pitch : g.XH * rowp;
        cuuint64_t strides[3] = {(cuuint64_t)g.ldx * 2, (cuuint64_t)rowp * 2, (cuuint64_t)imgp * 2};
        cuuint32_t box[4] = {(cuuint32_t)kBlockK, (cuuint32_t)row_pix, (cuuint32_t)(BH + hh), (cuuint32_t)BB};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(X), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TWN_OK;
    }
    // output and residual: 32 consecutive tile pixels (one epilogue warp) are a sub-box of the tile;
    // rows of 128 bytes (64 bf16 or 32 fp32 channels), 128-byte swizzle.  The virtual grid may sit in
    // the tensor with a stride and an offset (backward for data of a strided layer).
    CUtensorMap map_y, map_r;
    {
        const int lg_sbw = P.lgBW < 5 ? P.lgBW : 5;
        const int lg_sbh = P.lgBH < 5 - lg_sbw ? P.lgBH : 5 - lg_sbw;
        const int lg_sbb = 5 - lg_sbw - lg_sbh;
        cuuint32_t box[4] = {(cuuint32_t)(out_bf16 ? 64 : 32), (cuuint32_t)((1 << lg_sbw) * g.osw),
                             (cuuint32_t)((1 << lg_sbh) * g.osh), 1u << lg_sbb};
        if (box[1] > 256 || box[2] > 256) return TWN_OK;
        cuuint64_t dims[4] = {(cuuint64_t)g.Cout, (cuuint64_t)(g.OW - g.oow), (cuuint64_t)(g.OH - g.ooh), (cuuint64_t)g.Bv};
        cuuint32_t estr[4] = {1, (cuuint32_t)g.osw, (cuuint32_t)g.osh, 1};
        const long long base_pix = (long long)g.ooh * g.OW + g.oow;
        cuuint64_t strides[3] = {(cuuint64_t)g.ldy * es, (cuuint64_t)g.OW * g.ldy * es, (cuuint64_t)g.OH * g.OW * g.ldy * es};
        void *ybase = static_cast<char *>(Y) + base_pix * g.ldy * es;
        if (enc(&map_y, out_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ybase, dims, strides,
                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TWN_OK;
        map_r = map_y;
        if (epi.residual) {
            cuuint32_t rbox[4] = {64u, box[1], box[2], box[3]};
            cuuint64_t rstrides[3] = {(cuuint64_t)g.ldy * 2, (cuuint64_t)g.OW * g.ldy * 2, (cuuint64_t)g.OH * g.OW * g.ldy * 2};
            void *rbase = const_cast<char *>(static_cast<const char *>(epi.residual)) + base_pix * g.ldy * 2;
            if (enc(&map_r, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, rbase, dims, rstrides, rbox, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return TWN_OK;
        }
    }

    static bool attr_set[64] = {false};
    if (!attr_set[dev.ordinal]) {
        TWN_CUDA_OK(cudaFuncSetAttribute(tconv_res_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
        attr_set[dev.ordinal] = true;
    }
    const int grid = dev.sm_count < P.total_tiles ? dev.sm_count : P.total_tiles;
    TWN_CUDA_OK(twn_launch_pdl(grid * 2 >= dev.sm_count, tconv_res_kernel, grid, kThreads, (size_t)smem_bytes, s, map_x, map_y, map_r, P));
    TWN_CUDA_OK(cudaGetLastError());
    *handled = true;
    return TWN_OK;
}
