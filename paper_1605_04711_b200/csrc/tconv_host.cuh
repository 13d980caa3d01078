// Host-side description of one contraction launch, shared by the tensor-core kernels of the
// ternary-weight contraction: the sum over taps, the virtual output grid and its embedding in
// the output tensor, and the tensor-map encoder of the driver.
#pragma once

#include <cuda.h>
#include <stdint.h>
#include <string.h>

#include "common.cuh"

namespace twn_detail {

constexpr int kMaxTaps = 64;

struct Tap {
    int16_t dh, dw;   // input pixel offset of this tap
    int32_t koff;     // first code column of this tap in a packed row
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
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

struct Geometry {
    // input tensor X: NHWC [XB, XH, XW, XC] with pixel pitch ldx (elements)
    long long XB, XH, XW, XC, ldx;
    long long x_row_pitch, x_img_pitch;   // elements between rows / images; 0 = dense (XW*ldx, XH*XW*ldx)
    // virtual output grid and embedding
    int Bv, Hv, Wv, OH, OW, osh, osw, ooh, oow;
    long long ldy;
    int sh, sw;      // input step per virtual output pixel
    int Cout;
    long long ld_codes, code_cols;  // packed row pitch and used columns
    int code_bits;   // 2: ternary codes, 16 per word; 1: binary codes, 32 per word
    // batch statistics of the pre-activation output (optional): per-tile partial sums, then the totals
    float *bn_partial;
    size_t bn_partial_bytes;
    double *bn_sum, *bn_sumsq;
    int n_taps;
    Tap taps[kMaxTaps];
    long long Cin;   // channels per tap
};

// Picks the pixel-tile shape BW x BH x BB (BW and BH powers of two, product `pix`) that needs the
// fewest tiles.
inline long long pick_tile(const Geometry &g, int pix, int *lgBW, int *lgBH)
{
    int lg = 0;
    while (((pix >> lg) & 1) == 0) ++lg;      // BW * BH divides the power-of-two part of `pix`
    long long best = -1;
    int bw = 0, bh = 0;
    for (int a = 0; a <= lg; ++a)
        for (int b = 0; a + b <= lg; ++b) {
            const int BW = 1 << a, BH = 1 << b, BB = pix >> (a + b);
            if (BW * g.sw > 256 || BH * g.sh > 256 || BB > 256) continue;
            const long long tiles = ((g.Wv + BW - 1) / BW) * (long long)((g.Hv + BH - 1) / BH) * ((g.Bv + BB - 1) / BB);
            // prefer fewer tiles, then wider rows
            if (best < 0 || tiles < best || (tiles == best && a > bw)) { best = tiles; bw = a; bh = b; }
        }
    *lgBW = bw; *lgBH = bh;
    return best;
}

// What follows the contraction (twn_epilogue_t with the device scalar alpha resolved).
struct EpilogueArgs {
    const double *alpha;          // device scalar (twn_stats_t::alpha) or nullptr for 1
    const float *scale, *shift;
    const void *residual;
    int res_dtype, res_gate, relu, out_dtype;
};

// Contraction with the layer's decoded weights resident in shared memory (tconv_res.cu).  Launches
// and returns TWN_OK with *handled = true when the launch fits that kernel (at most 64 output
// channels, unit input stride, decoded weights that fit in shared memory, outputs that TMA can
// store); otherwise *handled = false and nothing has been launched.
int launch_conv_resident(const Geometry &g, const void *X, const uint32_t *T, const EpilogueArgs &epi, void *Y,
                         int32_t *dev_status, const twn_device_info &dev, cudaStream_t s, bool *handled);

}  // namespace twn_detail
