// The full-precision ends of a tiled convolution stack.  The paper tiles only layers above a size threshold (Sec. 3,
// hyperparameter lambda): in a ResNet-style stack the first convolution (a few thousand weights) and the classifier
// stay full precision.  These kernels run them, and the global average pooling between the last convolution and the
// classifier, so that the stack executes end to end on the device.  All three are small, memory-bound layers.
#include "common.cuh"

namespace tbn {

namespace {

constexpr int kDcCo = 8;              // output channels per thread
constexpr int kDcMaxW = 4096;         // weights of one group of kDcCo filters held in shared memory (fp32)

// Direct convolution with a dense fp32 weight (Cout, Cin, kh, kw) for layers with a short contraction (Cin*kh*kw up to
// 512): a thread owns one output pixel and kDcCo consecutive output channels; the weights of those channels sit in
// shared memory and are read as broadcasts; consecutive threads own consecutive pixels of a row, so every store
// instruction writes one contiguous run per channel plane.
template <typename XT, typename YT>
__global__ void __launch_bounds__(256)
dense_conv_kernel(const XT *__restrict__ x, const float *__restrict__ w, const float *__restrict__ bias, YT *__restrict__ y,
                  int32_t Nb, int32_t Cin, int32_t H, int32_t Wd, int32_t Cout, int32_t kh, int32_t kw, int32_t stride,
                  int32_t pad, int32_t Ho, int32_t Wo, int act)
{
    __shared__ float ws[kDcMaxW];
    const int32_t n = Cin * kh * kw;
    const int32_t co0 = blockIdx.y * kDcCo;
    for (int32_t i = threadIdx.x; i < kDcCo * n; i += blockDim.x) {
        const int32_t c = i / n, r = i - c * n;
        ws[i] = co0 + c < Cout ? __ldg(w + (int64_t)(co0 + c) * n + r) : 0.0f;
    }
    __syncthreads();
    const int64_t pixels = (int64_t)Nb * Ho * Wo;
    for (int64_t pix = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; pix < pixels; pix += (int64_t)gridDim.x * blockDim.x) {
        const int32_t ow = (int32_t)(pix % Wo);
        const int64_t t = pix / Wo;
        const int32_t oh = (int32_t)(t % Ho);
        const int64_t b = t / Ho;
        float acc[kDcCo];
#pragma unroll
        for (int c = 0; c < kDcCo; ++c) acc[c] = 0.0f;
        for (int32_t ci = 0; ci < Cin; ++ci)
            for (int32_t u = 0; u < kh; ++u) {
                const int32_t ih = oh * stride + u - pad;
                if (ih < 0 || ih >= H) continue;
                for (int32_t v = 0; v < kw; ++v) {
                    const int32_t iw = ow * stride + v - pad;
                    if (iw < 0 || iw >= Wd) continue;
                    const float xv = load_as_float(x, ((b * Cin + ci) * H + ih) * (int64_t)Wd + iw);
                    const int32_t r = (ci * kh + u) * kw + v;
#pragma unroll
                    for (int c = 0; c < kDcCo; ++c) acc[c] = fmaf(ws[c * n + r], xv, acc[c]);
                }
            }
#pragma unroll
        for (int c = 0; c < kDcCo; ++c) {
            if (co0 + c >= Cout) break;
            const float o = apply_act(acc[c] + (bias ? __ldg(bias + co0 + c) : 0.0f), act);
            store_from_float(y, ((b * Cout + co0 + c) * Ho + oh) * (int64_t)Wo + ow, o);
        }
    }
}

// The stack's own first layer, 3 input channels and a 3x3 filter (27 inputs per output).  A thread owns two
// horizontally adjacent output pixels and kFcCo output channels: the 27 inputs of each pixel are loaded once into
// registers (zero outside the image); the weights are laid out [input][channel] in shared memory so that four channels
// come with one broadcast 16-byte load, which then feeds both pixels; two channels share one packed fp32 FMA
// (fma.rn.f32x2), so an output costs half an FMA-pipe instruction per input.  The pixel pair is stored as one
// 4-byte bf16 pair where the row length allows it (a warp then writes 128 contiguous bytes per channel).
constexpr int kFcN = 27;
constexpr int kFcCo = 32;

template <typename XT, typename YT>
__global__ void __launch_bounds__(128)
first_conv3x3_kernel(const XT *__restrict__ x, const float *__restrict__ w, const float *__restrict__ bias, YT *__restrict__ y,
                     int32_t Nb, int32_t H, int32_t Wd, int32_t Cout, int32_t stride, int32_t pad, int32_t Ho, int32_t Wo, int act)
{
    __shared__ __align__(16) float ws[kFcN * kFcCo];
    __shared__ __align__(8) float bs[kFcCo];
    const int32_t co0 = blockIdx.y * kFcCo;
    for (int32_t i = threadIdx.x; i < kFcN * kFcCo; i += blockDim.x) {
        const int32_t r = i / kFcCo, c = i - r * kFcCo;
        ws[i] = co0 + c < Cout ? __ldg(w + (int64_t)(co0 + c) * kFcN + r) : 0.0f;
    }
    if (threadIdx.x < kFcCo) bs[threadIdx.x] = (bias && co0 + (int)threadIdx.x < Cout) ? __ldg(bias + co0 + threadIdx.x) : 0.0f;
    __syncthreads();
    const int32_t Wp = (Wo + 1) >> 1;                       // pixel pairs per output row
    const int64_t items = (int64_t)Nb * Ho * Wp;
    const bool pair_store = (Wo & 1) == 0;
    // one item per thread (no grid-stride loop: the compiler would keep the loop-invariant weights in registers)
    const int64_t it = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (it < items) {
        const int32_t ow = (int32_t)(it % Wp) * 2;
        const int64_t t = it / Wp;
        const int32_t oh = (int32_t)(t % Ho);
        const int64_t b = t / Ho;
        float xin[2][kFcN];
#pragma unroll
        for (int px = 0; px < 2; ++px)
#pragma unroll
            for (int ci = 0; ci < 3; ++ci)
#pragma unroll
                for (int u = 0; u < 3; ++u)
#pragma unroll
                    for (int v = 0; v < 3; ++v) {
                        const int32_t ih = oh * stride + u - pad, iw = (ow + px) * stride + v - pad;
                        const bool in = ow + px < Wo && ih >= 0 && ih < H && iw >= 0 && iw < Wd;
                        xin[px][(ci * 3 + u) * 3 + v] = in ? load_as_float(x, ((b * 3 + ci) * H + ih) * (int64_t)Wd + iw) : 0.0f;
                    }
        uint64_t acc[2][kFcCo / 2];                         // [pixel][channel pair]
#pragma unroll
        for (int c = 0; c < kFcCo / 2; ++c) acc[0][c] = acc[1][c] = *reinterpret_cast<const uint64_t *>(&bs[2 * c]);
#pragma unroll
        for (int r = 0; r < kFcN; ++r) {
            const uint64_t x0 = f32x2_pack(xin[0][r], xin[0][r]), x1 = f32x2_pack(xin[1][r], xin[1][r]);
#pragma unroll
            for (int c = 0; c < kFcCo / 2; c += 2) {
                const ulonglong2 w4 = *reinterpret_cast<const ulonglong2 *>(&ws[r * kFcCo + 2 * c]);
                acc[0][c] = f32x2_fma(w4.x, x0, acc[0][c]);
                acc[0][c + 1] = f32x2_fma(w4.y, x0, acc[0][c + 1]);
                acc[1][c] = f32x2_fma(w4.x, x1, acc[1][c]);
                acc[1][c + 1] = f32x2_fma(w4.y, x1, acc[1][c + 1]);
            }
        }
#pragma unroll
        for (int c = 0; c < kFcCo; ++c) {
            if (co0 + c >= Cout) break;
            float p0lo, p0hi, p1lo, p1hi;
            f32x2_unpack(acc[0][c >> 1], p0lo, p0hi);
            f32x2_unpack(acc[1][c >> 1], p1lo, p1hi);
            const float o0 = apply_act((c & 1) ? p0hi : p0lo, act), o1 = apply_act((c & 1) ? p1hi : p1lo, act);
            const int64_t yi = ((b * Cout + co0 + c) * Ho + oh) * (int64_t)Wo + ow;
            if constexpr (sizeof(YT) == 2) {
                if (pair_store) {                               // yi is even: 4-byte aligned
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(o0, o1);
                    *reinterpret_cast<__nv_bfloat162 *>(y + yi) = h2;
                    continue;
                }
            }
            store_from_float(y, yi, o0);
            if (ow + 1 < Wo) store_from_float(y, yi + 1, o1);
        }
    }
}

// Mean over the H*W positions of every (image, channel) plane: one warp per plane, fp32 accumulation.
template <typename XT, typename YT>
__global__ void __launch_bounds__(256)
global_avgpool_kernel(const XT *__restrict__ x, int64_t planes, int32_t hw, YT *__restrict__ y)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t p = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; p < planes; p += warps) {
        float s = 0.0f;
        for (int32_t i = lane; i < hw; i += 32) s += load_as_float(x, p * hw + i);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) store_from_float(y, p, s / (float)hw);
    }
}

}  // namespace

// Global average pooling and a dense classifier in one launch: a block per image first leaves the C channel means (fp32) in
// shared memory, then its warps take the classes in turn (lanes split the channels, shuffle tree, bias added last).
constexpr int kPlMaxC = 4096;
template <typename XT>
__global__ void __launch_bounds__(256)
avgpool_linear_kernel(const XT *__restrict__ x, int32_t C, int32_t hw, const float *__restrict__ w, const float *__restrict__ bias,
                      int32_t out_f, float *__restrict__ y)
{
    __shared__ float pooled[kPlMaxC];
    const int64_t b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (sizeof(XT) == 2 && hw % 8 == 0 && hw <= 512 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0) {
        // short bf16 planes (a few 16-byte pieces): a thread per channel, 16-byte loads
        for (int32_t c = threadIdx.x; c < C; c += blockDim.x) {
            const uint4 *plane = reinterpret_cast<const uint4 *>(x + (b * C + c) * (int64_t)hw);
            float s = 0.0f;
            for (int32_t i = 0; i < hw / 8; ++i) {
                const uint4 u = __ldg(plane + i);
                const uint32_t wv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) s += __uint_as_float(wv[e] << 16) + __uint_as_float(wv[e] & 0xffff0000u);
            }
            pooled[c] = s / (float)hw;
        }
    } else
    // a warp per channel plane: consecutive lanes read consecutive positions
    for (int32_t c = warp; c < C; c += 8) {
        const XT *plane = x + (b * C + c) * (int64_t)hw;
        float s = 0.0f;
        for (int32_t i = lane; i < hw; i += 32) s += load_as_float(plane, i);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) pooled[c] = s / (float)hw;
    }
    __syncthreads();
    for (int32_t o = warp; o < out_f; o += 8) {
        const float *wr = w + (int64_t)o * C;
        float s = 0.0f;
        for (int32_t c = lane; c < C; c += 32) s = fmaf(__ldg(wr + c), pooled[c], s);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) y[b * out_f + o] = s + (bias ? __ldg(bias + o) : 0.0f);
    }
}

bool avgpool_linear_supported(int32_t C) { return C > 0 && C <= kPlMaxC; }

cudaError_t launch_avgpool_linear(const void *x, int x_dtype, int32_t Nb, int32_t C, int32_t hw, const float *w, const float *bias,
                                  int32_t out_f, float *y, cudaStream_t s)
{
    if (!avgpool_linear_supported(C)) return cudaErrorInvalidValue;
    if (x_dtype == TBN_BF16)
        avgpool_linear_kernel<<<(unsigned)Nb, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(x), C, hw, w, bias, out_f, y);
    else
        avgpool_linear_kernel<<<(unsigned)Nb, 256, 0, s>>>(static_cast<const float *>(x), C, hw, w, bias, out_f, y);
    return cudaGetLastError();
}

bool dense_conv_supported(int32_t Cin, int32_t kh, int32_t kw) { return (int64_t)Cin * kh * kw * kDcCo <= kDcMaxW; }

cudaError_t launch_dense_conv(const void *x, int x_dtype, const float *w, const float *bias, void *y, int y_dtype, int32_t Nb,
                              int32_t Cin, int32_t H, int32_t Wd, int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                              int act, cudaStream_t s)
{
    const int32_t Ho = (H + 2 * pad - kh) / stride + 1, Wo = (Wd + 2 * pad - kw) / stride + 1;
    const int64_t pixels = (int64_t)Nb * Ho * Wo;
    const int64_t bx = (pixels + 255) / 256;
    if (Cin == 3 && kh == 3 && kw == 3) {
        const int64_t pb = ((int64_t)Nb * Ho * ((Wo + 1) / 2) + 127) / 128;       // a thread owns two pixels
        if (pb > 0x7fffffffLL) return cudaErrorInvalidValue;
        const dim3 grid((unsigned)(pb > 0 ? pb : 1), (unsigned)((Cout + kFcCo - 1) / kFcCo));
#define TBN_FC(XT, YT) first_conv3x3_kernel<XT, YT><<<grid, 128, 0, s>>>(static_cast<const XT *>(x), w, bias, static_cast<YT *>(y), Nb, \
                                                                         H, Wd, Cout, stride, pad, Ho, Wo, act)
        if (x_dtype == TBN_BF16 && y_dtype == TBN_BF16) TBN_FC(__nv_bfloat16, __nv_bfloat16);
        else if (x_dtype == TBN_BF16) TBN_FC(__nv_bfloat16, float);
        else if (y_dtype == TBN_BF16) TBN_FC(float, __nv_bfloat16);
        else TBN_FC(float, float);
#undef TBN_FC
        return cudaGetLastError();
    }
    const dim3 grid((unsigned)(bx < 148 * 64 ? (bx > 0 ? bx : 1) : 148 * 64), (unsigned)((Cout + kDcCo - 1) / kDcCo));
#define TBN_DC(XT, YT) dense_conv_kernel<XT, YT><<<grid, 256, 0, s>>>(static_cast<const XT *>(x), w, bias, static_cast<YT *>(y), Nb, \
                                                                       Cin, H, Wd, Cout, kh, kw, stride, pad, Ho, Wo, act)
    if (x_dtype == TBN_BF16 && y_dtype == TBN_BF16) TBN_DC(__nv_bfloat16, __nv_bfloat16);
    else if (x_dtype == TBN_BF16) TBN_DC(__nv_bfloat16, float);
    else if (y_dtype == TBN_BF16) TBN_DC(float, __nv_bfloat16);
    else TBN_DC(float, float);
#undef TBN_DC
    return cudaGetLastError();
}

cudaError_t launch_global_avgpool(const void *x, int x_dtype, int64_t planes, int32_t hw, void *y, int y_dtype, cudaStream_t s)
{
    const int64_t bx = (planes + 7) / 8;
    const unsigned grid = (unsigned)(bx < 148 * 16 ? (bx > 0 ? bx : 1) : 148 * 16);
#define TBN_GAP(XT, YT) global_avgpool_kernel<XT, YT><<<grid, 256, 0, s>>>(static_cast<const XT *>(x), planes, hw, static_cast<YT *>(y))
    if (x_dtype == TBN_BF16 && y_dtype == TBN_BF16) TBN_GAP(__nv_bfloat16, __nv_bfloat16);
    else if (x_dtype == TBN_BF16) TBN_GAP(__nv_bfloat16, float);
    else if (y_dtype == TBN_BF16) TBN_GAP(float, __nv_bfloat16);
    else TBN_GAP(float, float);
#undef TBN_GAP
    return cudaGetLastError();
}

}  // namespace tbn
