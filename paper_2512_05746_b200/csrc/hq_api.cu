// Entry points that are not a kernel of their own: status helpers and the fused layer calls, which run
// transform+quantize (Eq. 10, Eq. 3) and then the integer product with its rescale (Eq. 12 / Eq. 14) on one stream.
#include <mutex>

#include "hq_common.cuh"

// Scratch of hq_qlinear_noalloc: part of the library's device image, one copy per GPU that loads the library.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char hq_noalloc_scratch[HQ_NOALLOC_SCRATCH_BYTES];

namespace hq {
hq_status launch_hadamard_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, int had_block,
                                int bits, hq_scale_mode mode, const float* static_scale, void* codes,
                                hq_container cont, int64_t ld_codes, float* scales, cudaStream_t st);
hq_status launch_qgemm(const void* a_codes, hq_container cont, int a_bits, int64_t M, int64_t K, int64_t lda,
                       const hq_weight_desc* desc, const void* w_dev, const float* scale_a, int scale_a_is_scalar,
                       const float* scale_w, const float* bias, float alpha, int32_t* acc_out, void* y,
                       hq_dtype ydt, int64_t ldy, int32_t* dev_status, cudaStream_t st, bool after_quant);
hq_status launch_qconv2d(const void* a_codes, hq_container cont, int a_bits, int64_t Nb, int64_t H, int64_t W,
                         int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                         const float* scale_a, int scale_a_is_scalar, const float* scale_w, const float* bias,
                         float alpha, int32_t* acc_out, void* y, hq_dtype ydt, int32_t* dev_status, cudaStream_t st,
                         bool after_quant);

hq_status launch_gn_silu_quant(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups,
                               const float* gamma, const float* beta, float eps, int had_block, int bits,
                               hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont,
                               int64_t ld_codes, float* scales, void* scratch, size_t scratch_bytes, cudaStream_t st,
                               int silu, const void* pre_bias, const void* x2, int64_t split);
hq_status launch_hadamard_quant_cat(const void* x, int64_t ldx, const void* x2, int64_t ldx2, int64_t split, hq_dtype xdt,
                                    int64_t rows, int64_t cols, int had_block, int bits, hq_scale_mode mode,
                                    const float* static_scale, void* codes, hq_container cont, int64_t ld_codes,
                                    float* scales, cudaStream_t st);
hq_status launch_ln_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, const float* weight,
                          const float* bias, int64_t rows_per_group, float eps, int had_block, int bits,
                          hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont, int64_t ld_codes,
                          float* scales, cudaStream_t st);
hq_status launch_hadamard_quant_width(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                      int had_block_w, int bits, const float* static_scale, void* z, float* scale_out,
                                      cudaStream_t st);
hq_status launch_hadamard_quant_width2(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                       int had_block_w, int bits, const float* static_scale, void* z_limbs,
                                       float* scale_out, cudaStream_t st);

namespace {
int64_t code_pitch(int64_t cols, hq_container cont) {
    const int64_t b = cont == HQ_CODES_NIBBLE ? cols / 2 : cols;
    return (b + 15) / 16 * 16;
}
int64_t scales_offset(int64_t rows, int64_t cols, hq_container cont) {
    return (rows * code_pitch(cols, cont) + 255) / 256 * 256;
}
}  // namespace
}  // namespace hq

extern "C" int hq_version(void) { return 100; }

extern "C" const char* hq_status_string(hq_status s) {
    switch (s) {
        case HQ_OK: return "ok";
        case HQ_ERR_INVALID_ARG: return "invalid argument";
        case HQ_ERR_SHAPE: return "inconsistent shape";
        case HQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case HQ_ERR_ALIGNMENT: return "misaligned pointer or pitch";
        case HQ_ERR_WORKSPACE: return "workspace too small";
        case HQ_ERR_OVERFLOW_RISK: return "int32 accumulator could overflow";
        case HQ_ERR_CUDA: return "CUDA call failed";
        case HQ_ERR_TIMEOUT: return "device-side wait timed out";
        case HQ_ERR_SCRATCH_LIMIT: return "layer exceeds the built-in scratch of the no-allocation entry point";
    }
    return "unknown status";
}

extern "C" hq_status hq_check_status(const int32_t* dev_status_host_copy) {
    if (dev_status_host_copy == nullptr) return HQ_ERR_INVALID_ARG;
    return *dev_status_host_copy == 0 ? HQ_OK : HQ_ERR_TIMEOUT;
}

extern "C" hq_status hq_workspace_size(int64_t rows, int64_t cols, hq_container cont, size_t* bytes) {
    if (bytes == nullptr) return HQ_ERR_INVALID_ARG;
    if (cont != HQ_CODES_NIBBLE && cont != HQ_CODES_INT8) return HQ_ERR_INVALID_ARG;
    if (rows < 0 || cols <= 0) return HQ_ERR_SHAPE;
    *bytes = size_t(hq::scales_offset(rows, cols, cont)) + size_t(rows > 0 ? rows : 1) * sizeof(float);
    return HQ_OK;
}

extern "C" hq_status hq_qlinear(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx,
                                const hq_weight_desc* desc, const void* w_dev, const float* scale_w,
                                const float* bias, int a_bits, hq_scale_mode mode, const float* static_scale, void* y,
                                hq_dtype ydt, int64_t ldy, void* workspace, size_t ws_bytes, int32_t* dev_status,
                                void* stream) {
    using namespace hq;
    if (desc == nullptr || workspace == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
    const hq_container cont = hq_container(desc->container);
    size_t need = 0;
    hq_status s = hq_workspace_size(M, K, cont, &need);
    if (s != HQ_OK) return s;
    if (ws_bytes < need) return HQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* codes = static_cast<unsigned char*>(workspace);
    float* scales = reinterpret_cast<float*>(codes + scales_offset(M, K, cont));
    const int64_t ldc = code_pitch(K, cont);
    s = launch_hadamard_quant(x, xdt, M, K, ldx, desc->had_block, a_bits, mode, static_scale, codes, cont, ldc, scales, st);
    if (s != HQ_OK) return s;
    return launch_qgemm(codes, cont, a_bits, M, K, ldc, desc, w_dev, scales, mode == HQ_SCALE_STATIC, scale_w, bias,
                        hq_alpha_for(desc), nullptr, y, ydt, ldy, dev_status, st, true);
}

extern "C" hq_status hq_ln_qlinear(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx, const float* ln_weight,
                                   const float* ln_bias, int64_t rows_per_group, float eps, const hq_weight_desc* desc,
                                   const void* w_dev, const float* scale_w, const float* bias, int a_bits, void* y,
                                   hq_dtype ydt, int64_t ldy, void* workspace, size_t ws_bytes, int32_t* dev_status,
                                   void* stream) {
    using namespace hq;
    if (desc == nullptr || workspace == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
    const hq_container cont = hq_container(desc->container);
    size_t need = 0;
    hq_status s = hq_workspace_size(M, K, cont, &need);
    if (s != HQ_OK) return s;
    if (ws_bytes < need) return HQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* codes = static_cast<unsigned char*>(workspace);
    float* scales = reinterpret_cast<float*>(codes + scales_offset(M, K, cont));
    const int64_t ldc = code_pitch(K, cont);
    s = launch_ln_quant(x, xdt, M, K, ldx, ln_weight, ln_bias, rows_per_group, eps, desc->had_block, a_bits, HQ_SCALE_PER_ROW,
                        nullptr, codes, cont, ldc, scales, st);
    if (s != HQ_OK) return s;
    return launch_qgemm(codes, cont, a_bits, M, K, ldc, desc, w_dev, scales, 0, scale_w, bias, hq_alpha_for(desc), nullptr,
                        y, ydt, ldy, dev_status, st, true);
}

static hq_status gn_silu_qconv_impl(const void* x, const void* x2, int64_t split, hq_dtype xdt, int64_t Nb, int64_t H,
                                    int64_t W, int64_t C, int groups,
                                      const float* gamma, const float* beta, const void* pre_bias, float eps,
                                      const hq_weight_desc* desc,
                                      const void* w_dev, int R, int S, int stride, int pad, const float* scale_w,
                                      const float* bias, int a_bits, hq_scale_mode mode, const float* static_scale, void* y,
                                      hq_dtype ydt, void* workspace, size_t ws_bytes, void* scratch, size_t scratch_bytes,
                                      int32_t* dev_status, void* stream) {
    using namespace hq;
    if (desc == nullptr || workspace == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
    const hq_container cont = hq_container(desc->container);
    const int64_t rows = Nb * H * W;
    size_t need = 0;
    hq_status s = hq_workspace_size(rows, C, cont, &need);
    if (s != HQ_OK) return s;
    if (ws_bytes < need) return HQ_ERR_WORKSPACE;
    const int64_t ldc = code_pitch(C, cont);
    if (ldc != (cont == HQ_CODES_NIBBLE ? C / 2 : C)) return HQ_ERR_ALIGNMENT;   // conv needs densely packed pixels
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* codes = static_cast<unsigned char*>(workspace);
    float* scales = reinterpret_cast<float*>(codes + scales_offset(rows, C, cont));
    s = launch_gn_silu_quant(x, xdt, Nb, H, W, C, groups, gamma, beta, eps, desc->had_block, a_bits, mode, static_scale, codes,
                             cont, ldc, scales, scratch, scratch_bytes, st, 1, pre_bias, x2, split);
    if (s != HQ_OK) return s;
    return launch_qconv2d(codes, cont, a_bits, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scales,
                          mode == HQ_SCALE_STATIC, scale_w, bias, hq_alpha_for(desc), nullptr, y, ydt, dev_status, st, true);
}

extern "C" hq_status hq_gn_silu_qconv(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups,
                                      const float* gamma, const float* beta, const void* pre_bias, float eps,
                                      const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                                      const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                                      const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                                      void* scratch, size_t scratch_bytes, int32_t* dev_status, void* stream) {
    return gn_silu_qconv_impl(x, nullptr, 0, xdt, Nb, H, W, C, groups, gamma, beta, pre_bias, eps, desc, w_dev, R, S, stride,
                              pad, scale_w, bias, a_bits, mode, static_scale, y, ydt, workspace, ws_bytes, scratch,
                              scratch_bytes, dev_status, stream);
}

// The same layer on the channel concatenation of two NHWC tensors (x: channels [0, C1), x2: channels [C1, C)), read in
// place: a skip connection joined to the up-sampling path without the concatenated tensor being written.
extern "C" hq_status hq_gn_silu_qconv_cat(const void* x, const void* x2, int64_t C1, hq_dtype xdt, int64_t Nb, int64_t H,
                                          int64_t W, int64_t C, int groups, const float* gamma, const float* beta,
                                          const void* pre_bias, float eps, const hq_weight_desc* desc, const void* w_dev,
                                          int R, int S, int stride, int pad, const float* scale_w, const float* bias,
                                          int a_bits, hq_scale_mode mode, const float* static_scale, void* y, hq_dtype ydt,
                                          void* workspace, size_t ws_bytes, void* scratch, size_t scratch_bytes,
                                          int32_t* dev_status, void* stream) {
    if (x2 == nullptr) return HQ_ERR_INVALID_ARG;
    return gn_silu_qconv_impl(x, x2, C1, xdt, Nb, H, W, C, groups, gamma, beta, pre_bias, eps, desc, w_dev, R, S, stride, pad,
                              scale_w, bias, a_bits, mode, static_scale, y, ydt, workspace, ws_bytes, scratch, scratch_bytes,
                              dev_status, stream);
}

// The fused linear layer on the pixels of an NHWC tensor with GroupNorm (optionally + SiLU) in front: the QKV
// projection of an attention block, whose input is the normalised feature map.  Rows = Nb * rows_per_sample pixels.
extern "C" hq_status hq_gn_qlinear(const void* x, hq_dtype xdt, int64_t Nb, int64_t rows_per_sample, int64_t C, int groups,
                                   const float* gamma, const float* beta, float eps, int silu, const hq_weight_desc* desc,
                                   const void* w_dev, const float* scale_w, const float* bias, int a_bits, void* y,
                                   hq_dtype ydt, int64_t ldy, void* workspace, size_t ws_bytes, void* scratch,
                                   size_t scratch_bytes, int32_t* dev_status, void* stream) {
    using namespace hq;
    if (desc == nullptr || workspace == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
    if (Nb <= 0 || rows_per_sample <= 0) return HQ_ERR_SHAPE;
    const hq_container cont = hq_container(desc->container);
    const int64_t M = Nb * rows_per_sample;
    size_t need = 0;
    hq_status s = hq_workspace_size(M, C, cont, &need);
    if (s != HQ_OK) return s;
    if (ws_bytes < need) return HQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* codes = static_cast<unsigned char*>(workspace);
    float* scales = reinterpret_cast<float*>(codes + scales_offset(M, C, cont));
    const int64_t ldc = code_pitch(C, cont);
    s = launch_gn_silu_quant(x, xdt, Nb, rows_per_sample, 1, C, groups, gamma, beta, eps, desc->had_block, a_bits,
                             HQ_SCALE_PER_ROW, nullptr, codes, cont, ldc, scales, scratch, scratch_bytes, st, silu != 0,
                             nullptr, nullptr, 0);
    if (s != HQ_OK) return s;
    return launch_qgemm(codes, cont, a_bits, M, C, ldc, desc, w_dev, scales, 0, scale_w, bias, hq_alpha_for(desc), nullptr,
                        y, ydt, ldy, dev_status, st, true);
}

static hq_status qconv_impl(const void* x, const void* x2, int64_t split, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W,
                            int64_t C,
                              const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                              const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                              const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                              int32_t* dev_status, void* stream) {
    using namespace hq;
    if (desc == nullptr || workspace == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
    const hq_container cont = hq_container(desc->container);
    const int64_t rows = Nb * H * W;
    size_t need = 0;
    hq_status s = hq_workspace_size(rows, C, cont, &need);
    if (s != HQ_OK) return s;
    if (ws_bytes < need) return HQ_ERR_WORKSPACE;
    const int64_t ldc = code_pitch(C, cont);
    if (ldc != (cont == HQ_CODES_NIBBLE ? C / 2 : C)) return HQ_ERR_ALIGNMENT;   // conv needs densely packed pixels
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* codes = static_cast<unsigned char*>(workspace);
    float* scales = reinterpret_cast<float*>(codes + scales_offset(rows, C, cont));
    if (x2 != nullptr)
        s = launch_hadamard_quant_cat(x, split, x2, C - split, split, xdt, rows, C, desc->had_block, a_bits, mode, static_scale,
                                      codes, cont, ldc, scales, st);
    else
        s = launch_hadamard_quant(x, xdt, rows, C, C, desc->had_block, a_bits, mode, static_scale, codes, cont, ldc, scales, st);
    if (s != HQ_OK) return s;
    return launch_qconv2d(codes, cont, a_bits, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scales,
                          mode == HQ_SCALE_STATIC, scale_w, bias, hq_alpha_for(desc), nullptr, y, ydt, dev_status, st, true);
}

extern "C" hq_status hq_qconv(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                              const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                              const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                              const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                              int32_t* dev_status, void* stream) {
    return qconv_impl(x, nullptr, 0, xdt, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scale_w, bias, a_bits, mode,
                      static_scale, y, ydt, workspace, ws_bytes, dev_status, stream);
}

// The fused convolution layer on the channel concatenation of two NHWC tensors read in place (see hq_gn_silu_qconv_cat).
extern "C" hq_status hq_qconv_cat(const void* x, const void* x2, int64_t C1, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W,
                                  int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride,
                                  int pad, const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                                  const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                                  int32_t* dev_status, void* stream) {
    if (x2 == nullptr) return HQ_ERR_INVALID_ARG;
    return qconv_impl(x, x2, C1, xdt, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scale_w, bias, a_bits, mode, static_scale,
                      y, ydt, workspace, ws_bytes, dev_status, stream);
}

// Convolution exactly as Eq. 13-14 state it: transform along the width axis, quantization with one static scale,
// integer factor q * H_raw, integer convolution with untransformed (PLAIN, one-limb, INT8-container) weights.
// The int8 activations z and the scale S * 2^(-k/2) live in `workspace` (hq_workspace_size(Nb*H*W, C, INT8)).
extern "C" hq_status hq_qconv_width(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                    const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                                    const float* scale_w, const float* bias, int a_bits, int had_block_w,
                                    const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                                    int32_t* dev_status, void* stream) {
    using namespace hq;
    if (desc == nullptr || workspace == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (desc->mode == HQ_W_PLAIN_A2) {
        // blocks wider than a signed byte allows: z travels as two int8 limbs per channel, [hi(C) | lo(C)] per pixel,
        // and meets weights whose "hi" rows are [Q(W) | 0] and "lo" rows [0 | Q(W)] in the two-limb product
        if (desc->limbs != 2 || desc->container != HQ_CODES_INT8 || desc->C != 2 * C) return HQ_ERR_SHAPE;
        if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
        const int64_t rows2 = Nb * H * W;
        size_t need2 = 0;
        hq_status s2 = hq_workspace_size(rows2, 2 * C, HQ_CODES_INT8, &need2);
        if (s2 != HQ_OK) return s2;
        if (ws_bytes < need2) return HQ_ERR_WORKSPACE;
        if ((2 * C) % 16 != 0) return HQ_ERR_ALIGNMENT;
        cudaStream_t st2 = static_cast<cudaStream_t>(stream);
        unsigned char* z2 = static_cast<unsigned char*>(workspace);
        float* scale2 = reinterpret_cast<float*>(z2 + scales_offset(rows2, 2 * C, HQ_CODES_INT8));
        s2 = launch_hadamard_quant_width2(x, xdt, Nb, H, W, C, had_block_w, a_bits, static_scale, z2, scale2, st2);
        if (s2 != HQ_OK) return s2;
        return launch_qconv2d(z2, HQ_CODES_INT8, 8, Nb, H, W, 2 * C, desc, w_dev, R, S, stride, pad, scale2, 1, scale_w, bias,
                              1.0f, nullptr, y, ydt, dev_status, st2, true);
    }
    if (desc->mode != HQ_W_PLAIN || desc->limbs != 1 || desc->container != HQ_CODES_INT8) return HQ_ERR_SHAPE;
    if (!aligned16(workspace)) return HQ_ERR_ALIGNMENT;
    const int64_t rows = Nb * H * W;
    size_t need = 0;
    hq_status s = hq_workspace_size(rows, C, HQ_CODES_INT8, &need);
    if (s != HQ_OK) return s;
    if (ws_bytes < need) return HQ_ERR_WORKSPACE;
    if (C % 16 != 0) return HQ_ERR_ALIGNMENT;              // densely packed pixels for the convolution's TMA boxes
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* z = static_cast<unsigned char*>(workspace);
    float* scale = reinterpret_cast<float*>(z + scales_offset(rows, C, HQ_CODES_INT8));
    s = launch_hadamard_quant_width(x, xdt, Nb, H, W, C, had_block_w, a_bits, static_scale, z, scale, st);
    if (s != HQ_OK) return s;
    // |z| <= 128: the accumulator bound is that of 8-bit codes; the 2^(-k/2) is already inside `scale`
    return launch_qconv2d(z, HQ_CODES_INT8, 8, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scale, 1, scale_w, bias, 1.0f,
                          nullptr, y, ydt, dev_status, st, true);
}

namespace hq {
namespace {
// Device address of hq_noalloc_scratch on the current device, looked up once per device.
hq_status noalloc_scratch_address(unsigned char** out) {
    static std::mutex mu;
    static unsigned char* addr[64] = {};
    int dev = 0;
    HQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return HQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, hq_noalloc_scratch) != cudaSuccess || p == nullptr) return HQ_ERR_CUDA;
        addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = addr[dev];
    return HQ_OK;
}
}  // namespace
}  // namespace hq

// hq_qlinear for callers that cannot allocate: the codes and scales between the two kernels go to the library's
// own fixed device array (shared by all calls on a device, contents left over from the previous call, fully
// overwritten before they are read).  The first call per device resolves the array's address.
extern "C" hq_status hq_qlinear_noalloc(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx,
                                        const hq_weight_desc* desc, const void* w_dev, const float* scale_w,
                                        const float* bias, int a_bits, hq_scale_mode mode, const float* static_scale,
                                        void* y, hq_dtype ydt, int64_t ldy, int32_t* dev_status, void* stream) {
    using namespace hq;
    if (desc == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    const hq_container cont = hq_container(desc->container);
    size_t need = 0;
    hq_status s = hq_workspace_size(M, K, cont, &need);
    if (s != HQ_OK) return s;
    if (need > size_t(HQ_NOALLOC_SCRATCH_BYTES)) return HQ_ERR_SCRATCH_LIMIT;
    unsigned char* codes = nullptr;
    s = noalloc_scratch_address(&codes);
    if (s != HQ_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* scales = reinterpret_cast<float*>(codes + scales_offset(M, K, cont));
    const int64_t ldc = code_pitch(K, cont);
    s = launch_hadamard_quant(x, xdt, M, K, ldx, desc->had_block, a_bits, mode, static_scale, codes, cont, ldc, scales, st);
    if (s != HQ_OK) return s;
    return launch_qgemm(codes, cont, a_bits, M, K, ldc, desc, w_dev, scales, mode == HQ_SCALE_STATIC, scale_w, bias,
                        hq_alpha_for(desc), nullptr, y, ydt, ldy, dev_status, st, true);
}
