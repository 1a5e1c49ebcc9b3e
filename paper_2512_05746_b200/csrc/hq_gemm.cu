// Integer GEMM / implicit-GEMM convolution with a fused rescale epilogue (Eq. 12, Eq. 14).
//
//   acc[m][o] = sum_k a[m][k] * B[o][k]   int8 x int8 -> int32 on the 5th-generation tensor cores
//   y[m][o]   = alpha * S_a[m] * S_w[o] * acc[m][o] + bias[o]
//
// Host side: argument checks, tensor maps, shared-memory planning and the choice of kernel instantiation.  The kernel
// itself (one persistent CTA per SM walking output tiles of 128 rows x 256 operand rows, warp-specialised into a TMA
// producer, one or two MMA issuers, eight epilogue warps and, for the nibble container, four unpack warps) is in
// hq_gemm_kernel.cuh; hq_gemm_inst_*.cu instantiate it per container and problem kind.
// Weights: when the whole reduction fits (K_pad <= 512 bytes per operand row, 128 KB per tile) the weight tile
// stays resident in shared memory and the CTA walks a contiguous range of row tiles under it (only activations
// stream); otherwise weights stream through the same ring as the activations.
// Every wait is bounded; on expiry a status word is written and the CTA drains and exits.
#include <cuda.h>

#include <cmath>

#include "hq_gemm_kernel.cuh"

namespace hq {
using namespace gemm;

// hq_gemm_pair.cu: the same product on pairs of SMs (tcgen05.mma.cta_group::2) for the shapes it covers
bool pair_kernel_covers(hq_container cont, const hq_weight_desc* desc, int64_t M, const void* y, hq_dtype ydt, int64_t ldy,
                        const int32_t* acc_out, bool combine_fast);
hq_status launch_qgemm_pair(const void* a_codes, int64_t M, int64_t K, int64_t lda, const hq_weight_desc* desc,
                            const void* w_dev, const float* scale_a, int scale_a_is_scalar, const float* scale_w,
                            const float* bias, float alpha, void* y, int64_t ldy, int32_t* dev_status, cudaStream_t st,
                            bool after_quant);
bool pair_kernel_pays(const hq_weight_desc* desc, int64_t M);
bool pair_stream_covers_gemm(hq_container cont, const hq_weight_desc* desc, int64_t M, const void* y, hq_dtype ydt, int64_t ldy,
                             const int32_t* acc_out, bool combine_fast);
bool pair_stream_covers_conv(hq_container cont, const gemm::GemmParams& g);
hq_status launch_qgemm_pair_stream(const void* a_codes, int64_t M, int64_t K, int64_t lda, const hq_weight_desc* desc,
                                   const void* w_dev, const float* scale_a, int scale_a_is_scalar, const float* scale_w,
                                   const float* bias, float alpha, void* y, int64_t ldy, int32_t* dev_status, cudaStream_t st,
                                   bool after_quant);
hq_status launch_qconv_pair(const gemm::GemmParams& g, const CUtensorMap& tmA, const CUtensorMap& tmY,
                            const hq_weight_desc* desc, const void* w_dev, cudaStream_t st);
int g_pair_gemm = 2;       // hq_set_pair_gemm: 0 never, 1 wherever the pair kernels cover, 2 where they measured faster

namespace {

// ---- issue-rate probe: back-to-back MMAs on resident tiles ---------------------------------------------
__global__ void __launch_bounds__(128, 1) mma_probe_kernel(int iters, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t done_bar;
    __shared__ uint32_t tmem_slot;
    for (int i = threadIdx.x; i < (kABytes + kBBytes) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u;
    if (threadIdx.x == 0) { mbar_init(&done_bar, 1); fence_barrier_init(); }
    fence_proxy_async_smem();
    if (threadIdx.x < 32) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    if (threadIdx.x == 0) {
        const uint32_t idesc = make_idesc_i8(kBM, kBN);
        const uint64_t a_desc = make_sw128_kmajor_desc(smem_u32(smem));
        const uint64_t b_desc = make_sw128_kmajor_desc(smem_u32(smem + kABytes));
        for (int i = 0; i < iters; ++i)
            mma_i8(tmem_base, a_desc + uint64_t((i & 3) * 2), b_desc + uint64_t((i & 3) * 2), idesc, i != 0 ? 1u : 0u);
        mma_commit(&done_bar);
        mbar_wait(&done_bar, 0, dev_status, kStatusAccumWait);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem_base, 256);
}

}  // namespace

// ---- host side ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// A tensor map is a pure function of the arguments it is encoded from (address, extents, pitch, box, swizzle), so the
// encoded 128 bytes are kept per calling thread in a small direct-mapped table keyed by those arguments: a layer that
// is called again on the same buffers (every step of a sampler) pays for a lookup and a copy instead of three driver
// calls, which matters for the few-row layers whose kernels are as short as their host-side set-up.
struct TmapKey {
    uint64_t v[8];
    bool operator==(const TmapKey& o) const {
        for (int i = 0; i < 8; ++i)
            if (v[i] != o.v[i]) return false;
        return true;
    }
};
struct TmapSlot { TmapKey key; CUtensorMap map; bool used; };
constexpr int kTmapSlots = 512;

template <typename Encode>
bool cached_tensor_map(CUtensorMap* tm, const TmapKey& key, Encode&& encode) {
    static thread_local TmapSlot table[kTmapSlots] = {};
    uint64_t h = 0x9E3779B97F4A7C15ull;
    for (int i = 0; i < 8; ++i) h = (h ^ key.v[i]) * 0xFF51AFD7ED558CCDull + (h >> 29);
    TmapSlot& slot = table[(h >> 20) % kTmapSlots];
    if (slot.used && slot.key == key) {
        *tm = slot.map;
        return true;
    }
    if (!encode(tm)) return false;
    slot.key = key;
    slot.map = *tm;
    slot.used = true;
    return true;
}

bool encode_2d(CUtensorMap* tm, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
               uint32_t box_inner, uint32_t box_rows, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const TmapKey key{{1, reinterpret_cast<uint64_t>(base), inner_bytes, rows, pitch_bytes,
                       (uint64_t(box_inner) << 32) | box_rows, uint64_t(swizzle128), 0}};
    return cached_tensor_map(tm, key, [&](CUtensorMap* out) {
        cuuint64_t dims[2] = {inner_bytes, rows};
        cuuint64_t strides[1] = {pitch_bytes};
        cuuint32_t box[2] = {box_inner, box_rows};
        cuuint32_t estr[2] = {1, 1};
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

bool encode_4d(CUtensorMap* tm, const void* base, const uint64_t dims_in[4], const uint32_t box_in[4],
               const uint32_t estr_in[4], bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    // boxes and element strides are small numbers: 16 bits each in the key
    const TmapKey key{{3, reinterpret_cast<uint64_t>(base), dims_in[0], dims_in[1], dims_in[2], dims_in[3],
                       (uint64_t(box_in[0]) << 48) | (uint64_t(box_in[1]) << 32) | (uint64_t(box_in[2]) << 16) | box_in[3],
                       (uint64_t(estr_in[0]) << 48) | (uint64_t(estr_in[1]) << 32) | (uint64_t(estr_in[2]) << 16) |
                           (uint64_t(estr_in[3]) << 1) | uint64_t(swizzle128)}};
    return cached_tensor_map(tm, key, [&](CUtensorMap* out) {
        cuuint64_t dims[4] = {dims_in[0], dims_in[1], dims_in[2], dims_in[3]};
        cuuint64_t strides[3] = {dims_in[0], dims_in[0] * dims_in[1], dims_in[0] * dims_in[1] * dims_in[2]};
        cuuint32_t box[4] = {box_in[0], box_in[1], box_in[2], box_in[3]};
        cuuint32_t estr[4] = {estr_in[0], estr_in[1], estr_in[2], estr_in[3]};
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// bf16 matrix [rows][cols] with a row pitch, boxes of box_rows x 64 columns (128 bytes) in the 128-byte swizzle: the
// operand tiles of the attention kernel.
bool encode_2d_bf16_sw128(CUtensorMap* tm, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                          uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const TmapKey key{{4, reinterpret_cast<uint64_t>(base), cols, rows, pitch_bytes, box_rows, 0, 0}};
    return cached_tensor_map(tm, key, [&](CUtensorMap* out) {
        cuuint64_t dims[2] = {cols, rows};
        cuuint64_t strides[1] = {pitch_bytes};
        cuuint32_t box[2] = {64, box_rows};
        cuuint32_t estr[2] = {1, 1};
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Output tensor map for the epilogue's bulk stores: bf16 [rows][N] with pitch ldy, boxes of 32 rows x 32 columns
// in the 64-byte swizzle the staging buffers are written in.
bool encode_y(CUtensorMap* tm, const void* y, uint64_t N, uint64_t rows, uint64_t ldy) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const TmapKey key{{2, reinterpret_cast<uint64_t>(y), N, rows, ldy, 0, 0, 0}};
    return cached_tensor_map(tm, key, [&](CUtensorMap* out) {
        cuuint64_t dims[2] = {N, rows};
        cuuint64_t strides[1] = {ldy * 2};
        cuuint32_t box[2] = {32, 32};
        cuuint32_t estr[2] = {1, 1};
        return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(y), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

// Ring depth and weight residency for a problem; fills p.stages / p.b_resident and returns the shared-memory size.
size_t plan_smem(GemmParams& p, bool frag) {
    const int num_kb = p.kb_per_tap * p.taps;
    p.b_resident = num_kb <= kResidentKb ? 1 : 0;
    for (int stages = kMaxStages; stages >= 2; --stages) {
        const SmemLayout L = smem_layout(stages, p.b_resident != 0, num_kb, frag);
        if (L.total <= kSmemLimit) { p.stages = stages; return size_t(L.total); }
    }
    return 0;
}

hq_status launch(bool nibble, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY, GemmParams& p,
                 cudaStream_t st) {
    // the kernel's fast epilogue assumes exactly these conditions
    const bool fast = p.tma_store && !p.per_tap && p.y != nullptr && p.acc_out == nullptr && p.combine_fast;
    const int mode = p.per_tap ? kModePerTap : fast ? kModeFast : kModeGeneric;
    p.frag = use_frag(nibble, fast, p.limbs, p.kb_per_tap * p.taps) ? 1 : 0;
    const size_t smem = plan_smem(p, p.frag != 0);
    if (smem == 0) return HQ_ERR_UNSUPPORTED;
    const int tiles = p.tiles_m * p.tiles_n;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    cudaError_t e;
    if (nibble) e = p.conv ? launch_nibble_conv(mode, grid, smem, st, tmA, tmB, tmY, p)
                           : launch_nibble_gemm(mode, grid, smem, st, tmA, tmB, tmY, p);
    else e = p.conv ? launch_i8_conv(mode, grid, smem, st, tmA, tmB, tmY, p)
                    : launch_i8_gemm(mode, grid, smem, st, tmA, tmB, tmY, p);
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

// Epilogue settings shared by the GEMM and the convolution.
void fill_epilogue(GemmParams& p, hq_container cont, int a_bits, const hq_weight_desc* desc, int64_t K_total,
                   const float* scale_a, int scale_a_is_scalar, const float* scale_w, const float* bias, float alpha,
                   int32_t* acc_out, void* y, hq_dtype ydt, int64_t ldy, int32_t* dev_status) {
    p.a_shift = cont == HQ_CODES_NIBBLE ? 4 : 0;
    // 256*hi + lo (one limb: the accumulator itself) of the shifted accumulators is (true value) << a_shift
    const double bound = double(K_total) * double(1 << (a_bits - 1)) * double(desc->max_abs_b > 0 ? desc->max_abs_b : 1);
    p.combine_fast = bound * double(1 << p.a_shift) < 2147483648.0 ? 1 : 0;
    p.scale_a = scale_a; p.sa_scalar = scale_a_is_scalar; p.scale_w = scale_w; p.bias = bias; p.alpha = alpha;
    p.acc_out = acc_out; p.y = y; p.y_bf16 = ydt == HQ_BF16; p.ldy = ldy; p.dev_status = dev_status;
    const int yelt = ydt == HQ_BF16 ? 2 : 4;
    p.y_vec_ok = y != nullptr && aligned16(y) && (ldy * yelt) % 16 == 0;
    p.acc_vec_ok = acc_out != nullptr && aligned16(acc_out) && (int64_t(desc->N) * 4) % 16 == 0;
}

hq_status check_common(const void* a_codes, hq_container cont, int a_bits, const hq_weight_desc* desc,
                       const void* w_dev, const float* scale_a, const float* scale_w, int32_t* acc_out, void* y,
                       hq_dtype ydt, int64_t K_total) {
    if (a_codes == nullptr || desc == nullptr || w_dev == nullptr) return HQ_ERR_INVALID_ARG;
    if (cont != HQ_CODES_NIBBLE && cont != HQ_CODES_INT8) return HQ_ERR_INVALID_ARG;
    if (a_bits != 3 && a_bits != 4 && a_bits != 8) return HQ_ERR_INVALID_ARG;
    if (cont == HQ_CODES_NIBBLE && a_bits > 4) return HQ_ERR_SHAPE;
    if (int(cont) != desc->container) return HQ_ERR_SHAPE;
    if (acc_out == nullptr && y == nullptr) return HQ_ERR_INVALID_ARG;
    if (y != nullptr && (scale_a == nullptr || scale_w == nullptr)) return HQ_ERR_INVALID_ARG;
    if (ydt != HQ_F32 && ydt != HQ_BF16) return HQ_ERR_INVALID_ARG;
    if (desc->limbs != 1 && desc->limbs != 2) return HQ_ERR_INVALID_ARG;
    if (!aligned16(a_codes) || !aligned16(w_dev)) return HQ_ERR_ALIGNMENT;
    // |acc| <= K * 2^(a_bits-1) * max|B| must stay below 2^31 (also per limb after the x16 of the nibble path).
    const double bound = double(K_total) * double(1 << (a_bits - 1)) * double(desc->max_abs_b > 0 ? desc->max_abs_b : 1);
    if (bound >= 2147483648.0) return HQ_ERR_OVERFLOW_RISK;
    if (cont == HQ_CODES_NIBBLE && double(K_total) * 8.0 * 16.0 * 128.0 >= 2147483648.0) return HQ_ERR_OVERFLOW_RISK;
    return HQ_OK;
}

}  // namespace

hq_status launch_qgemm(const void* a_codes, hq_container cont, int a_bits, int64_t M, int64_t K, int64_t lda,
                       const hq_weight_desc* desc, const void* w_dev, const float* scale_a, int scale_a_is_scalar,
                       const float* scale_w, const float* bias, float alpha, int32_t* acc_out, void* y,
                       hq_dtype ydt, int64_t ldy, int32_t* dev_status, cudaStream_t st, bool after_quant) {
    hq_status s = check_common(a_codes, cont, a_bits, desc, w_dev, scale_a, scale_w, acc_out, y, ydt, K);
    if (s != HQ_OK) return s;
    if (desc->RS != 1 || desc->C != K) return HQ_ERR_SHAPE;
    if (M < 0 || K <= 0) return HQ_ERR_SHAPE;
    const int64_t row_bytes = cont == HQ_CODES_NIBBLE ? K / 2 : K;
    if (lda < row_bytes) return HQ_ERR_SHAPE;
    if (lda % 16 != 0) return HQ_ERR_ALIGNMENT;
    if (y != nullptr && ldy < desc->N) return HQ_ERR_SHAPE;
    if (M == 0) return HQ_OK;
    if (M > (int64_t(1) << 30)) return HQ_ERR_UNSUPPORTED;

    GemmParams p{};
    p.M = M; p.N = int(desc->N); p.limbs = desc->limbs;
    p.kb_per_tap = int(desc->C_pad / kBK); p.taps = 1;
    p.tiles_m = int((M + kBM - 1) / kBM);
    p.tiles_n = int(desc->limbs == 2 ? desc->N_pad / 128 : (desc->N_pad + 255) / 256);
    p.a_box_bytes = cont == HQ_CODES_NIBBLE ? kRawBytes : kABytes;
    p.conv = 0;
    p.pdl = after_quant ? 1 : 0;
    fill_epilogue(p, cont, a_bits, desc, K, scale_a, scale_a_is_scalar, scale_w, bias, alpha, acc_out, y, ydt, ldy,
                  dev_status);

    if (g_pair_gemm && pair_kernel_covers(cont, desc, M, y, ydt, ldy, acc_out, p.combine_fast != 0) &&
        (g_pair_gemm == 1 || pair_kernel_pays(desc, M)))
        return launch_qgemm_pair(a_codes, M, K, lda, desc, w_dev, scale_a, scale_a_is_scalar, scale_w, bias, alpha, y, ldy,
                                 dev_status, st, after_quant);
    if (g_pair_gemm && pair_stream_covers_gemm(cont, desc, M, y, ydt, ldy, acc_out, p.combine_fast != 0))
        return launch_qgemm_pair_stream(a_codes, M, K, lda, desc, w_dev, scale_a, scale_a_is_scalar, scale_w, bias, alpha, y,
                                        ldy, dev_status, st, after_quant);

    CUtensorMap tmA, tmB, tmY{};
    const bool nib = cont == HQ_CODES_NIBBLE;
    if (!encode_2d(&tmA, a_codes, uint64_t(row_bytes), uint64_t(M), uint64_t(lda), nib ? kBK / 2 : kBK, kBM, !nib))
        return HQ_ERR_CUDA;
    // bf16 output: the epilogue hands 32 x 32 blocks to the copy engine (rows of a GEMM tile are consecutive)
    p.tma_store = (y != nullptr && acc_out == nullptr && p.y_bf16 && p.y_vec_ok && p.combine_fast) ? 1 : 0;
    if (p.tma_store && !encode_y(&tmY, y, uint64_t(desc->N), uint64_t(M), uint64_t(ldy))) return HQ_ERR_CUDA;
    const uint64_t Kp = uint64_t(desc->C_pad);
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, kBN, true)) return HQ_ERR_CUDA;
    return launch(nib, tmA, tmB, tmY, p, st);
}

hq_status launch_qconv2d(const void* a_codes, hq_container cont, int a_bits, int64_t Nb, int64_t H, int64_t W,
                         int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                         const float* scale_a, int scale_a_is_scalar, const float* scale_w, const float* bias,
                         float alpha, int32_t* acc_out, void* y, hq_dtype ydt, int32_t* dev_status, cudaStream_t st,
                         bool after_quant) {
    hq_status s = check_common(a_codes, cont, a_bits, desc, w_dev, scale_a, scale_w, acc_out, y, ydt,
                               int64_t(R) * S * C);
    if (s != HQ_OK) return s;
    if (R != S || (R != 1 && R != 3)) return HQ_ERR_UNSUPPORTED;
    if (stride != 1 && stride != 2) return HQ_ERR_UNSUPPORTED;
    if (pad != 0 && pad != 1) return HQ_ERR_UNSUPPORTED;
    if (desc->RS != R * S || desc->C != C) return HQ_ERR_SHAPE;
    if (Nb <= 0 || H <= 0 || W <= 0 || C <= 0) return HQ_ERR_SHAPE;
    const int64_t row_bytes = cont == HQ_CODES_NIBBLE ? C / 2 : C;
    if (row_bytes % 16 != 0) return HQ_ERR_ALIGNMENT;      // TMA strides are multiples of 16 bytes
    const int64_t Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
    if (Ho <= 0 || Wo <= 0) return HQ_ERR_SHAPE;
    if (Nb * Ho * Wo > (int64_t(1) << 30)) return HQ_ERR_UNSUPPORTED;
    // One scale per input pixel under a window of several taps: the accumulator is drained per tap (see the kernel).
    const bool per_tap = !scale_a_is_scalar && y != nullptr && R * S > 1;
    if (per_tap && acc_out != nullptr) {
        // the whole-window integer sums never exist in that mode: produce them with a launch of their own
        s = launch_qconv2d(a_codes, cont, a_bits, Nb, H, W, C, desc, w_dev, R, S, stride, pad, nullptr, 1, nullptr,
                           nullptr, 1.0f, acc_out, nullptr, ydt, dev_status, st, after_quant);
        if (s != HQ_OK) return s;
        acc_out = nullptr;
    }

    GemmParams p{};
    p.N = int(desc->N); p.limbs = desc->limbs;
    p.kb_per_tap = int(desc->C_pad / kBK); p.taps = R * S;
    p.pdl = (after_quant && !per_tap) ? 1 : 0;       // a per-tap layer may take several launches: keep those plain
    p.conv = 1; p.Nb = int(Nb); p.H = int(H); p.W = int(W); p.Ho = int(Ho); p.Wo = int(Wo);
    p.R = R; p.S = S; p.stride = stride; p.pad = pad;
    p.bw = int(Wo < kBM ? Wo : kBM);
    p.bh = int(Wo < kBM ? (Ho < kBM / p.bw ? Ho : kBM / p.bw) : 1);
    if (p.bh < 1) p.bh = 1;
    p.bn = kBM / (p.bw * p.bh);
    if (p.bn > Nb) p.bn = int(Nb);
    if (p.bn < 1) p.bn = 1;
    p.tiles_w = int((Wo + p.bw - 1) / p.bw);
    p.tiles_h = int((Ho + p.bh - 1) / p.bh);
    const int tiles_nb = int((Nb + p.bn - 1) / p.bn);
    p.tiles_m = p.tiles_w * p.tiles_h * tiles_nb;
    p.tiles_n = int(desc->limbs == 2 ? desc->N_pad / 128 : (desc->N_pad + 255) / 256);
    const bool nib = cont == HQ_CODES_NIBBLE;
    const int box_rows = p.bw * p.bh * p.bn;
    p.a_box_bytes = uint32_t(box_rows) * (nib ? kBK / 2 : kBK);
    fill_epilogue(p, cont, a_bits, desc, int64_t(R) * S * C, scale_a, scale_a_is_scalar, scale_w, bias, alpha, acc_out,
                  y, ydt, desc->N, dev_status);

    CUtensorMap tmA, tmB, tmY{};
    // Bulk stores need the 128 rows of a tile to be 128 consecutive output pixels: full-width tiles that are either
    // whole images or a whole number of row groups per image.
    const bool rows_consecutive = p.bw == Wo && p.bw * p.bh * p.bn == kBM && (p.bh == Ho || (p.bn == 1 && Ho % p.bh == 0));
    p.per_tap = per_tap ? 1 : 0;
    p.tma_store = (!per_tap && y != nullptr && acc_out == nullptr && p.y_bf16 && p.y_vec_ok && p.combine_fast && rows_consecutive) ? 1 : 0;
    if (p.tma_store && !encode_y(&tmY, y, uint64_t(desc->N), uint64_t(Nb * Ho * Wo), uint64_t(desc->N))) return HQ_ERR_CUDA;
    const uint64_t dims[4] = {uint64_t(row_bytes), uint64_t(W), uint64_t(H), uint64_t(Nb)};
    // With a traversal stride the box extent is given in input elements: stride * (pixels wanted).
    const uint32_t box[4] = {uint32_t(nib ? kBK / 2 : kBK), uint32_t(p.bw * stride), uint32_t(p.bh * stride), uint32_t(p.bn)};
    const uint32_t estr[4] = {1, uint32_t(stride), uint32_t(stride), 1};
    if (!encode_4d(&tmA, a_codes, dims, box, estr, !nib)) return HQ_ERR_CUDA;
    const uint64_t Kp = uint64_t(desc->C_pad) * desc->RS;
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, kBN, true)) return HQ_ERR_CUDA;
    if (g_pair_gemm && pair_stream_covers_conv(cont, p)) return launch_qconv_pair(p, tmA, tmY, desc, w_dev, st);
    s = launch(nib, tmA, tmB, tmY, p, st);
    if (s == HQ_OK && per_tap && desc->limbs == 1) {      // the other 64 of every warp's 128 columns
        p.col_pass = 1;
        s = launch(nib, tmA, tmB, tmY, p, st);
    }
    return s;
}

}  // namespace hq

extern "C" hq_status hq_qgemm(const void* a_codes, hq_container cont, int a_bits, int64_t M, int64_t K, int64_t lda,
                              const hq_weight_desc* desc, const void* w_dev, const float* scale_a,
                              int scale_a_is_scalar, const float* scale_w, const float* bias, float alpha,
                              int32_t* acc_out, void* y, hq_dtype ydt, int64_t ldy, int32_t* dev_status,
                              void* stream) {
    return hq::launch_qgemm(a_codes, cont, a_bits, M, K, lda, desc, w_dev, scale_a, scale_a_is_scalar, scale_w, bias,
                            alpha, acc_out, y, ydt, ldy, dev_status, static_cast<cudaStream_t>(stream), false);
}

extern "C" hq_status hq_qconv2d(const void* a_codes, hq_container cont, int a_bits, int64_t Nb, int64_t H, int64_t W,
                                int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride,
                                int pad, const float* scale_a, int scale_a_is_scalar, const float* scale_w,
                                const float* bias, float alpha, int32_t* acc_out, void* y, hq_dtype ydt,
                                int32_t* dev_status, void* stream) {
    return hq::launch_qconv2d(a_codes, cont, a_bits, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scale_a,
                              scale_a_is_scalar, scale_w, bias, alpha, acc_out, y, ydt, dev_status,
                              static_cast<cudaStream_t>(stream), false);
}

extern "C" int hq_set_pair_gemm(int mode) {
    const int before = hq::g_pair_gemm;
    hq::g_pair_gemm = mode < 0 ? 0 : (mode > 2 ? 2 : mode);
    return before;
}

extern "C" hq_status hq_mma_i8_probe(int ctas, int iters, int32_t* dev_status, void* stream) {
    if (ctas <= 0 || iters <= 0) return HQ_ERR_INVALID_ARG;
    const size_t smem = 1024 + hq::gemm::kABytes + hq::gemm::kBBytes;
    HQ_CUDA_OK(cudaFuncSetAttribute(hq::mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    hq::mma_probe_kernel<<<ctas, 128, smem, static_cast<cudaStream_t>(stream)>>>(iters, dev_status);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
