// Integer GEMM / implicit-GEMM convolution with a fused rescale epilogue (Eq. 12, Eq. 14).
//
//   acc[m][o] = sum_k a[m][k] * B[o][k]   int8 x int8 -> int32 on the 5th-generation tensor cores
//   y[m][o]   = alpha * S_a[m] * S_w[o] * acc[m][o] + bias[o]
//
// One persistent CTA per SM walks output tiles of 128 rows x 256 operand rows (256 output channels with
// one weight limb, 128 with two).  Roles:
//   warp 0      TMA producer: activation tile (2-D box for a GEMM, 4-D NHWC box per filter tap for a
//               convolution, out-of-bounds = zero padding) and weight tile into a 4-stage shared-memory ring
//   warp 1      issues tcgen05.mma.kind::i8 (128x256x32) into one of two 256-column TMEM accumulators
//   warps 2-5   epilogue: tcgen05.ld, limb recombination (256*hi + lo), rescale, bf16/fp32/int32 stores;
//               runs on accumulator t while the MMA warp fills accumulator t+1
//   warps 6-9   (NIBBLE container only) unpack 4-bit codes from a raw TMA tile into the swizzled int8 operand
//               tile.  A code q is written as the byte q<<4 (= 16q, no sign extension needed), so the accumulator
//               is 16x the true one and is shifted back exactly in the epilogue.
// Every wait is bounded; on expiry a status word is written and the CTA drains and exits.
#include <cuda.h>

#include <cmath>

#include "hq_common.cuh"

namespace hq {
namespace {

constexpr int kBM = 128;             // rows per tile (TMEM lanes)
constexpr int kBN = 256;             // operand-B rows per tile (TMEM columns)
constexpr int kBK = 128;             // bytes of K per stage (one 128-byte swizzle row)
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK;           // 16 KB
constexpr int kBBytes = kBN * kBK;           // 32 KB
constexpr int kRawBytes = kBM * kBK / 2;     // 8 KB packed activation tile
constexpr int kTmemCols = 512;

struct GemmParams {
    int64_t M;            // GEMM rows (unused for conv)
    int N;                // output channels
    int limbs;
    int a_shift;          // 4 when activation bytes are q<<4 (nibble container), else 0
    int kb_per_tap;       // 128-byte K blocks per filter tap
    int taps;
    int tiles_m, tiles_n;
    uint32_t a_box_bytes; // bytes one activation TMA box delivers
    // convolution geometry (conv != 0)
    int conv, Nb, H, W, Ho, Wo, R, S, stride, pad;
    int bw, bh, bn, tiles_w, tiles_h;
    // epilogue
    const float* scale_a; int sa_scalar;
    const float* scale_w; const float* bias; float alpha;
    int32_t* acc_out; void* y; int y_bf16; int64_t ldy;
    int32_t* dev_status;
};

struct SharedCtl {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t unpacked[kStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile unsigned int issued;    // stages the producer has armed (for the drain on abort)
};

template <bool NIBBLE>
constexpr size_t smem_bytes() {
    return 1024 + size_t(kStages) * (kABytes + kBBytes + (NIBBLE ? kRawBytes : 0)) + sizeof(SharedCtl) + 64;
}

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SharedCtl* ctl, int32_t* dev_status,
                                              int32_t code) {
    for (int it = 0; it < 4096; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000000LL) {
        if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
        __nanosleep(32);
    }
    ctl->abort_flag = 1;
    if (dev_status) atomicExch(dev_status, code);
    return false;
}

struct TileCoord {
    int m_tile, n_tile;
    int n0, h0, w0;      // conv: first image / output row / output column of the tile
};

__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int tile) {
    TileCoord t;
    t.m_tile = tile / p.tiles_n;
    t.n_tile = tile - t.m_tile * p.tiles_n;
    t.n0 = t.h0 = t.w0 = 0;
    if (p.conv) {
        const int tw = t.m_tile % p.tiles_w;
        const int th = (t.m_tile / p.tiles_w) % p.tiles_h;
        const int tn = t.m_tile / (p.tiles_w * p.tiles_h);
        t.w0 = tw * p.bw; t.h0 = th * p.bh; t.n0 = tn * p.bn;
    }
    return t;
}

template <bool NIBBLE>
__global__ void __launch_bounds__(NIBBLE ? 320 : 192, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sA = smem;
    unsigned char* sB = sA + kStages * kABytes;
    unsigned char* sRaw = sB + kStages * kBBytes;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(sRaw + (NIBBLE ? kStages * kRawBytes : 0));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int num_kb = p.kb_per_tap * p.taps;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
            mbar_init(&ctl->unpacked[s], 128);
        }
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], 4); }
        ctl->abort_flag = 0;
        ctl->issued = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) { tmem_alloc(&ctl->tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const TileCoord tc = tile_coord(p, tile);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!wait_or_abort(&ctl->empty[stage], phase ^ 1, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    mbar_expect_tx(&ctl->full[stage], p.a_box_bytes + kBBytes);
                    unsigned char* a_dst = NIBBLE ? sRaw + stage * kRawBytes : sA + stage * kABytes;
                    const int a_k = (NIBBLE ? kBK / 2 : kBK);
                    if (p.conv) {
                        const int tap = kb / p.kb_per_tap, kc = kb - tap * p.kb_per_tap;
                        const int r = tap / p.S, s = tap - r * p.S;
                        tma_load_4d(a_dst, &tmA, &ctl->full[stage], kc * a_k, tc.w0 * p.stride + s - p.pad,
                                    tc.h0 * p.stride + r - p.pad, tc.n0);
                    } else {
                        tma_load_2d(a_dst, &tmA, &ctl->full[stage], kb * a_k, tc.m_tile * kBM);
                    }
                    tma_load_2d(sB + stage * kBBytes, &tmB, &ctl->full[stage], kb * kBK, tc.n_tile * kBN);
                    ctl->issued = ctl->issued + 1;
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_i8(kBM, kBN);
            int stage = 0; uint32_t phase = 0;
            unsigned int consumed = 0;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
                const int as = it & 1;
                const uint32_t aphase = (it >> 1) & 1;
                if (!wait_or_abort(&ctl->tempty[as], aphase ^ 1, ctl, p.dev_status, kStatusAccumFree)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + uint32_t(as * kBN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!wait_or_abort(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                    ++consumed;
                    if (NIBBLE) {
                        if (!wait_or_abort(&ctl->unpacked[stage], phase, ctl, p.dev_status, kStatusUnpackWait)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint64_t a_desc = make_sw128_kmajor_desc(smem_u32(sA + stage * kABytes));
                    const uint64_t b_desc = make_sw128_kmajor_desc(smem_u32(sB + stage * kBBytes));
#pragma unroll
                    for (int k = 0; k < kBK / 32; ++k)
                        mma_i8(d_tmem, a_desc + uint64_t(k * 2), b_desc + uint64_t(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
                    mma_commit(&ctl->empty[stage]);
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (ok) mma_commit(&ctl->tfull[as]);
            }
            if (!ok) {
                // Abort path: wait (bounded) for TMA copies already in flight so none lands after exit.
                const unsigned int issued = ctl->issued;
                while (consumed < issued) {
                    mbar_wait(&ctl->full[stage], phase, nullptr, 0);
                    ++consumed;
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int r_in_tile = q * 32 + lane;
        int it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
            const int as = it & 1;
            const uint32_t aphase = (it >> 1) & 1;
            const TileCoord tc = tile_coord(p, tile);
            if (!wait_or_abort(&ctl->tfull[as], aphase, ctl, p.dev_status, kStatusAccumWait)) { ok = false; break; }
            tc_fence_after();

            int64_t out_row; bool row_ok;
            if (p.conv) {
                const int iw = r_in_tile % p.bw;
                const int ih = (r_in_tile / p.bw) % p.bh;
                const int in = r_in_tile / (p.bw * p.bh);
                const int n = tc.n0 + in, ho = tc.h0 + ih, wo = tc.w0 + iw;
                row_ok = in < p.bn && n < p.Nb && ho < p.Ho && wo < p.Wo;
                out_row = (int64_t(n) * p.Ho + ho) * p.Wo + wo;
            } else {
                out_row = int64_t(tc.m_tile) * kBM + r_in_tile;
                row_ok = out_row < p.M;
            }
            float sa = 0.f;
            if (row_ok && p.y != nullptr) sa = p.alpha * (p.sa_scalar ? __ldg(p.scale_a) : __ldg(p.scale_a + out_row));
            const int cols_per_tile = p.limbs == 2 ? kBN / 2 : kBN;
            const int col_base = tc.n_tile * cols_per_tile;
            const uint32_t t_row = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN);

            for (int ch = 0; ch < cols_per_tile / 32; ++ch) {
                const int col0 = col_base + ch * 32;
                if (col0 >= p.N) break;                 // uniform across the warp
                uint32_t v[32];
                tmem_ld_32x32(t_row + uint32_t(ch * 32), v);
                if (p.limbs == 2) {
                    uint32_t lo[32];
                    tmem_ld_32x32(t_row + uint32_t(kBN / 2 + ch * 32), lo);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        v[j] = uint32_t(((int32_t(v[j]) >> p.a_shift) << 8) + (int32_t(lo[j]) >> p.a_shift));
                } else {
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = uint32_t(int32_t(v[j]) >> p.a_shift);
                }
                if (!row_ok) continue;
                const bool full_chunk = col0 + 32 <= p.N;
                if (p.acc_out != nullptr) {
                    int32_t* dst = p.acc_out + out_row * int64_t(p.N) + col0;
                    if (full_chunk && (p.N & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (col0 + j < p.N) dst[j] = int32_t(v[j]);
                    }
                }
                if (p.y != nullptr) {
                    float f[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int c = col0 + j < p.N ? col0 + j : p.N - 1;
                        const float sw = __ldg(p.scale_w + c);
                        const float b = p.bias != nullptr ? __ldg(p.bias + c) : 0.f;
                        f[j] = fmaf(float(int32_t(v[j])), sa * sw, b);
                    }
                    if (p.y_bf16) {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.y) + out_row * p.ldy + col0;
                        if (full_chunk && (p.ldy & 7) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                uint4 pk;
                                __nv_bfloat162 h0 = __floats2bfloat162_rn(f[j], f[j + 1]);
                                __nv_bfloat162 h1 = __floats2bfloat162_rn(f[j + 2], f[j + 3]);
                                __nv_bfloat162 h2 = __floats2bfloat162_rn(f[j + 4], f[j + 5]);
                                __nv_bfloat162 h3 = __floats2bfloat162_rn(f[j + 6], f[j + 7]);
                                pk.x = *reinterpret_cast<uint32_t*>(&h0); pk.y = *reinterpret_cast<uint32_t*>(&h1);
                                pk.z = *reinterpret_cast<uint32_t*>(&h2); pk.w = *reinterpret_cast<uint32_t*>(&h3);
                                *reinterpret_cast<uint4*>(dst + j) = pk;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (col0 + j < p.N) dst[j] = __float2bfloat16_rn(f[j]);
                        }
                    } else {
                        float* dst = reinterpret_cast<float*>(p.y) + out_row * p.ldy + col0;
                        if (full_chunk && (p.ldy & 3) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<float4*>(dst + j) = make_float4(f[j], f[j + 1], f[j + 2], f[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (col0 + j < p.N) dst[j] = f[j];
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->tempty[as]);
        }
    } else if (NIBBLE) {
        // ------------------------------------------------------------------ nibble -> int8 unpack (warps 6-9)
        const int t = threadIdx.x - 192;              // 0..127
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!wait_or_abort(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                const uint4* raw = reinterpret_cast<const uint4*>(sRaw + stage * kRawBytes);
                unsigned char* dstA = sA + stage * kABytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int id = i * 128 + t;           // 16-byte chunk of the packed tile: row = id/4, part = id%4
                    const int row = id >> 2, part = id & 3;
                    const uint4 w = raw[id];
                    uint4 o0, o1;
                    o0.x = (w.x << 4) & 0xF0F0F0F0u; o0.y = w.x & 0xF0F0F0F0u;
                    o0.z = (w.y << 4) & 0xF0F0F0F0u; o0.w = w.y & 0xF0F0F0F0u;
                    o1.x = (w.z << 4) & 0xF0F0F0F0u; o1.y = w.z & 0xF0F0F0F0u;
                    o1.z = (w.w << 4) & 0xF0F0F0F0u; o1.w = w.w & 0xF0F0F0F0u;
                    unsigned char* rowp = dstA + row * 128;
                    *reinterpret_cast<uint4*>(rowp + (((2 * part) ^ (row & 7)) << 4)) = o0;
                    *reinterpret_cast<uint4*>(rowp + (((2 * part + 1) ^ (row & 7)) << 4)) = o1;
                }
                fence_proxy_async_smem();
                mbar_arrive(&ctl->unpacked[stage]);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

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

bool encode_2d(CUtensorMap* tm, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
               uint32_t box_inner, uint32_t box_rows, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[2] = {inner_bytes, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_4d(CUtensorMap* tm, const void* base, const uint64_t dims_in[4], const uint32_t box_in[4],
               const uint32_t estr_in[4], bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[4] = {dims_in[0], dims_in[1], dims_in[2], dims_in[3]};
    cuuint64_t strides[3] = {dims_in[0], dims_in[0] * dims_in[1], dims_in[0] * dims_in[1] * dims_in[2]};
    cuuint32_t box[4] = {box_in[0], box_in[1], box_in[2], box_in[3]};
    cuuint32_t estr[4] = {estr_in[0], estr_in[1], estr_in[2], estr_in[3]};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
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

template <bool NIBBLE>
hq_status launch(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p, cudaStream_t st) {
    static bool attr_set[64] = {};
    constexpr size_t smem = smem_bytes<NIBBLE>();
    int dev = 0;
    HQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        HQ_CUDA_OK(cudaFuncSetAttribute(qgemm_kernel<NIBBLE>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const int tiles = p.tiles_m * p.tiles_n;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    qgemm_kernel<NIBBLE><<<grid, NIBBLE ? 320 : 192, smem, st>>>(tmA, tmB, p);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
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
                       hq_dtype ydt, int64_t ldy, int32_t* dev_status, cudaStream_t st) {
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
    p.M = M; p.N = int(desc->N); p.limbs = desc->limbs; p.a_shift = cont == HQ_CODES_NIBBLE ? 4 : 0;
    p.kb_per_tap = int(desc->C_pad / kBK); p.taps = 1;
    p.tiles_m = int((M + kBM - 1) / kBM);
    p.tiles_n = int(desc->limbs == 2 ? desc->N_pad / 128 : (desc->N_pad + 255) / 256);
    p.a_box_bytes = cont == HQ_CODES_NIBBLE ? kRawBytes : kABytes;
    p.conv = 0;
    p.scale_a = scale_a; p.sa_scalar = scale_a_is_scalar; p.scale_w = scale_w; p.bias = bias; p.alpha = alpha;
    p.acc_out = acc_out; p.y = y; p.y_bf16 = ydt == HQ_BF16; p.ldy = ldy; p.dev_status = dev_status;

    CUtensorMap tmA, tmB;
    const bool nib = cont == HQ_CODES_NIBBLE;
    if (!encode_2d(&tmA, a_codes, uint64_t(row_bytes), uint64_t(M), uint64_t(lda), nib ? kBK / 2 : kBK, kBM, !nib))
        return HQ_ERR_CUDA;
    const uint64_t Kp = uint64_t(desc->C_pad);
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, kBN, true)) return HQ_ERR_CUDA;
    return nib ? launch<true>(tmA, tmB, p, st) : launch<false>(tmA, tmB, p, st);
}

hq_status launch_qconv2d(const void* a_codes, hq_container cont, int a_bits, int64_t Nb, int64_t H, int64_t W,
                         int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                         const float* scale_a, int scale_a_is_scalar, const float* scale_w, const float* bias,
                         float alpha, int32_t* acc_out, void* y, hq_dtype ydt, int32_t* dev_status, cudaStream_t st) {
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
    if (!scale_a_is_scalar && y != nullptr && R * S > 1) return HQ_ERR_UNSUPPORTED;   // per-tap rescale: separate kernel

    GemmParams p{};
    p.N = int(desc->N); p.limbs = desc->limbs; p.a_shift = cont == HQ_CODES_NIBBLE ? 4 : 0;
    p.kb_per_tap = int(desc->C_pad / kBK); p.taps = R * S;
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
    p.scale_a = scale_a; p.sa_scalar = scale_a_is_scalar; p.scale_w = scale_w; p.bias = bias; p.alpha = alpha;
    p.acc_out = acc_out; p.y = y; p.y_bf16 = ydt == HQ_BF16; p.ldy = desc->N; p.dev_status = dev_status;

    CUtensorMap tmA, tmB;
    const uint64_t dims[4] = {uint64_t(row_bytes), uint64_t(W), uint64_t(H), uint64_t(Nb)};
    // With a traversal stride the box extent is given in input elements: stride * (pixels wanted).
    const uint32_t box[4] = {uint32_t(nib ? kBK / 2 : kBK), uint32_t(p.bw * stride), uint32_t(p.bh * stride), uint32_t(p.bn)};
    const uint32_t estr[4] = {1, uint32_t(stride), uint32_t(stride), 1};
    if (stride != 1) return HQ_ERR_UNSUPPORTED;          // strided boxes: not enabled yet
    if (!encode_4d(&tmA, a_codes, dims, box, estr, !nib)) return HQ_ERR_CUDA;
    const uint64_t Kp = uint64_t(desc->C_pad) * desc->RS;
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, kBN, true)) return HQ_ERR_CUDA;
    return nib ? launch<true>(tmA, tmB, p, st) : launch<false>(tmA, tmB, p, st);
}

}  // namespace hq

extern "C" hq_status hq_qgemm(const void* a_codes, hq_container cont, int a_bits, int64_t M, int64_t K, int64_t lda,
                              const hq_weight_desc* desc, const void* w_dev, const float* scale_a,
                              int scale_a_is_scalar, const float* scale_w, const float* bias, float alpha,
                              int32_t* acc_out, void* y, hq_dtype ydt, int64_t ldy, int32_t* dev_status,
                              void* stream) {
    return hq::launch_qgemm(a_codes, cont, a_bits, M, K, lda, desc, w_dev, scale_a, scale_a_is_scalar, scale_w, bias,
                            alpha, acc_out, y, ydt, ldy, dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" hq_status hq_qconv2d(const void* a_codes, hq_container cont, int a_bits, int64_t Nb, int64_t H, int64_t W,
                                int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride,
                                int pad, const float* scale_a, int scale_a_is_scalar, const float* scale_w,
                                const float* bias, float alpha, int32_t* acc_out, void* y, hq_dtype ydt,
                                int32_t* dev_status, void* stream) {
    return hq::launch_qconv2d(a_codes, cont, a_bits, Nb, H, W, C, desc, w_dev, R, S, stride, pad, scale_a,
                              scale_a_is_scalar, scale_w, bias, alpha, acc_out, y, ydt, dev_status,
                              static_cast<cudaStream_t>(stream));
}

extern "C" hq_status hq_mma_i8_probe(int ctas, int iters, int32_t* dev_status, void* stream) {
    if (ctas <= 0 || iters <= 0) return HQ_ERR_INVALID_ARG;
    const size_t smem = 1024 + hq::kABytes + hq::kBBytes;
    HQ_CUDA_OK(cudaFuncSetAttribute(hq::mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    hq::mma_probe_kernel<<<ctas, 128, smem, static_cast<cudaStream_t>(stream)>>>(iters, dev_status);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
