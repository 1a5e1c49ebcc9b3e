// Fused quantized linear layer in ONE kernel (Eq. 10, Eq. 3, Eq. 12): the Hadamard transform and the quantization run
// inside the GEMM CTA and write their int8 codes straight into the shared-memory operand tile the tensor core reads, so
// the codes and the activation scales never travel through global memory and no second kernel is launched.
//
// For reductions that fit one operand tile (K = 128, 256 or 512 channels) the activation tile is STATIONARY: a CTA owns a
// contiguous range of output tiles in row-major tile order; whenever the row tile changes, its eight epilogue warps read
// the 128 x K fp32 / bf16 activations, run the register butterflies of the stand-alone transform kernel (a row is held by
// K / 32 lanes of one warp, so every exchange and the row maximum stay inside the warp), round, and store the codes with
// the 128-byte swizzle of the MMA descriptor; the row scales stay in shared memory for the epilogue.  The weight tiles
// of the successive column tiles stream through a TMA ring; MMA issue, tensor-memory double buffering and the bulk-store
// epilogue are those of the two-kernel path.
#include <cuda.h>

#include <cmath>
#include <type_traits>

#include "hq_fwht.cuh"
#include "hq_gemm_kernel.cuh"

namespace hq {
namespace {
using namespace gemm;

constexpr int kFusedThreads = 320;           // producer warp, MMA warp, eight transform + epilogue warps
constexpr int kFusedMaxStages = 4;
constexpr int kXchBytesPerWarp = 5120;       // exchange buffers of the rows one warp transforms at a time
constexpr int kFusedParamBytes = kEpiWarps * 2 * (kBN / 2) * 4;

struct FusedParams {
    const void* x; int64_t ldx; int64_t M;
    int K, N, limbs, num_kb, tiles_m, tiles_n, stages, bits;
    float norm;                  // 2^(-k/2)
    const float* static_scale;   // STATIC instantiations
    const float* scale_w; const float* bias; float alpha;
    int32_t* dev_status;
};

struct FusedCtl {
    uint64_t full[kFusedMaxStages];
    uint64_t empty[kFusedMaxStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint64_t a_ready;
    uint32_t tmem_base;
    volatile int abort_flag;
};

struct FusedLayout { int a_off, b_off, staging_off, param_off, xch_off, scale_off, ctl_off, total; };
__host__ __device__ inline FusedLayout fused_layout(int num_kb, int stages) {
    FusedLayout L;
    L.a_off = 0;
    L.b_off = num_kb * kABytes;
    L.staging_off = L.b_off + stages * kBBytes;
    L.param_off = L.staging_off + kEpiWarps * kStagingBytes;
    L.xch_off = L.param_off + kFusedParamBytes;
    L.scale_off = L.xch_off + kEpiWarps * kXchBytesPerWarp;
    L.ctl_off = L.scale_off + 2 * kBM * 4;            // two sets of row scales: consecutive row tiles alternate
    L.total = L.ctl_off + int(sizeof(FusedCtl)) + 1024;
    return L;
}

__device__ __forceinline__ bool wait_fused(uint64_t* bar, uint32_t parity, FusedCtl* ctl, int32_t* dev_status,
                                           int32_t code) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000000LL) {
        if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
    }
    ctl->abort_flag = 1;
    if (dev_status) atomicExch(dev_status, code);
    return false;
}

// Transform + quantize the 128 rows of row tile `m_tile` into the swizzled operand tile sA (num_kb blocks of 128 rows x
// 128 bytes) and their scales into sScale.  Called by the eight epilogue warps (ew = 0..7).
template <int KLOG, typename InT, bool STATIC>
__device__ __forceinline__ void build_a_tile(const FusedParams& p, int m_tile, unsigned char* sA, float* sScale,
                                             unsigned char* xch_warp, int ew, int lane) {
    constexpr int E = 32;
    using Sh = FwhtShape<KLOG, E>;
    constexpr int N = Sh::N, P = Sh::P, TB = Sh::TB;
    const int tpr = p.K / E;                           // lanes per row: 4, 8 or 16
    const int rpw = 32 / tpr;                          // rows a warp transforms at a time
    const int row_in_warp = lane / tpr, tr = lane - row_in_warp * tpr;
    const int blk = tr / TB, tb = tr & (TB - 1);
    float4* grp = reinterpret_cast<float4*>(xch_warp) + (lane / TB) * Sh::GS;
    const float qmaxf = float((1 << (p.bits - 1)) - 1);
    // raw 16-byte (fp32) or 8-byte (bf16) pieces of a row as they come from memory; the next pass's pieces are requested
    // before the current pass is transformed, so that their latency hides behind its arithmetic
    using Raw = typename std::conditional<sizeof(InT) == 4, float4, uint2>::type;
    const int npass = kBM / (kEpiWarps * rpw);
    auto fetch = [&](int pass, Raw (&raw)[E / 4]) {
        const int rr = pass * (kEpiWarps * rpw) + ew * rpw + row_in_warp;
        const int64_t row = int64_t(m_tile) * kBM + rr;
        const InT* src = reinterpret_cast<const InT*>(p.x) + (row < p.M ? row : 0) * p.ldx + blk * N;
#pragma unroll
        for (int i = 0; i < E / 4; ++i) raw[i] = __ldcs(reinterpret_cast<const Raw*>(src + 4 * (tb + TB * i)));
    };
    Raw cur[E / 4], nxt[E / 4];
    fetch(0, cur);
    for (int pass = 0; pass < npass; ++pass) {
        const int r = pass * (kEpiWarps * rpw) + ew * rpw + row_in_warp;
        const int64_t row = int64_t(m_tile) * kBM + r;
        const bool valid = row < p.M;
        if (pass + 1 < npass) fetch(pass + 1, nxt);
        f32x2 v[P];
#pragma unroll
        for (int i = 0; i < E / 4; ++i) {
            float4 f;
            if constexpr (sizeof(InT) == 4) {
                f = cur[i];
            } else {
                f = make_float4(__uint_as_float(cur[i].x << 16), __uint_as_float(cur[i].x & 0xFFFF0000u),
                                __uint_as_float(cur[i].y << 16), __uint_as_float(cur[i].y & 0xFFFF0000u));
            }
            if (!valid) f = make_float4(0.f, 0.f, 0.f, 0.f);
            v[2 * i] = pk2(f.x, f.y);
            v[2 * i + 1] = pk2(f.z, f.w);
        }
        fwht_stages<KLOG, E, false>(v, grp, tb);
        float inv, scale;
        if (!STATIC) {
            float amax = 0.f;
#pragma unroll
            for (int e = 0; e < P; ++e) {
                float a, b;
                upk2(v[e], a, b);
                amax = fmaxf(fmaxf(amax, fabsf(a)), fabsf(b));
            }
            for (int off = 1; off < tpr; off <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
            if (amax > 0.f) {
                scale = amax * (p.norm / qmaxf);
                inv = qmaxf / amax;
                if (!(scale > 0.f)) { scale = 1.0f; inv = p.norm; }
            } else {
                scale = 1.0f;
                inv = 0.f;
            }
        } else {
            scale = __ldg(p.static_scale);
            inv = p.norm / scale;
        }
        uint32_t w[E / 4];
        pack_codes<KLOG, E, true, STATIC>(v, inv, p.bits, tb, w);
        // the thread's 32 codes are channels c0 .. c0 + 31 of its row: two 16-byte pieces of K block c0 / 128
        const int c0 = blk * N + E * tb;
        unsigned char* rowp = sA + (c0 >> 7) * kABytes + r * 128;
        const int j0 = (c0 & 127) >> 4;
        *reinterpret_cast<uint4*>(rowp + (((j0) ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(rowp + (((j0 + 1) ^ (r & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
        if (tr == 0) sScale[r] = scale;
        __syncwarp();                                  // the exchange buffer is written again by the next pass
#pragma unroll
        for (int i = 0; i < E / 4; ++i) cur[i] = nxt[i];
    }
}

template <int KLOG, typename InT, int LIMBS, bool STATIC>
__global__ void __launch_bounds__(kFusedThreads, 1)
qlinear_fused_kernel(const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmY,
                     const FusedParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const FusedLayout L = fused_layout(p.num_kb, p.stages);
    unsigned char* sA = smem + L.a_off;
    unsigned char* sB = smem + L.b_off;
    unsigned char* sStage = smem + L.staging_off;
    float* sParam = reinterpret_cast<float*>(smem + L.param_off);
    unsigned char* sXch = smem + L.xch_off;
    float* sScale = reinterpret_cast<float*>(smem + L.scale_off);
    FusedCtl* ctl = reinterpret_cast<FusedCtl*>(smem + L.ctl_off);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nstages = p.stages, num_kb = p.num_kb;
    // this CTA's contiguous range of tiles in row-major tile order (column tile fastest)
    const int T = p.tiles_m * p.tiles_n, G = gridDim.x, c = blockIdx.x;
    const int first = int(int64_t(c) * T / G);
    const int count = int(int64_t(c + 1) * T / G) - first;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFusedMaxStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], kEpiWarps); }
        mbar_init(&ctl->a_ready, kEpiWarps);
        ctl->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmY);
    }
    if (warp == 1) { __syncwarp(); tmem_alloc(&ctl->tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: weight tiles only
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            long long armed = 0;
            bool ok = true;
            for (int i = 0; i < count && ok; ++i) {
                const int n_tile = (first + i) % p.tiles_n;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!wait_fused(&ctl->empty[stage], phase ^ 1, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    mbar_expect_tx(&ctl->full[stage], uint32_t(kBBytes));
                    tma_load_2d(sB + stage * kBBytes, &tmB, &ctl->full[stage], kb * kBK, n_tile * kBN);
                    ++armed;
                    if (++stage == nstages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // abort path: wait (bounded) for the copies in flight so that none lands after the CTA has exited
                const int back = armed < nstages ? int(armed) : nstages;
                for (int j = 0; j < back; ++j) {
                    if (--stage < 0) { stage = nstages - 1; phase ^= 1; }
                    mbar_wait(&ctl->full[stage], phase, nullptr, 0);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_i8(kBM, kBN);
            int stage = 0; uint32_t phase = 0;
            int cur_m = -1, builds = 0;
            bool ok = true;
            for (int i = 0; i < count && ok; ++i) {
                const int m_tile = (first + i) / p.tiles_n;
                if (m_tile != cur_m) {                     // a new activation tile: wait until its codes are in place
                    cur_m = m_tile;
                    if (!wait_fused(&ctl->a_ready, uint32_t(builds) & 1u, ctl, p.dev_status, kStatusUnpackWait)) { ok = false; break; }
                    ++builds;
                }
                const int as = i & 1;
                if (!wait_fused(&ctl->tempty[as], (uint32_t(i >> 1) & 1u) ^ 1u, ctl, p.dev_status, kStatusAccumFree)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + uint32_t(as * kBN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!wait_fused(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_sw128_kmajor_desc(smem_u32(sA + kb * kABytes));
                    const uint64_t b_desc = make_sw128_kmajor_desc(smem_u32(sB + stage * kBBytes));
#pragma unroll
                    for (int k = 0; k < kBK / 32; ++k)
                        mma_i8(d_tmem, a_desc + uint64_t(k * 2), b_desc + uint64_t(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
                    mma_commit(&ctl->empty[stage]);
                    if (++stage == nstages) { stage = 0; phase ^= 1; }
                }
                if (ok) mma_commit(&ctl->tfull[as]);
            }
        }
    } else {
        // ------------------------------------------------------------------ transform + epilogue (warps 2-9)
        const int ew = warp - 2;
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int chalf = ew >> 2;                    // which half of the tile's columns this warp takes
        unsigned char* stg = sStage + ew * kStagingBytes;
        float* prm_sw = sParam + ew * 2 * (kBN / 2);
        float* prm_b = prm_sw + kBN / 2;
        constexpr int cols_per_tile = LIMBS == 2 ? kBN / 2 : kBN;
        constexpr int cols_per_warp = cols_per_tile / 2;
        const int wc0 = chalf * cols_per_warp;
        int cur_m = -1, last_n = -1, builds = 0;
        bool ok = true;
        for (int i = 0; i < count && ok; ++i) {
            const int m_tile = (first + i) / p.tiles_n, n_tile = (first + i) - m_tile * p.tiles_n;
            if (m_tile != cur_m) {
                // The accumulators of the previous row tile were drained by this loop, so every MMA that read the old
                // codes has completed: the operand tile may be rewritten.  The row scales go to the set the previous
                // row tile does not use (a slower warp may still need those).
                cur_m = m_tile;
                build_a_tile<KLOG, InT, STATIC>(p, m_tile, sA, sScale + (builds & 1) * kBM, sXch + ew * kXchBytesPerWarp, ew, lane);
                fence_proxy_async_smem();             // the codes become visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->a_ready);
                // all eight warps' codes and scales are in place (the MMA issuer waits on the same barrier)
                if (!wait_fused(&ctl->a_ready, uint32_t(builds) & 1u, ctl, p.dev_status, kStatusUnpackWait)) { ok = false; break; }
                ++builds;
            }
            const int as = i & 1;
            const int col_base = n_tile * cols_per_tile;
            if (n_tile != last_n) {
                last_n = n_tile;
                __syncwarp();
                for (int cc = lane; cc < cols_per_warp; cc += 32) {
                    const int col = col_base + wc0 + cc;
                    prm_sw[cc] = col < p.N ? __ldg(p.scale_w + col) : 0.f;
                    prm_b[cc] = (p.bias != nullptr && col < p.N) ? __ldg(p.bias + col) : 0.f;
                }
                __syncwarp();
            }
            const float sa_eff = p.alpha * sScale[((builds - 1) & 1) * kBM + q * 32 + lane];
            if (!wait_fused(&ctl->tfull[as], uint32_t(i >> 1) & 1u, ctl, p.dev_status, kStatusAccumWait)) { ok = false; break; }
            tc_fence_after();
            const int row0 = m_tile * kBM + q * 32;
            const uint32_t t_fast = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN + wc0);
            epilogue_fast<LIMBS>(t_fast, stg, lane, prm_sw, prm_b, sa_eff, &tmY, col_base + wc0, row0, &ctl->tempty[as]);
        }
        if (lane == 0) bulk_wait_read_all();           // shared memory must outlive the copy engine's reads
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

template <int KLOG, typename InT>
cudaError_t launch_fused(const FusedParams& p, bool is_static, int grid, size_t smem, cudaStream_t st,
                         const CUtensorMap& tmB, const CUtensorMap& tmY) {
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        kern<<<grid, kFusedThreads, smem, st>>>(tmB, tmY, p);
        return cudaGetLastError();
    };
    if (p.limbs == 2) return is_static ? go(qlinear_fused_kernel<KLOG, InT, 2, true>) : go(qlinear_fused_kernel<KLOG, InT, 2, false>);
    return is_static ? go(qlinear_fused_kernel<KLOG, InT, 1, true>) : go(qlinear_fused_kernel<KLOG, InT, 1, false>);
}

template <typename InT>
cudaError_t dispatch_fused(int klog, const FusedParams& p, bool is_static, int grid, size_t smem, cudaStream_t st,
                           const CUtensorMap& tmB, const CUtensorMap& tmY) {
    switch (klog) {
        case 5: return launch_fused<5, InT>(p, is_static, grid, smem, st, tmB, tmY);
        case 6: return launch_fused<6, InT>(p, is_static, grid, smem, st, tmB, tmY);
        case 7: return launch_fused<7, InT>(p, is_static, grid, smem, st, tmB, tmY);
        case 8: return launch_fused<8, InT>(p, is_static, grid, smem, st, tmB, tmY);
        case 9: return launch_fused<9, InT>(p, is_static, grid, smem, st, tmB, tmY);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace
}  // namespace hq

extern "C" hq_status hq_qlinear_fused(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx,
                                      const hq_weight_desc* desc, const void* w_dev, const float* scale_w,
                                      const float* bias, int a_bits, hq_scale_mode mode, const float* static_scale,
                                      void* y, int64_t ldy, int32_t* dev_status, void* stream) {
    using namespace hq;
    using namespace hq::gemm;
    if (x == nullptr || desc == nullptr || w_dev == nullptr || scale_w == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if (xdt != HQ_F32 && xdt != HQ_BF16) return HQ_ERR_INVALID_ARG;
    if (mode != HQ_SCALE_PER_ROW && mode != HQ_SCALE_STATIC) return HQ_ERR_INVALID_ARG;
    if (mode == HQ_SCALE_STATIC && static_scale == nullptr) return HQ_ERR_INVALID_ARG;
    if (a_bits != 3 && a_bits != 4 && a_bits != 8) return HQ_ERR_INVALID_ARG;
    if (desc->container != HQ_CODES_INT8 || desc->RS != 1 || desc->C != K) return HQ_ERR_SHAPE;
    if (desc->limbs != 1 && desc->limbs != 2) return HQ_ERR_INVALID_ARG;
    if (M < 0 || ldx < K || ldy < desc->N) return HQ_ERR_SHAPE;
    if (M == 0) return HQ_OK;
    // shapes this kernel covers: the whole reduction in one operand tile, a row held by 4, 8 or 16 lanes
    if (K != 128 && K != 256 && K != 512) return HQ_ERR_UNSUPPORTED;
    const int n = desc->had_block;
    if (n < 32 || n > K || !is_pow2(n) || K % n != 0) return HQ_ERR_UNSUPPORTED;
    if (M > (int64_t(1) << 30)) return HQ_ERR_UNSUPPORTED;
    const int elt = xdt == HQ_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(x) % (4 * elt) != 0 || ldx % 4 != 0) return HQ_ERR_ALIGNMENT;
    if (!aligned16(w_dev) || !aligned16(y) || (ldy * 2) % 16 != 0) return HQ_ERR_ALIGNMENT;
    const double bound = double(K) * double(1 << (a_bits - 1)) * double(desc->max_abs_b > 0 ? desc->max_abs_b : 1);
    if (bound >= 2147483648.0) return HQ_ERR_OVERFLOW_RISK;

    FusedParams p{};
    p.x = x; p.ldx = ldx; p.M = M; p.K = int(K); p.N = int(desc->N); p.limbs = desc->limbs;
    p.num_kb = int(desc->C_pad / kBK);
    p.tiles_m = int((M + kBM - 1) / kBM);
    p.tiles_n = int(desc->limbs == 2 ? desc->N_pad / 128 : (desc->N_pad + 255) / 256);
    p.bits = a_bits;
    p.norm = float(exp2(-0.5 * double(ilog2(n))));
    p.static_scale = mode == HQ_SCALE_STATIC ? static_scale : nullptr;
    p.scale_w = scale_w; p.bias = bias; p.alpha = hq_alpha_for(desc); p.dev_status = dev_status;
    size_t smem = 0;
    for (int stages = kFusedMaxStages; stages >= 2; --stages) {
        const FusedLayout L = fused_layout(p.num_kb, stages);
        if (L.total <= kSmemLimit) { p.stages = stages; smem = size_t(L.total); break; }
    }
    if (smem == 0) return HQ_ERR_UNSUPPORTED;
    CUtensorMap tmB, tmY;
    const uint64_t Kp = uint64_t(desc->C_pad);
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, kBN, true)) return HQ_ERR_CUDA;
    if (!encode_y(&tmY, y, uint64_t(desc->N), uint64_t(M), uint64_t(ldy))) return HQ_ERR_CUDA;
    const int tiles = p.tiles_m * p.tiles_n;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool is_static = mode == HQ_SCALE_STATIC;
    cudaError_t e = xdt == HQ_F32 ? dispatch_fused<float>(ilog2(n), p, is_static, grid, smem, st, tmB, tmY)
                                  : dispatch_fused<__nv_bfloat16>(ilog2(n), p, is_static, grid, smem, st, tmB, tmY);
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
