// Fused online Hadamard transform + symmetric quantization (Eq. 10 with Eq. 5-7, then Eq. 3), and its variants.
//
// HBM-bound: every input element is read once (16-byte loads) and 0.5 or 1 byte is written.
//   fwht_quant_fast     Hadamard blocks of n = 2^k channels, k = 5..12: a block is owned by n/E threads that hold E = 32
//                       (64 for k >= 10) values each as two-wide fp32 registers; two in-register butterfly phases around
//                       one trip through a padded shared-memory buffer cover all k stages (k = 12: one lane exchange
//                       more); then the row maximum (shuffles, plus a shared-memory maximum when a row spans several
//                       blocks or warps), the scale, round-half-even by a magic-number add, packing, 16-byte stores.
//                       Optional prologues applied as the values are loaded: GroupNorm (+ SiLU) with given statistics,
//                       or LayerNorm over the row with a per-sample affine.
//   fwht_quant_generic  every other block size, including the identity: one row per CTA in shared memory.
//   width_quant_kernel  the transform along the width axis of an NHWC tensor (Eq. 13-14 as stated), static scale,
//                       followed by the integer factor q * H_raw.
//   gn_stats_kernel     per-(sample, group) mean and 1/sqrt(var + eps) for the GroupNorm prologue, in one launch.
// The butterflies run unnormalised (H_raw); 2^(-k/2) is folded into the scale (Eq. 7).
#include <type_traits>

#include "hq_common.cuh"
#include "hq_fwht.cuh"

namespace hq {
int sm_count();             // hq_gemm.cu: SM count of the current device

namespace {

struct QuantParams {
    const void* x;
    int64_t rows, cols, ldx;
    // optional second source: columns [split, cols) of every row come from x2 (pitch ldx2), columns [0, split) from x --
    // the channel concatenation of two tensors read in place (split is a multiple of the Hadamard block)
    const void* x2;
    int64_t split, ldx2;
    int m;               // Hadamard blocks per row
    int rows_per_cta;
    int threads_per_row;
    int bits;
    float norm;          // 2^(-k/2) (1 for the identity)
    const float* static_scale;
    uint8_t* codes;
    int64_t ld_codes;
    float* scales;
    // optional GroupNorm + SiLU applied to the values as they are loaded (gn_stats == nullptr: off)
    const float* gn_stats;   // [samples][groups][2]: mean, 1/sqrt(var + eps)
    const float* gn_gamma;   // [cols]
    const float* gn_beta;    // [cols]
    int gn_groups;
    int gn_silu;             // 1: SiLU after the normalisation, 0: none
    const __nv_bfloat16* gn_pre_bias;   // [samples][cols] added to x before the normalisation, or nullptr
    int gn_sets_per_sample;  // CTAs per sample (a CTA never straddles two samples)
    int gn_cg;               // channels per group, and its log2 when it is a power of two (else -1)
    int gn_cg_shift;
    // optional LayerNorm over each row with a per-sample affine, applied before the transform (ln_on != 0)
    int ln_on;
    const float* ln_w;       // [groups][cols] or nullptr (= 1)
    const float* ln_b;       // [groups][cols] or nullptr (= 0)
    int64_t ln_rows_per_group;   // rows that share one affine vector pair; 0: all rows
    float ln_eps;
};

// y * sigmoid(y) = y / (1 + 2^(-y log2 e)) for two values: the exponential and the reciprocal are one special-function
// instruction each (the flush-to-zero forms: the plain forms are expanded into sequences that rescale subnormal operands,
// which tripled the instruction count of the prologue); everything else is two-wide.  A large negative y gives
// 2^(...) = inf, 1 / inf = 0 and y * 0 = -0; a subnormal exponential is flushed to 0 and leaves y.
__device__ __forceinline__ float ex2_ftz(float x) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float rcp_ftz(float x) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ f32x2 silu2(f32x2 y) {
    constexpr float kNegLog2e = -1.4426950408889634f;
    float z0, z1, d0, d1;
    upk2(mul2(y, pk2(kNegLog2e, kNegLog2e)), z0, z1);
    upk2(add2(pk2(ex2_ftz(z0), ex2_ftz(z1)), pk2(1.0f, 1.0f)), d0, d1);
    return mul2(y, pk2(rcp_ftz(d0), rcp_ftz(d1)));
}

__device__ __forceinline__ float4 load4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
    uint2 raw = __ldcs(reinterpret_cast<const uint2*>(p));
    float4 f;
    f.x = __uint_as_float(raw.x << 16);
    f.y = __uint_as_float(raw.x & 0xFFFF0000u);
    f.z = __uint_as_float(raw.y << 16);
    f.w = __uint_as_float(raw.y & 0xFFFF0000u);
    return f;
}

// Fast path.  A Hadamard block of n = 2^KLOG channels is owned by TB = n / E threads that hold E values each, as
// E/2 two-wide registers (butterflies between pairs are one instruction per two values).
//   phase A  thread t holds the float4s {t + TB i}: coalesced 16-byte loads; the E-point in-register transform
//            covers index bits {0, 1} and the top log2(E) - 2 bits;
//   exchange one trip through shared memory; float4 slot f sits at f + f / J (one slot of padding per J), which
//            makes both access patterns conflict-free with addresses that are a base plus compile-time offsets;
//   phase B  the remaining R = KLOG - log2(E) index bits {2 .. R+1} are done in registers again.  If R leaves room
//            for both low bits, thread u holds the E contiguous channels E u ..; otherwise (PAIR) it holds the
//            channel pairs {4 j, 4 j + 1} + 2 (u & 1) of a 2E-channel group, read as float2, and after packing the
//            two threads of a group interleave their bytes with one shuffle so that each stores contiguous bytes.
//            KLOG = 12 needs one more stage than fits and takes it with a lane exchange.
// Dynamic scales never need the clamp (|t| * qmax / max|t| rounds to at most qmax); static scales do.
// PRO: prologue applied to the values before the transform: 0 none, 1 GroupNorm + SiLU (statistics given), 2 LayerNorm
// over the row (statistics taken here: the row is in the registers of its threads) with a per-sample affine, 3 GroupNorm
// alone (the normalisation in front of an attention block's QKV projection).
template <int KLOG, int E, typename InT, bool INT8_OUT, bool STATIC, int PRO>
__global__ void __launch_bounds__(320) fwht_quant_fast(const QuantParams p) {
    constexpr bool GN = PRO == 1 || PRO == 3;          // 3: GroupNorm without the SiLU
    constexpr bool GN_SILU = PRO == 1;
    constexpr bool LN = PRO == 2;
    griddep_launch();      // a GEMM launched as a programmatic dependent may start its prologue as this grid drains
    constexpr int N = 1 << KLOG;
    constexpr int LE = ilog2_c(E);
    constexpr int P = E / 2;                           // two-wide registers per thread
    constexpr int TB = N / E;                          // threads per Hadamard block
    constexpr int R = KLOG - LE;                       // index bits left for phase B
    constexpr bool PAIR = R >= LE - 1;
    static_assert(R <= LE, "block too large for this thread shape");
    constexpr int J = PAIR ? E / 2 : E / 4;            // float4 slots a phase-B thread (pair) walks
    constexpr int S = ilog2_c(J);
    static_assert(TB % J == 0 || J % TB == 0, "exchange layout needs TB and J to divide one another");
    constexpr int GS = N / 4 + (N / 4) / J;            // padded float4 slots per Hadamard block
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4* xch = reinterpret_cast<float4*>(smem_raw);
    unsigned int* rowmax = reinterpret_cast<unsigned int*>(smem_raw + size_t(blockDim.x / TB) * GS * 16);

    const int tid = threadIdx.x;
    const int row_in_cta = tid / p.threads_per_row;
    const int tr = tid - row_in_cta * p.threads_per_row;
    const int blk = tr / TB;
    const int tb = tr & (TB - 1);
    const bool shared_max = (p.m > 1) || (TB > 32);

    if (!STATIC && tid < p.rows_per_cta) rowmax[tid] = 0u;

    // GroupNorm + SiLU prologue: per-channel y = x * a[c] + b[c] with a = rstd * gamma, b = beta - mean * a of the
    // sample the CTA's rows belong to (the host makes sure a CTA never straddles two samples), then y * sigmoid(y).
    float* gn_a = reinterpret_cast<float*>(rowmax + ((p.rows_per_cta + 3) & ~3));
    float* gn_b = gn_a + p.cols;
    // LayerNorm prologue: two sums per row, gathered in shared memory (the affine vectors of the CTA's sample are read
    // from global memory as they are used: a CTA holds only a few rows, a table of its own would cost more than it saves)
    float* lnacc = gn_a;                               // [rows_per_cta][2]
    if (LN) {
        if (tid < 2 * p.rows_per_cta) lnacc[tid] = 0.f;
        __syncthreads();
    }

    // The rows' values are requested first, so that the table below is built while they are on their way.
    using Raw = typename std::conditional<sizeof(InT) == 4, float4, uint2>::type;
    const int64_t row = int64_t(blockIdx.x) * p.rows_per_cta + row_in_cta;
    const bool valid = row < p.rows;                   // rows past the end work on row 0's values and store nothing
    Raw cur[E / 4];
    {
        const int64_t c0 = int64_t(blk) * N, r = valid ? row : 0;
        const InT* src = (p.x2 != nullptr && c0 >= p.split)
                             ? reinterpret_cast<const InT*>(p.x2) + r * p.ldx2 + (c0 - p.split)
                             : reinterpret_cast<const InT*>(p.x) + r * p.ldx + c0;
#pragma unroll
        for (int i = 0; i < E / 4; ++i) cur[i] = __ldcs(reinterpret_cast<const Raw*>(src + 4 * (tb + TB * i)));
    }
    if (GN) {
        const unsigned sample = blockIdx.x / unsigned(p.gn_sets_per_sample);
        const float2* st = reinterpret_cast<const float2*>(p.gn_stats) + size_t(sample) * p.gn_groups;
        for (int c = 4 * tid; c < int(p.cols); c += 4 * blockDim.x) {      // a channel quad lies in one group
            const float2 ms = __ldg(st + (p.gn_cg_shift >= 0 ? c >> p.gn_cg_shift : c / p.gn_cg));
            const float4 gm = __ldg(reinterpret_cast<const float4*>(p.gn_gamma + c));
            const float4 bt = __ldg(reinterpret_cast<const float4*>(p.gn_beta + c));
            const float4 a = make_float4(ms.y * gm.x, ms.y * gm.y, ms.y * gm.z, ms.y * gm.w);
            // (x + e - mean) a + beta = x a + (beta + (e - mean) a): the per-sample addend e costs nothing per element
            float4 sh = make_float4(-ms.x, -ms.x, -ms.x, -ms.x);
            if (p.gn_pre_bias != nullptr) {
                const uint2 er = __ldg(reinterpret_cast<const uint2*>(p.gn_pre_bias + size_t(sample) * p.cols + c));
                sh.x += __uint_as_float(er.x << 16); sh.y += __uint_as_float(er.x & 0xFFFF0000u);
                sh.z += __uint_as_float(er.y << 16); sh.w += __uint_as_float(er.y & 0xFFFF0000u);
            }
            *reinterpret_cast<float4*>(gn_a + c) = a;
            *reinterpret_cast<float4*>(gn_b + c) = make_float4(fmaf(sh.x, a.x, bt.x), fmaf(sh.y, a.y, bt.y),
                                                               fmaf(sh.z, a.z, bt.z), fmaf(sh.w, a.w, bt.w));
        }
        __syncthreads();
    }

    f32x2 v[P];
    {
#pragma unroll
        for (int i = 0; i < E / 4; ++i) {
            float4 f;
            if constexpr (sizeof(InT) == 4) {
                f = cur[i];
            } else {
                f = make_float4(__uint_as_float(cur[i].x << 16), __uint_as_float(cur[i].x & 0xFFFF0000u),
                                __uint_as_float(cur[i].y << 16), __uint_as_float(cur[i].y & 0xFFFF0000u));
            }
            v[2 * i] = pk2(f.x, f.y);
            v[2 * i + 1] = pk2(f.z, f.w);
            if (GN) {
                const int ch = blk * N + 4 * (tb + TB * i);
                const float4 a4 = *reinterpret_cast<const float4*>(gn_a + ch);
                const float4 b4 = *reinterpret_cast<const float4*>(gn_b + ch);
                v[2 * i] = fma2(v[2 * i], pk2(a4.x, a4.y), pk2(b4.x, b4.y));
                v[2 * i + 1] = fma2(v[2 * i + 1], pk2(a4.z, a4.w), pk2(b4.z, b4.w));
                if (GN_SILU) { v[2 * i] = silu2(v[2 * i]); v[2 * i + 1] = silu2(v[2 * i + 1]); }
            }
        }
    }
    if (LN) {
        // mean, then the sum of squared deviations (two passes over the registers), each gathered per row through a
        // shared-memory sum; y = (x - mean) * rstd * w[c] + b[c]
        // four neighbouring lanes belong to one row when the row's thread count is a multiple of 4: add them up by
        // shuffles first, so that a quarter of the threads go to shared memory
        const bool quad = (p.threads_per_row & 3) == 0;
        f32x2 acc = v[0];
#pragma unroll
        for (int i = 1; i < P; ++i) acc = add2(acc, v[i]);
        float lo, hi;
        upk2(acc, lo, hi);
        float part = lo + hi;
        if (quad) { part += __shfl_xor_sync(0xffffffffu, part, 1); part += __shfl_xor_sync(0xffffffffu, part, 2); }
        if (!quad || (tid & 3) == 0) atomicAdd(&lnacc[2 * row_in_cta], part);
        __syncthreads();
        const float mean = lnacc[2 * row_in_cta] / float(p.cols);
        const f32x2 mean2 = pk2(mean, mean);
        acc = pk2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < P; ++i) { v[i] = sub2(v[i], mean2); acc = fma2(v[i], v[i], acc); }
        upk2(acc, lo, hi);
        part = lo + hi;
        if (quad) { part += __shfl_xor_sync(0xffffffffu, part, 1); part += __shfl_xor_sync(0xffffffffu, part, 2); }
        if (!quad || (tid & 3) == 0) atomicAdd(&lnacc[2 * row_in_cta + 1], part);
        __syncthreads();
        const float rstd = rsqrtf(lnacc[2 * row_in_cta + 1] / float(p.cols) + p.ln_eps);
        const f32x2 rstd2 = pk2(rstd, rstd);
        const int64_t g = p.ln_rows_per_group > 0 ? (int64_t(blockIdx.x) * p.rows_per_cta) / p.ln_rows_per_group : 0;
        const float* wrow = p.ln_w != nullptr ? p.ln_w + g * p.cols : nullptr;
        const float* brow = p.ln_b != nullptr ? p.ln_b + g * p.cols : nullptr;
#pragma unroll
        for (int i = 0; i < E / 4; ++i) {
            const int ch = blk * N + 4 * (tb + TB * i);
            const float4 a4 = wrow != nullptr ? __ldg(reinterpret_cast<const float4*>(wrow + ch)) : make_float4(1.f, 1.f, 1.f, 1.f);
            const float4 b4 = brow != nullptr ? __ldg(reinterpret_cast<const float4*>(brow + ch)) : make_float4(0.f, 0.f, 0.f, 0.f);
            v[2 * i] = valid ? fma2(mul2(v[2 * i], rstd2), pk2(a4.x, a4.y), pk2(b4.x, b4.y)) : pk2(0.f, 0.f);
            v[2 * i + 1] = valid ? fma2(mul2(v[2 * i + 1], rstd2), pk2(a4.z, a4.w), pk2(b4.z, b4.w)) : pk2(0.f, 0.f);
        }
    }
    float4* grp = xch + (tid / TB) * GS;
    if (TB > 32 || shared_max) fwht_stages<KLOG, E, true>(v, grp, tb);
    else fwht_stages<KLOG, E, false>(v, grp, tb);

    float inv, scale;
    if (!STATIC) {
        float amax = 0.f;
#pragma unroll
        for (int e = 0; e < P; ++e) {
            float a, b;
            upk2(v[e], a, b);
            amax = max3(amax, fabsf(a), fabsf(b));
        }
#pragma unroll
        for (int off = 1; off < (TB < 32 ? TB : 32); off <<= 1)
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
        if (shared_max) {
            if ((tb & 31) == 0) atomicMax(&rowmax[row_in_cta], __float_as_uint(amax));
            __syncthreads();
            amax = __uint_as_float(rowmax[row_in_cta]);
        }
        const float qmaxf = float((1 << (p.bits - 1)) - 1);
        if (amax > 0.f) {
            scale = amax * (p.norm / qmaxf);
            inv = qmaxf / amax;
            if (!(scale > 0.f)) { scale = 1.0f; inv = p.norm; }   // scale underflowed: same rule as an all-zero row
        } else {
            scale = 1.0f;
            inv = 0.f;
        }
    } else {
        scale = __ldg(p.static_scale);
        inv = p.norm / scale;
    }

    constexpr int NW = INT8_OUT ? E / 4 : E / 8;       // packed words per thread
    uint32_t w[NW];
    pack_codes<KLOG, E, INT8_OUT, STATIC>(v, inv, p.bits, tb, w);
    if (valid) {
        uint8_t* dst = p.codes + row * p.ld_codes + (int64_t(blk) * N + E * tb) / (INT8_OUT ? 1 : 2);
#pragma unroll
        for (int i = 0; i < NW / 4; ++i)
            reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        if (p.scales != nullptr) {
            if (!STATIC) { if (tr == 0) p.scales[row] = scale; }
            else if (row == 0 && tr == 0) p.scales[0] = scale;
        }
    }
}

// Generic path: one CTA per row (grid-stride), the row lives in shared memory, one __syncthreads per stage.
template <typename InT>
__global__ void __launch_bounds__(256) fwht_quant_generic(const QuantParams p, int had_block, int int8_out) {
    griddep_launch();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* buf = reinterpret_cast<float*>(smem_raw);
    __shared__ float red[8];
    __shared__ float s_amax;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int cols = int(p.cols);
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
        const InT* src = reinterpret_cast<const InT*>(p.x) + row * p.ldx;
        for (int j = tid; j < cols; j += nthr) {
            float f;
            if (sizeof(InT) == 4) f = reinterpret_cast<const float*>(src)[j];
            else f = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(src)[j]);
            buf[j] = f;
        }
        __syncthreads();
        for (int h = 1; h < had_block; h <<= 1) {
            for (int pr = tid; pr < cols / 2; pr += nthr) {
                const int i = (pr / h) * 2 * h + (pr % h);
                const float a = buf[i], b = buf[i + h];
                buf[i] = a + b;
                buf[i + h] = a - b;
            }
            __syncthreads();
        }
        float inv, scale;
        if (p.static_scale == nullptr) {
            float amax = 0.f;
            for (int j = tid; j < cols; j += nthr) amax = fmaxf(amax, fabsf(buf[j]));
            for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
            if ((tid & 31) == 0) red[tid >> 5] = amax;
            __syncthreads();
            if (tid == 0) {
                float a = 0.f;
                for (int w = 0; w < (nthr + 31) / 32; ++w) a = fmaxf(a, red[w]);
                s_amax = a;
            }
            __syncthreads();
            amax = s_amax;
            const float qmaxf = float((1 << (p.bits - 1)) - 1);
            if (amax > 0.f) {
                scale = amax * (p.norm / qmaxf);
                inv = qmaxf / amax;
                if (!(scale > 0.f)) { scale = 1.0f; inv = p.norm; }
            } else { scale = 1.0f; inv = 0.f; }
        } else {
            scale = __ldg(p.static_scale);
            inv = p.norm / scale;
        }
        const float lo = kMagic + float(-(1 << (p.bits - 1))), hi = kMagic + float((1 << (p.bits - 1)) - 1);
        uint8_t* dst = p.codes + row * p.ld_codes;
        if (int8_out) {
            for (int j = tid; j < cols; j += nthr) {
                const float f = fminf(fmaxf(fmaf(buf[j], inv, kMagic), lo), hi);
                dst[j] = uint8_t(__float_as_uint(f) & 0xFFu);
            }
        } else {
            for (int j = tid; j < cols / 2; j += nthr) {
                const float f0 = fminf(fmaxf(fmaf(buf[2 * j], inv, kMagic), lo), hi);
                const float f1 = fminf(fmaxf(fmaf(buf[2 * j + 1], inv, kMagic), lo), hi);
                dst[j] = uint8_t((__float_as_uint(f0) & 0xFu) | ((__float_as_uint(f1) & 0xFu) << 4));
            }
        }
        if (tid == 0 && p.scales != nullptr) {
            if (p.static_scale == nullptr) p.scales[row] = scale;
            else if (row == 0) p.scales[0] = scale;
        }
        __syncthreads();
    }
}

// ---- width-axis variant (Eq. 13-14 as stated): transform along w, quantize, integer factor q * H_raw ---------
// x is NHWC; a thread owns 4 consecutive channels of one block of NB positions along w (loads and stores of a warp
// are contiguous over channels).  Per channel: NB-point transform in registers, static-scale quantization
// (ties to even, clamp), then the +-1 transform again on the codes (exact small integers in fp32) and a byte store.
struct WidthParams {
    const void* x;
    int64_t items;        // Nb * H * (W / NB) * (C / 4)
    int64_t C;
    int c4;               // C / 4
    int wblocks;          // W / NB
    int bits;
    float norm;           // 2^(-k/2)
    const float* static_scale;
    int8_t* z;
    float* scale_out;     // receives S * 2^(-k/2), the one activation scale of the integer convolution
};

template <int NB, typename InT>
__global__ void __launch_bounds__(256) width_quant_kernel(const WidthParams p) {
    griddep_launch();
    const int64_t item = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const float S = __ldg(p.static_scale);
    if (item == 0 && p.scale_out != nullptr) p.scale_out[0] = S * p.norm;
    if (item >= p.items) return;
    const int c4 = int(item % p.c4);
    const int64_t rest = item / p.c4;
    const int b = int(rest % p.wblocks);
    const int64_t nh = rest / p.wblocks;
    const int64_t base = ((nh * p.wblocks + b) * NB) * p.C + 4 * c4;      // element offset of (nh, w = b*NB, c)
    const InT* src = reinterpret_cast<const InT*>(p.x) + base;

    f32x2 v[NB][2];                                   // [position along w][channel pair]
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        const float4 f = load4(src + int64_t(i) * p.C);
        v[i][0] = pk2(f.x, f.y);
        v[i][1] = pk2(f.z, f.w);
    }
#pragma unroll
    for (int h = 1; h < NB; h <<= 1) {
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            if (!(i & h)) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const f32x2 a = v[i][c], bb = v[i | h][c];
                    v[i][c] = add2(a, bb);
                    v[i | h][c] = sub2(a, bb);
                }
            }
        }
    }
    // codes as integer-valued floats: round by the magic add, clamp, take the magic off again
    const float inv = p.norm / S;
    const float lo = kMagic + float(-(1 << (p.bits - 1))), hi = kMagic + float((1 << (p.bits - 1)) - 1);
    const f32x2 inv2 = pk2(inv, inv), mg2 = pk2(kMagic, kMagic);
#pragma unroll
    for (int i = 0; i < NB; ++i) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            float a, bb;
            upk2(fma2(v[i][c], inv2, mg2), a, bb);
            a = fminf(fmaxf(a, lo), hi) - kMagic;
            bb = fminf(fmaxf(bb, lo), hi) - kMagic;
            v[i][c] = pk2(a, bb);
        }
    }
#pragma unroll
    for (int h = 1; h < NB; h <<= 1) {
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            if (!(i & h)) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const f32x2 a = v[i][c], bb = v[i | h][c];
                    v[i][c] = add2(a, bb);
                    v[i | h][c] = sub2(a, bb);
                }
            }
        }
    }
    int8_t* dst = p.z + base;
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        float a0, a1, a2, a3;
        upk2(add2(v[i][0], mg2), a0, a1);
        upk2(add2(v[i][1], mg2), a2, a3);
        // the low byte of (magic + z) is z in two's complement
        const uint32_t w01 = __byte_perm(__float_as_uint(a0), __float_as_uint(a1), 0x0040);
        const uint32_t w23 = __byte_perm(__float_as_uint(a2), __float_as_uint(a3), 0x0040);
        *reinterpret_cast<uint32_t*>(dst + int64_t(i) * p.C) = __byte_perm(w01, w23, 0x5410);
    }
}

// The same for blocks of 32 or 64 positions, where z = q * H_raw needs more than a signed byte: a thread owns 2 consecutive
// channels of one block of NB positions, and z leaves as two int8 limbs, z = 256 * hi + lo with lo in [-128, 127], laid
// out per pixel as [hi(C) | lo(C)] (the operand of a convolution whose weights were prepared for two activation limbs).
struct Width2Params {
    const void* x;
    int64_t items;        // Nb * H * (W / NB) * (C / 2)
    int64_t C;
    int c2;               // C / 2
    int wblocks;          // W / NB
    int bits;
    float norm;           // 2^(-k/2)
    const float* static_scale;
    int8_t* z;            // [pixels][2 C]
    float* scale_out;
};

template <int NB, typename InT>
__global__ void __launch_bounds__(128) width_quant2_kernel(const Width2Params p) {
    griddep_launch();
    const int64_t item = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const float S = __ldg(p.static_scale);
    if (item == 0 && p.scale_out != nullptr) p.scale_out[0] = S * p.norm;
    if (item >= p.items) return;
    const int c2 = int(item % p.c2);
    const int64_t rest = item / p.c2;
    const int b = int(rest % p.wblocks);
    const int64_t nh = rest / p.wblocks;
    const int64_t pix0 = (nh * p.wblocks + b) * NB;                 // first pixel of the block
    const InT* src = reinterpret_cast<const InT*>(p.x) + pix0 * p.C + 2 * c2;

    f32x2 v[NB];                                                    // [position along w], one channel pair
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        if (sizeof(InT) == 4) {
            const float2 f = __ldcs(reinterpret_cast<const float2*>(src + int64_t(i) * p.C));
            v[i] = pk2(f.x, f.y);
        } else {
            const uint32_t raw = __ldcs(reinterpret_cast<const uint32_t*>(src + int64_t(i) * p.C));
            v[i] = pk2(__uint_as_float(raw << 16), __uint_as_float(raw & 0xFFFF0000u));
        }
    }
    butterflies_pairs<NB, 1, NB / 2>(v);
    const float inv = p.norm / S;
    const float lo = kMagic + float(-(1 << (p.bits - 1))), hi = kMagic + float((1 << (p.bits - 1)) - 1);
    const f32x2 inv2 = pk2(inv, inv), mg2 = pk2(kMagic, kMagic);
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        float a, bb;
        upk2(fma2(v[i], inv2, mg2), a, bb);
        v[i] = pk2(fminf(fmaxf(a, lo), hi) - kMagic, fminf(fmaxf(bb, lo), hi) - kMagic);
    }
    butterflies_pairs<NB, 1, NB / 2>(v);                            // z = q * H_raw: small integers, exact in fp32
    int8_t* dst = p.z + pix0 * 2 * p.C + 2 * c2;
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        float a, bb;
        upk2(v[i], a, bb);
        const int z0 = __float2int_rn(a), z1 = __float2int_rn(bb);
        const int l0 = ((z0 + 128) & 255) - 128, l1 = ((z1 + 128) & 255) - 128;
        const int h0 = (z0 - l0) >> 8, h1 = (z1 - l1) >> 8;
        int8_t* px = dst + int64_t(i) * 2 * p.C;
        *reinterpret_cast<uint16_t*>(px) = uint16_t((h0 & 255) | ((h1 & 255) << 8));
        *reinterpret_cast<uint16_t*>(px + p.C) = uint16_t((l0 & 255) | ((l1 & 255) << 8));
    }
}

// ---- GroupNorm statistics: sums and sums of squares per (sample, group), then mean and 1/sqrt(var + eps) --------
// x NHWC; one wave of CTAs, each with an equal share of the pixels of all samples, cut into segments where it crosses a
// sample boundary.  A thread owns one 16-byte (bf16 with VEC = 4: 8-byte) piece of a pixel's
// channels -- VEC / 4 channel quads, and a quad never straddles two groups -- and walks the pixels of the segment
// with eight loads in flight; the 32 values a quad collects per round are added two-wide in fp32 and then carried in
// fp64.  The pixel lanes of the CTA meet in shared memory, one fp64 atomic pair per quad (per piece when it lies in one
// group) and segment goes to global memory, and the CTA whose segment completes a sample's pixel count turns the
// sample's sums into the statistics.  The pixel counter is the sample's first statistics word (cleared with the sums by the host,
// overwritten by the mean at the end).
template <int VEC>
struct GnPiece;
template <>
struct GnPiece<4> { float4 d; };
template <>
struct GnPiece<8> { uint4 d; };
__device__ __forceinline__ GnPiece<4> gn_load(const float* p, GnPiece<4>*) { return {__ldg(reinterpret_cast<const float4*>(p))}; }
__device__ __forceinline__ GnPiece<4> gn_load(const __nv_bfloat16* p, GnPiece<4>*) {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(p));
    return {make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xFFFF0000u), __uint_as_float(r.y << 16),
                        __uint_as_float(r.y & 0xFFFF0000u))};
}
__device__ __forceinline__ GnPiece<8> gn_load(const __nv_bfloat16* p, GnPiece<8>*) { return {__ldg(reinterpret_cast<const uint4*>(p))}; }
// The two value pairs of quad q of a piece.
__device__ __forceinline__ void gn_quad(const GnPiece<4>& r, int, f32x2& lo, f32x2& hi) {
    lo = pk2(r.d.x, r.d.y);
    hi = pk2(r.d.z, r.d.w);
}
__device__ __forceinline__ void gn_quad(const GnPiece<8>& r, int q, f32x2& lo, f32x2& hi) {
    const uint32_t w0 = q == 0 ? r.d.x : r.d.z, w1 = q == 0 ? r.d.y : r.d.w;
    lo = pk2(__uint_as_float(w0 << 16), __uint_as_float(w0 & 0xFFFF0000u));
    hi = pk2(__uint_as_float(w1 << 16), __uint_as_float(w1 & 0xFFFF0000u));
}

template <typename InT, int VEC>
__global__ void __launch_bounds__(256, 4) gn_stats_kernel(const InT* x, const InT* x2, int split,
                                                          const __nv_bfloat16* pre_bias, int64_t hw, int64_t total_px,
                                                          int64_t span, int C, int groups, double* sums, float* stats,
                                                          double inv_count, double eps) {
    constexpr int Q = VEC / 4;                         // channel quads per piece
    constexpr int U = 8;                               // loads in flight per thread
    __shared__ double red[2 * Q][256];
    __shared__ int s_last;
    const int tid = threadIdx.x;
    const int pieces = C / VEC;
    const int nq = pieces < 256 ? pieces : 256;        // pieces walked side by side
    const int ppl = 256 / nq;                          // pixels walked side by side
    const int col0 = tid % nq, pl = tid / nq;
    const int cg = C / groups;
    // the CTA's share of the pixels of all samples, cut into segments at the sample boundaries
    int64_t r0 = int64_t(blockIdx.x) * span;
    const int64_t r1 = r0 + span < total_px ? r0 + span : total_px;
    while (r0 < r1) {
        const int64_t sample = r0 / hw;
        const int64_t seg_end = (sample + 1) * hw < r1 ? (sample + 1) * hw : r1;
        double* out = sums + sample * 2 * groups;
        for (int cbase = 0; cbase < pieces; cbase += nq) {
            const int col = cbase + col0;
            double s1[Q], s2[Q];
            f32x2 e_lo[Q], e_hi[Q];                    // the sample's addend on this thread's channels (zero: none)
#pragma unroll
            for (int q = 0; q < Q; ++q) { s1[q] = 0.0; s2[q] = 0.0; e_lo[q] = pk2(0.f, 0.f); e_hi[q] = pk2(0.f, 0.f); }
            if (pl < ppl && col < pieces) {
                if (pre_bias != nullptr) {
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        const uint2 er = __ldg(reinterpret_cast<const uint2*>(pre_bias + sample * C + int64_t(col) * VEC + 4 * q));
                        e_lo[q] = pk2(__uint_as_float(er.x << 16), __uint_as_float(er.x & 0xFFFF0000u));
                        e_hi[q] = pk2(__uint_as_float(er.y << 16), __uint_as_float(er.y & 0xFFFF0000u));
                    }
                }
                // channels [split, C) of a pixel come from the second tensor when there is one (a piece lies in one of them)
                const int ch = col * VEC;
                const bool second = x2 != nullptr && ch >= split;
                const InT* src = second ? x2 + (ch - split) : x + ch;
                const int64_t pitch = x2 == nullptr ? C : (second ? C - split : split);
                int64_t px = r0 + pl;
                for (; px + (U - 1) * ppl < seg_end; px += U * ppl) {
                    GnPiece<VEC> raw[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) raw[u] = gn_load(src + (px + u * ppl) * pitch, static_cast<GnPiece<VEC>*>(nullptr));
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        f32x2 a = pk2(0.f, 0.f), b = pk2(0.f, 0.f);
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            f32x2 lo, hi;
                            gn_quad(raw[u], q, lo, hi);
                            lo = add2(lo, e_lo[q]);
                            hi = add2(hi, e_hi[q]);
                            a = add2(a, add2(lo, hi));
                            b = fma2(lo, lo, fma2(hi, hi, b));
                        }
                        float a0, a1, b0, b1;
                        upk2(a, a0, a1);
                        upk2(b, b0, b1);
                        s1[q] += double(a0 + a1);
                        s2[q] += double(b0 + b1);
                    }
                }
                for (; px < seg_end; px += ppl) {
                    const GnPiece<VEC> raw = gn_load(src + px * pitch, static_cast<GnPiece<VEC>*>(nullptr));
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        f32x2 lo, hi;
                        gn_quad(raw, q, lo, hi);
                        lo = add2(lo, e_lo[q]);
                        hi = add2(hi, e_hi[q]);
                        float a0, a1, b0, b1;
                        upk2(add2(lo, hi), a0, a1);
                        upk2(fma2(lo, lo, mul2(hi, hi)), b0, b1);
                        s1[q] += double(a0 + a1);
                        s2[q] += double(b0 + b1);
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < Q; ++q) { red[2 * q][tid] = s1[q]; red[2 * q + 1][tid] = s2[q]; }
            __syncthreads();
            if (pl == 0 && col < pieces) {
                double t[2 * Q];
#pragma unroll
                for (int k = 0; k < 2 * Q; ++k) {
                    t[k] = 0.0;
                    for (int j = 0; j < ppl; ++j) t[k] += red[k][j * nq + col0];
                }
                const int g0 = col * VEC / cg;
                const int g1 = (col * VEC + 4 * (Q - 1)) / cg;
                if (g1 == g0) {
                    atomicAdd(out + 2 * g0, Q == 2 ? t[0] + t[2 * (Q - 1)] : t[0]);
                    atomicAdd(out + 2 * g0 + 1, Q == 2 ? t[1] + t[2 * (Q - 1) + 1] : t[1]);
                } else {
                    atomicAdd(out + 2 * g0, t[0]);
                    atomicAdd(out + 2 * g0 + 1, t[1]);
                    atomicAdd(out + 2 * g1, t[2 * (Q - 1)]);
                    atomicAdd(out + 2 * g1 + 1, t[2 * (Q - 1) + 1]);
                }
                __threadfence();
            }
            __syncthreads();
        }
        // tickets count pixels: the CTA whose segment completes the sample sees every CTA's sums
        float* st = stats + sample * 2 * groups;
        if (tid == 0) {
            const unsigned int cnt = unsigned(seg_end - r0);
            s_last = atomicAdd(reinterpret_cast<unsigned int*>(st), cnt) + cnt == unsigned(hw);
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int g = tid; g < groups; g += 256) {
                const double mean = __ldcg(out + 2 * g) * inv_count;
                double var = __ldcg(out + 2 * g + 1) * inv_count - mean * mean;
                if (var < 0.0) var = 0.0;
                *reinterpret_cast<float2*>(st + 2 * g) = make_float2(float(mean), float(1.0 / sqrt(var + eps)));
            }
        }
        __syncthreads();                               // s_last is written again by the next segment
        r0 = seg_end;
    }
}

template <int KLOG, int E, typename InT>
cudaError_t launch_fast(const QuantParams& p, bool int8_out, int grid, int threads, size_t smem, cudaStream_t st) {
    const bool stat = p.static_scale != nullptr;
    auto go = [&](auto kern) -> cudaError_t {
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
            if (e != cudaSuccess) return e;
        }
        kern<<<grid, threads, smem, st>>>(p);
        return cudaGetLastError();
    };
    if (p.gn_stats != nullptr && p.gn_silu) {
        if (int8_out) return stat ? go(fwht_quant_fast<KLOG, E, InT, true, true, 1>) : go(fwht_quant_fast<KLOG, E, InT, true, false, 1>);
        return stat ? go(fwht_quant_fast<KLOG, E, InT, false, true, 1>) : go(fwht_quant_fast<KLOG, E, InT, false, false, 1>);
    }
    if (p.gn_stats != nullptr) {
        if (int8_out) return stat ? go(fwht_quant_fast<KLOG, E, InT, true, true, 3>) : go(fwht_quant_fast<KLOG, E, InT, true, false, 3>);
        return stat ? go(fwht_quant_fast<KLOG, E, InT, false, true, 3>) : go(fwht_quant_fast<KLOG, E, InT, false, false, 3>);
    }
    if (p.ln_on) {
        if (int8_out) return stat ? go(fwht_quant_fast<KLOG, E, InT, true, true, 2>) : go(fwht_quant_fast<KLOG, E, InT, true, false, 2>);
        return stat ? go(fwht_quant_fast<KLOG, E, InT, false, true, 2>) : go(fwht_quant_fast<KLOG, E, InT, false, false, 2>);
    }
    if (int8_out) return stat ? go(fwht_quant_fast<KLOG, E, InT, true, true, 0>) : go(fwht_quant_fast<KLOG, E, InT, true, false, 0>);
    return stat ? go(fwht_quant_fast<KLOG, E, InT, false, true, 0>) : go(fwht_quant_fast<KLOG, E, InT, false, false, 0>);
}

// Values per thread for a block of 2^klog channels.
constexpr int fast_e(int klog) { return klog <= 9 ? 32 : 64; }

template <typename InT>
cudaError_t dispatch_fast(int klog, const QuantParams& p, bool int8_out, int grid, int threads, size_t smem,
                          cudaStream_t st) {
    switch (klog) {
        case 5: return launch_fast<5, 32, InT>(p, int8_out, grid, threads, smem, st);
        case 6: return launch_fast<6, 32, InT>(p, int8_out, grid, threads, smem, st);
        case 7: return launch_fast<7, 32, InT>(p, int8_out, grid, threads, smem, st);
        case 8: return launch_fast<8, fast_e(8), InT>(p, int8_out, grid, threads, smem, st);
        case 9: return launch_fast<9, fast_e(9), InT>(p, int8_out, grid, threads, smem, st);
        case 10: return launch_fast<10, fast_e(10), InT>(p, int8_out, grid, threads, smem, st);
        case 11: return launch_fast<11, fast_e(11), InT>(p, int8_out, grid, threads, smem, st);
        case 12: return launch_fast<12, fast_e(12), InT>(p, int8_out, grid, threads, smem, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

// Launches the transform+quantize kernel; shared by the public entry point and the fused layer calls.
struct GnArgs { const float* stats; const float* gamma; const float* beta; int groups; int64_t rows_per_sample; int silu;
                const __nv_bfloat16* pre_bias; };
struct LnArgs { const float* w; const float* b; int64_t rows_per_group; float eps; };

struct SplitArgs { const void* x2; int64_t split, ldx2; };

static hq_status launch_quant_impl(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, int had_block,
                                   int bits, hq_scale_mode mode, const float* static_scale, void* codes,
                                   hq_container cont, int64_t ld_codes, float* scales, const GnArgs* gn,
                                   cudaStream_t st, const LnArgs* ln = nullptr, const SplitArgs* sp = nullptr) {
    if (rows == 0 && cols > 0) return HQ_OK;                       // nothing to do; pointers may be NULL
    if (x == nullptr || codes == nullptr) return HQ_ERR_INVALID_ARG;
    if (xdt != HQ_F32 && xdt != HQ_BF16) return HQ_ERR_INVALID_ARG;
    if (cont != HQ_CODES_NIBBLE && cont != HQ_CODES_INT8) return HQ_ERR_INVALID_ARG;
    if (mode != HQ_SCALE_PER_ROW && mode != HQ_SCALE_STATIC) return HQ_ERR_INVALID_ARG;
    if (mode == HQ_SCALE_STATIC && static_scale == nullptr) return HQ_ERR_INVALID_ARG;
    if (mode == HQ_SCALE_PER_ROW && scales == nullptr) return HQ_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4 && bits != 8) return HQ_ERR_INVALID_ARG;
    if (rows < 0 || cols <= 0 || ldx < ((sp != nullptr && sp->x2 != nullptr) ? sp->split : cols)) return HQ_ERR_SHAPE;
    if (cont == HQ_CODES_NIBBLE && (bits > 4 || (cols & 1))) return HQ_ERR_SHAPE;
    const int64_t row_bytes = cont == HQ_CODES_NIBBLE ? cols / 2 : cols;
    if (ld_codes < row_bytes) return HQ_ERR_SHAPE;
    if (had_block > 1 && (!is_pow2(had_block) || cols % had_block != 0)) return HQ_ERR_SHAPE;
    const int n = had_block > 1 ? had_block : 1;
    const int klog = ilog2(n);

    QuantParams p{};
    p.x = x; p.rows = rows; p.cols = cols; p.ldx = ldx;
    if (sp != nullptr && sp->x2 != nullptr) {
        // the two-source form exists in the fast kernel only; a Hadamard block never straddles the two tensors
        if (sp->split <= 0 || sp->split >= cols || sp->split % n != 0 || sp->ldx2 < cols - sp->split || ldx < sp->split)
            return HQ_ERR_SHAPE;
        if (reinterpret_cast<uintptr_t>(sp->x2) % (4 * (xdt == HQ_F32 ? 4 : 2)) != 0 || sp->ldx2 % 4 != 0) return HQ_ERR_ALIGNMENT;
        p.x2 = sp->x2; p.split = sp->split; p.ldx2 = sp->ldx2;
    }
    p.m = int(cols / n);
    p.bits = bits;
    p.norm = float(exp2(-0.5 * double(klog)));
    p.static_scale = mode == HQ_SCALE_STATIC ? static_scale : nullptr;
    p.codes = static_cast<uint8_t*>(codes);
    p.ld_codes = ld_codes;
    p.scales = scales;
    if (gn != nullptr) {
        p.gn_stats = gn->stats; p.gn_gamma = gn->gamma; p.gn_beta = gn->beta; p.gn_groups = gn->groups;
        p.gn_silu = gn->silu;
        p.gn_pre_bias = gn->pre_bias;
        p.gn_cg = int(cols / gn->groups);
        p.gn_cg_shift = is_pow2(p.gn_cg) ? ilog2(p.gn_cg) : -1;
    }
    if (ln != nullptr) {
        p.ln_on = 1; p.ln_w = ln->w; p.ln_b = ln->b; p.ln_rows_per_group = ln->rows_per_group; p.ln_eps = ln->eps;
    }

    const int elt = xdt == HQ_F32 ? 4 : 2;
    const int E = fast_e(klog);
    const bool fast_ok = klog >= 5 && klog <= 12 && cols / E <= 256 &&
                         (reinterpret_cast<uintptr_t>(x) % (4 * elt) == 0) && (ldx % 4 == 0) &&
                         aligned16(codes) && (ld_codes % 16 == 0);
    if (fast_ok) {
        // CTAs of about 128 threads (whole warps, whole rows): small enough that many are resident per SM and the
        // load phases of some overlap the arithmetic of others.
        const int tr = int(cols / E);
        int rpc = 1;
        while ((rpc * tr) % 32 != 0) ++rpc;                 // whole warps
        const int base = rpc;
        while ((rpc + base) * tr <= 128) rpc += base;
        p.threads_per_row = tr;
        p.rows_per_cta = rpc;
        const int threads = rpc * tr;
        if (gn != nullptr) {
            if (gn->rows_per_sample % rpc != 0) return HQ_ERR_UNSUPPORTED;               // a CTA must stay in one sample
            if (gn->rows_per_sample / rpc > 0x7fffffff || cols % 4 != 0) return HQ_ERR_UNSUPPORTED;
            if (!aligned16(gn->gamma) || !aligned16(gn->beta)) return HQ_ERR_ALIGNMENT;
            p.gn_sets_per_sample = int(gn->rows_per_sample / rpc);
        }
        if (ln != nullptr && ln->rows_per_group > 0 && ln->rows_per_group % rpc != 0) return HQ_ERR_UNSUPPORTED;
        if (threads <= 320) {                               // otherwise the generic kernel below takes the row shape
        // exchange buffer: per Hadamard block n/4 float4 slots plus one slot of padding per J (J = E/2 or E/4)
        const int jslots = (klog - ilog2(E) >= ilog2(E) - 1) ? E / 2 : E / 4;
        const size_t smem = size_t(threads / (n / E)) * size_t(n / 4 + n / 4 / jslots) * 16 + size_t((rpc + 3) & ~3) * 4 +
                            (gn != nullptr ? size_t(cols) * 8 : 0) + (ln != nullptr ? size_t(rpc) * 8 : 0);
        const int grid = int((rows + rpc - 1) / rpc);
        cudaError_t e = xdt == HQ_F32
                            ? dispatch_fast<float>(klog, p, cont == HQ_CODES_INT8, grid, threads, smem, st)
                            : dispatch_fast<__nv_bfloat16>(klog, p, cont == HQ_CODES_INT8, grid, threads, smem, st);
        return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
        }
    }
    if (gn != nullptr || ln != nullptr || p.x2 != nullptr) return HQ_ERR_UNSUPPORTED;   // these exist in the fast kernel only
    const size_t smem = size_t(cols) * 4;
    if (smem > 200 * 1024) return HQ_ERR_UNSUPPORTED;
    const int grid = int(rows < 148 * 8 ? rows : 148 * 8);
    cudaError_t e;
    if (xdt == HQ_F32) {
        if (smem > 48 * 1024)
            HQ_CUDA_OK(cudaFuncSetAttribute(fwht_quant_generic<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            int(smem)));
        fwht_quant_generic<float><<<grid, 256, smem, st>>>(p, n, cont == HQ_CODES_INT8);
    } else {
        if (smem > 48 * 1024)
            HQ_CUDA_OK(cudaFuncSetAttribute(fwht_quant_generic<__nv_bfloat16>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        fwht_quant_generic<__nv_bfloat16><<<grid, 256, smem, st>>>(p, n, cont == HQ_CODES_INT8);
    }
    e = cudaGetLastError();
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

hq_status launch_hadamard_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, int had_block,
                                int bits, hq_scale_mode mode, const float* static_scale, void* codes,
                                hq_container cont, int64_t ld_codes, float* scales, cudaStream_t st) {
    return launch_quant_impl(x, xdt, rows, cols, ldx, had_block, bits, mode, static_scale, codes, cont, ld_codes, scales,
                             nullptr, st);
}

// The same on the column concatenation [x | x2] of two matrices read in place: x holds columns [0, split), x2 the rest.
hq_status launch_hadamard_quant_cat(const void* x, int64_t ldx, const void* x2, int64_t ldx2, int64_t split, hq_dtype xdt,
                                    int64_t rows, int64_t cols, int had_block, int bits, hq_scale_mode mode,
                                    const float* static_scale, void* codes, hq_container cont, int64_t ld_codes,
                                    float* scales, cudaStream_t st) {
    if (x2 == nullptr) return HQ_ERR_INVALID_ARG;
    const SplitArgs sp{x2, split, ldx2};
    return launch_quant_impl(x, xdt, rows, cols, ldx, had_block, bits, mode, static_scale, codes, cont, ld_codes, scales,
                             nullptr, st, nullptr, &sp);
}

// GroupNorm statistics of an NHWC tensor (hw pixels per sample): fp64 sums per (sample, group) in `scratch` (cleared
// here), then mean and 1/sqrt(var + eps) as floats behind them.  scratch: Nb * groups * (2 doubles + 2 floats).
hq_status launch_gn_stats(const void* x, hq_dtype xdt, int64_t Nb, int64_t hw, int64_t C, int groups, float eps,
                          void* scratch, size_t scratch_bytes, const float** stats_out, cudaStream_t st,
                          const void* pre_bias, const void* x2, int64_t split) {
    if (x == nullptr || scratch == nullptr) return HQ_ERR_INVALID_ARG;
    if (xdt != HQ_F32 && xdt != HQ_BF16) return HQ_ERR_INVALID_ARG;
    if (Nb <= 0 || hw <= 0 || C <= 0 || groups <= 0) return HQ_ERR_SHAPE;
    if (C % groups != 0 || (C / groups) % 4 != 0) return HQ_ERR_SHAPE;      // whole channel quads per group
    if (groups > 1024) return HQ_ERR_UNSUPPORTED;
    const size_t need = size_t(Nb) * groups * (2 * sizeof(double) + 2 * sizeof(float));
    if (scratch_bytes < need) return HQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(scratch) % 16 != 0) return HQ_ERR_ALIGNMENT;
    const int elt = xdt == HQ_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(x) % (4 * elt) != 0) return HQ_ERR_ALIGNMENT;
    if (pre_bias != nullptr && reinterpret_cast<uintptr_t>(pre_bias) % 8 != 0) return HQ_ERR_ALIGNMENT;
    const __nv_bfloat16* pre = static_cast<const __nv_bfloat16*>(pre_bias);
    double* sums = static_cast<double*>(scratch);
    float* stats = reinterpret_cast<float*>(sums + size_t(Nb) * groups * 2);
    HQ_CUDA_OK(cudaMemsetAsync(scratch, 0, need, st));             // the sums and the ticket counters
    if (hw > 0x7fffffff) return HQ_ERR_UNSUPPORTED;                // the tickets count pixels in 32 bits
    // 16-byte pieces (bf16: eight channels) where the shape allows them
    if (x2 != nullptr) {                                           // channels [split, C) of every pixel live in x2
        if (split <= 0 || split >= C || split % 8 != 0 || (C - split) % 8 != 0) return HQ_ERR_SHAPE;
        if (reinterpret_cast<uintptr_t>(x2) % 16 != 0 || reinterpret_cast<uintptr_t>(x) % 16 != 0) return HQ_ERR_ALIGNMENT;
    }
    const bool wide = xdt == HQ_BF16 && C % 8 == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0;
    const int64_t pieces = C / (wide ? 8 : 4);
    const int64_t ppl = pieces < 256 ? 256 / pieces : 1;
    // one wave of CTAs (four per SM) that share the pixels of all samples evenly, in whole rounds of loads; small
    // tensors get fewer CTAs so that a thread still walks a round of eight pixels
    const int64_t total_px = Nb * hw;
    const int64_t round = ppl * 8;
    int64_t ctas = int64_t(sm_count()) * 4;
    int64_t span = ((total_px + ctas - 1) / ctas + round - 1) / round * round;
    ctas = (total_px + span - 1) / span;
    const double inv_count = 1.0 / (double(hw) * double(C / groups));
    const unsigned grid = unsigned(ctas);
    if (xdt == HQ_F32)
        gn_stats_kernel<float, 4><<<grid, 256, 0, st>>>(static_cast<const float*>(x), static_cast<const float*>(x2), int(split), pre, hw, total_px, span, int(C), groups, sums,
                                                       stats, inv_count, double(eps));
    else if (wide)
        gn_stats_kernel<__nv_bfloat16, 8><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(x2), int(split), pre, hw, total_px, span, int(C),
                                                               groups, sums, stats, inv_count, double(eps));
    else
        gn_stats_kernel<__nv_bfloat16, 4><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(x2), int(split), pre, hw, total_px, span, int(C),
                                                               groups, sums, stats, inv_count, double(eps));
    if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
    *stats_out = stats;
    return HQ_OK;
}

// GroupNorm (+ SiLU when `silu`) of an NHWC tensor fused into the transform+quantize kernel: statistics per (sample,
// group) first, then the quantize kernel applies x * a[c] + b[c] and the activation as it loads.
hq_status launch_gn_silu_quant(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups,
                               const float* gamma, const float* beta, float eps, int had_block, int bits,
                               hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont,
                               int64_t ld_codes, float* scales, void* scratch, size_t scratch_bytes, cudaStream_t st,
                               int silu, const void* pre_bias, const void* x2, int64_t split) {
    if (gamma == nullptr || beta == nullptr) return HQ_ERR_INVALID_ARG;
    if (H <= 0 || W <= 0) return HQ_ERR_SHAPE;
    const int64_t hw = H * W;
    const float* stats = nullptr;
    hq_status s = launch_gn_stats(x, xdt, Nb, hw, C, groups, eps, scratch, scratch_bytes, &stats, st, pre_bias, x2, split);
    if (s != HQ_OK) return s;
    const GnArgs gn{stats, gamma, beta, groups, hw, silu, static_cast<const __nv_bfloat16*>(pre_bias)};
    if (x2 != nullptr) {
        const SplitArgs sp{x2, split, C - split};
        return launch_quant_impl(x, xdt, Nb * hw, C, split, had_block, bits, mode, static_scale, codes, cont, ld_codes, scales,
                                 &gn, st, nullptr, &sp);
    }
    return launch_quant_impl(x, xdt, Nb * hw, C, C, had_block, bits, mode, static_scale, codes, cont, ld_codes, scales, &gn,
                             st);
}

// LayerNorm over each row with a per-sample affine, fused into the transform+quantize kernel (one pass: the row's
// statistics are taken from the registers that already hold it).
hq_status launch_ln_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, const float* weight,
                          const float* bias, int64_t rows_per_group, float eps, int had_block, int bits,
                          hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont, int64_t ld_codes,
                          float* scales, cudaStream_t st) {
    if (rows_per_group < 0 || !(eps >= 0.f)) return HQ_ERR_INVALID_ARG;
    if ((weight != nullptr && !aligned16(weight)) || (bias != nullptr && !aligned16(bias)) || cols % 4 != 0) return HQ_ERR_ALIGNMENT;
    const LnArgs ln{weight, bias, rows_per_group, eps};
    return launch_quant_impl(x, xdt, rows, cols, ldx, had_block, bits, mode, static_scale, codes, cont, ld_codes, scales,
                             nullptr, st, &ln);
}

// Width-axis transform + quantization + integer factor of Eq. 13-14: x NHWC fp32/bf16 -> z int8 NHWC.
hq_status launch_hadamard_quant_width(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                      int had_block_w, int bits, const float* static_scale, void* z, float* scale_out,
                                      cudaStream_t st) {
    if (x == nullptr || z == nullptr || static_scale == nullptr) return HQ_ERR_INVALID_ARG;
    if (xdt != HQ_F32 && xdt != HQ_BF16) return HQ_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4 && bits != 8) return HQ_ERR_INVALID_ARG;
    if (Nb <= 0 || H <= 0 || W <= 0 || C <= 0) return HQ_ERR_SHAPE;
    const int nb = had_block_w > 1 ? had_block_w : 1;
    if (!is_pow2(nb) || W % nb != 0) return HQ_ERR_SHAPE;
    // z = q * H_raw must fit a signed byte: nb * 2^(bits-1) <= 128 (16 positions at 4 bits, 32 at 3 bits)
    if (int64_t(nb) << (bits - 1) > 128) return HQ_ERR_OVERFLOW_RISK;
    if (C % 4 != 0) return HQ_ERR_UNSUPPORTED;
    const int elt = xdt == HQ_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(x) % (4 * elt) != 0 || reinterpret_cast<uintptr_t>(z) % 4 != 0) return HQ_ERR_ALIGNMENT;

    WidthParams p{};
    p.x = x; p.C = C; p.c4 = int(C / 4); p.wblocks = int(W / nb); p.bits = bits;
    p.items = Nb * H * (W / nb) * (C / 4);
    p.norm = float(exp2(-0.5 * double(ilog2(nb))));
    p.static_scale = static_scale; p.z = static_cast<int8_t*>(z); p.scale_out = scale_out;
    const int threads = 256;
    const int64_t grid64 = (p.items + threads - 1) / threads;
    if (grid64 > 0x7FFFFFFF) return HQ_ERR_UNSUPPORTED;
    const int grid = int(grid64);
#define HQ_WIDTH_CASE(NBV)                                                                              \
    case NBV:                                                                                           \
        if (xdt == HQ_F32) width_quant_kernel<NBV, float><<<grid, threads, 0, st>>>(p);                 \
        else width_quant_kernel<NBV, __nv_bfloat16><<<grid, threads, 0, st>>>(p);                       \
        break;
    switch (nb) {
        HQ_WIDTH_CASE(1) HQ_WIDTH_CASE(2) HQ_WIDTH_CASE(4) HQ_WIDTH_CASE(8) HQ_WIDTH_CASE(16) HQ_WIDTH_CASE(32)
        default: return HQ_ERR_UNSUPPORTED;
    }
#undef HQ_WIDTH_CASE
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

// Width-axis transform + quantization + integer factor for blocks of up to 64 positions: z as two int8 limbs per channel.
hq_status launch_hadamard_quant_width2(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                       int had_block_w, int bits, const float* static_scale, void* z_limbs,
                                       float* scale_out, cudaStream_t st) {
    if (x == nullptr || z_limbs == nullptr || static_scale == nullptr) return HQ_ERR_INVALID_ARG;
    if (xdt != HQ_F32 && xdt != HQ_BF16) return HQ_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4 && bits != 8) return HQ_ERR_INVALID_ARG;
    if (Nb <= 0 || H <= 0 || W <= 0 || C <= 0) return HQ_ERR_SHAPE;
    const int nb = had_block_w > 1 ? had_block_w : 1;
    if (!is_pow2(nb) || W % nb != 0) return HQ_ERR_SHAPE;
    if (nb > 64) return HQ_ERR_UNSUPPORTED;                       // 64 two-wide registers per thread is the limit here
    if ((int64_t(nb) << (bits - 1)) > 32768) return HQ_ERR_OVERFLOW_RISK;     // z must fit two limbs
    if (C % 2 != 0) return HQ_ERR_UNSUPPORTED;
    const int elt = xdt == HQ_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(x) % (2 * elt) != 0 || reinterpret_cast<uintptr_t>(z_limbs) % 2 != 0) return HQ_ERR_ALIGNMENT;

    Width2Params p{};
    p.x = x; p.C = C; p.c2 = int(C / 2); p.wblocks = int(W / nb); p.bits = bits;
    p.items = Nb * H * (W / nb) * (C / 2);
    p.norm = float(exp2(-0.5 * double(ilog2(nb))));
    p.static_scale = static_scale; p.z = static_cast<int8_t*>(z_limbs); p.scale_out = scale_out;
    const int threads = 128;
    const int64_t grid64 = (p.items + threads - 1) / threads;
    if (grid64 > 0x7FFFFFFF) return HQ_ERR_UNSUPPORTED;
    const int grid = int(grid64);
#define HQ_WIDTH2_CASE(NBV)                                                                             \
    case NBV:                                                                                           \
        if (xdt == HQ_F32) width_quant2_kernel<NBV, float><<<grid, threads, 0, st>>>(p);                \
        else width_quant2_kernel<NBV, __nv_bfloat16><<<grid, threads, 0, st>>>(p);                      \
        break;
    switch (nb) {
        HQ_WIDTH2_CASE(2) HQ_WIDTH2_CASE(4) HQ_WIDTH2_CASE(8) HQ_WIDTH2_CASE(16) HQ_WIDTH2_CASE(32) HQ_WIDTH2_CASE(64)
        default: return HQ_ERR_UNSUPPORTED;
    }
#undef HQ_WIDTH2_CASE
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

}  // namespace hq

extern "C" hq_status hq_ln_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, const float* weight,
                                 const float* bias, int64_t rows_per_group, float eps, int had_block, int bits,
                                 hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont,
                                 int64_t ld_codes, float* scales, void* stream) {
    return hq::launch_ln_quant(x, xdt, rows, cols, ldx, weight, bias, rows_per_group, eps, had_block, bits, mode,
                               static_scale, codes, cont, ld_codes, scales, static_cast<cudaStream_t>(stream));
}

extern "C" hq_status hq_gn_silu_quant(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                      int groups, const float* gamma, const float* beta, const void* pre_bias, float eps,
                                      int had_block, int bits, hq_scale_mode mode, const float* static_scale, void* codes,
                                      hq_container cont, int64_t ld_codes, float* scales, void* scratch,
                                      size_t scratch_bytes, void* stream) {
    return hq::launch_gn_silu_quant(x, xdt, Nb, H, W, C, groups, gamma, beta, eps, had_block, bits, mode, static_scale, codes,
                                    cont, ld_codes, scales, scratch, scratch_bytes, static_cast<cudaStream_t>(stream), 1,
                                    pre_bias, nullptr, 0);
}

extern "C" hq_status hq_gn_silu_quant_cat(const void* x, const void* x2, int64_t C1, hq_dtype xdt, int64_t Nb, int64_t H,
                                          int64_t W, int64_t C, int groups, const float* gamma, const float* beta,
                                          const void* pre_bias, float eps, int had_block, int bits, hq_scale_mode mode,
                                          const float* static_scale, void* codes, hq_container cont, int64_t ld_codes,
                                          float* scales, void* scratch, size_t scratch_bytes, void* stream) {
    if (x2 == nullptr) return HQ_ERR_INVALID_ARG;
    return hq::launch_gn_silu_quant(x, xdt, Nb, H, W, C, groups, gamma, beta, eps, had_block, bits, mode, static_scale, codes,
                                    cont, ld_codes, scales, scratch, scratch_bytes, static_cast<cudaStream_t>(stream), 1,
                                    pre_bias, x2, C1);
}

extern "C" hq_status hq_hadamard_quant_cat(const void* x, int64_t ldx, const void* x2, int64_t ldx2, int64_t cols1,
                                           hq_dtype xdt, int64_t rows, int64_t cols, int had_block, int bits,
                                           hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont,
                                           int64_t ld_codes, float* scales, void* stream) {
    return hq::launch_hadamard_quant_cat(x, ldx, x2, ldx2, cols1, xdt, rows, cols, had_block, bits, mode, static_scale, codes,
                                         cont, ld_codes, scales, static_cast<cudaStream_t>(stream));
}

extern "C" hq_status hq_hadamard_quant_width(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                             int had_block_w, int bits, const float* static_scale, void* z_codes,
                                             float* scale_out, void* stream) {
    return hq::launch_hadamard_quant_width(x, xdt, Nb, H, W, C, had_block_w, bits, static_scale, z_codes, scale_out,
                                           static_cast<cudaStream_t>(stream));
}

extern "C" hq_status hq_hadamard_quant_width2(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                              int had_block_w, int bits, const float* static_scale, void* z_limbs,
                                              float* scale_out, void* stream) {
    return hq::launch_hadamard_quant_width2(x, xdt, Nb, H, W, C, had_block_w, bits, static_scale, z_limbs, scale_out,
                                            static_cast<cudaStream_t>(stream));
}

extern "C" hq_status hq_hadamard_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx,
                                       int had_block, int bits, hq_scale_mode mode, const float* static_scale,
                                       void* codes, hq_container cont, int64_t ld_codes, float* scales,
                                       void* stream) {
    return hq::launch_hadamard_quant(x, xdt, rows, cols, ldx, had_block, bits, mode, static_scale, codes, cont,
                                     ld_codes, scales, static_cast<cudaStream_t>(stream));
}
