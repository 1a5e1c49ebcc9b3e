// The unquantized operations that sit between the quantized layers of the noise-prediction network (the method replaces
// every linear and convolution; this is what is left): SiLU, residual and broadcast additions, the sinusoidal step
// embedding with the class-embedding lookup, nearest-neighbour up-sampling, channel concatenation, GroupNorm with an
// optional SiLU as a stand-alone pass, and the network's first and last convolution, which stay in floating point.
// All activations are bf16, row-major with the channel axis contiguous (NHWC); arithmetic is fp32.
// Every kernel is HBM-bound element-wise work: 16-byte loads and stores, one element group per thread.
#include "hq_common.cuh"
#include "hq_fwht.cuh"

namespace hq {

// GroupNorm statistics of an NHWC tensor into `scratch` (defined in hq_quant.cu): [samples][groups][2] fp64 sums,
// followed by [samples][groups][2] floats (mean, 1/sqrt(var + eps)).
hq_status launch_gn_stats(const void* x, hq_dtype xdt, int64_t Nb, int64_t hw, int64_t C, int groups, float eps,
                          void* scratch, size_t scratch_bytes, const float** stats_out, cudaStream_t st,
                          const void* pre_bias, const void* x2, int64_t split);

namespace {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
// y * sigmoid(y) with one special-function instruction each for the exponential and the reciprocal (every caller rounds
// the result to bf16)
__device__ __forceinline__ float silu_f(float y) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(y * -1.4426950408889634f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
    return y * r;
}

struct F8 { float v[8]; };
__device__ __forceinline__ F8 unpack8(const uint4 w) {
    F8 r;
    r.v[0] = bf16_lo(w.x); r.v[1] = bf16_hi(w.x); r.v[2] = bf16_lo(w.y); r.v[3] = bf16_hi(w.y);
    r.v[4] = bf16_lo(w.z); r.v[5] = bf16_hi(w.z); r.v[6] = bf16_lo(w.w); r.v[7] = bf16_hi(w.w);
    return r;
}
__device__ __forceinline__ uint4 pack8(const F8& f) {
    return make_uint4(pack2(f.v[0], f.v[1]), pack2(f.v[2], f.v[3]), pack2(f.v[4], f.v[5]), pack2(f.v[6], f.v[7]));
}

// out = silu(x), n8 groups of 8 values
__global__ void __launch_bounds__(256) silu_kernel(const uint4* x, uint4* out, int64_t n8) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    F8 f = unpack8(__ldg(x + i));
#pragma unroll
    for (int e = 0; e < 8; ++e) f.v[e] = silu_f(f.v[e]);
    out[i] = pack8(f);
}

// out = a + b
__global__ void __launch_bounds__(256) add_kernel(const uint4* a, const uint4* b, uint4* out, int64_t n8) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    F8 fa = unpack8(__ldcs(a + i));
    const F8 fb = unpack8(__ldcs(b + i));
#pragma unroll
    for (int e = 0; e < 8; ++e) fa.v[e] += fb.v[e];
    out[i] = pack8(fa);
}

// h[n][r][c] += e[n][c]   (c8 = C / 8 vectors per row)
__global__ void __launch_bounds__(256) add_rows_bcast_kernel(uint4* h, const uint4* e, int64_t n8, int c8,
                                                             int64_t vec_per_sample) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const int64_t n = i / vec_per_sample;
    const int c = int(i % c8);
    F8 fh = unpack8(h[i]);
    const F8 fe = unpack8(__ldg(e + n * c8 + c));
#pragma unroll
    for (int k = 0; k < 8; ++k) fh.v[k] += fe.v[k];
    h[i] = pack8(fh);
}

// emb[n][:] += table[labels[n]][:]
__global__ void __launch_bounds__(256) class_embed_add_kernel(__nv_bfloat16* emb, const __nv_bfloat16* table,
                                                              const int32_t* labels, int Nb, int dim, int classes) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Nb * dim) return;
    const int n = i / dim, d = i - n * dim;
    int lab = labels[n];
    lab = lab < 0 ? 0 : (lab >= classes ? classes - 1 : lab);
    emb[i] = __float2bfloat16_rn(__bfloat162float(emb[i]) + __bfloat162float(table[int64_t(lab) * dim + d]));
}

// out[n][i] = cos(t[n] f_i), out[n][half + i] = sin(t[n] f_i), f_i = exp(-ln(max_period) i / half)
__global__ void __launch_bounds__(256) timestep_embedding_kernel(const float* t, int Nb, int dim, float max_period,
                                                                 __nv_bfloat16* out) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int half = dim / 2;
    if (idx >= Nb * half) return;
    const int n = idx / half, i = idx - n * half;
    const float f = expf(-logf(max_period) * float(i) / float(half));
    const float a = t[n] * f;
    out[int64_t(n) * dim + i] = __float2bfloat16_rn(cosf(a));
    out[int64_t(n) * dim + half + i] = __float2bfloat16_rn(sinf(a));
}

// out[n][2h+i][2w+j][:] = x[n][h][w][:]; one thread per input vector, four stores
__global__ void __launch_bounds__(256) upsample2x_kernel(const uint4* x, uint4* out, int64_t n8, int c8, int W, int H) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const int c = int(i % c8);
    const int64_t pix = i / c8;
    const int w = int(pix % W);
    const int64_t nh = pix / W;                       // n * H + h
    const uint4 v = __ldcs(x + i);
    const int64_t o = ((2 * nh) * (2 * int64_t(W)) + 2 * w) * c8 + c;     // (n, 2h, 2w)
    out[o] = v;
    out[o + c8] = v;
    out[o + 2 * int64_t(W) * c8] = v;
    out[o + 2 * int64_t(W) * c8 + c8] = v;
}

// out[r][0..Ca) = a[r][:], out[r][Ca..Ca+Cb) = b[r][:]
__global__ void __launch_bounds__(256) concat_kernel(const uint4* a, int ca8, const uint4* b, int cb8, uint4* out,
                                                     int64_t n8) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const int c8 = ca8 + cb8;
    const int64_t r = i / c8;
    const int c = int(i - r * c8);
    out[i] = c < ca8 ? __ldcs(a + r * ca8 + c) : __ldcs(b + r * cb8 + (c - ca8));
}

// y = act((x - mean) rstd gamma + beta) with the statistics of the element's (sample, group).  A thread keeps one channel
// vector (8 channels) and walks pixels, so gamma / beta / the group's statistics are read once per thread and sample.
__global__ void __launch_bounds__(256) gn_apply_kernel(const uint4* x, uint4* out, int c8, int64_t pixels_per_sample,
                                                       int pixel_chunks, const float* stats, const float* gamma,
                                                       const float* beta, int groups, int cg, int act) {
    const int n = blockIdx.y;
    const int lanes_c = c8 < 256 ? c8 : 256;           // channel vectors walked side by side
    const int ppl = 256 / lanes_c;                      // pixels walked side by side
    const int cv0 = threadIdx.x % lanes_c, pl = threadIdx.x / lanes_c;
    if (pl >= ppl) return;
    const int64_t per = (pixels_per_sample + pixel_chunks - 1) / pixel_chunks;
    const int64_t p0 = int64_t(blockIdx.x) * per, p1 = p0 + per < pixels_per_sample ? p0 + per : pixels_per_sample;
    for (int cv = cv0; cv < c8; cv += lanes_c) {
        float a[8], b[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int c = cv * 8 + e;
            const float2 st = *reinterpret_cast<const float2*>(stats + (int64_t(n) * groups + c / cg) * 2);
            a[e] = st.y * __ldg(gamma + c);
            b[e] = fmaf(-st.x, a[e], __ldg(beta + c));
        }
        const uint4* src = x + int64_t(n) * pixels_per_sample * c8 + cv;
        uint4* dst = out + int64_t(n) * pixels_per_sample * c8 + cv;
        for (int64_t px = p0 + pl; px < p1; px += ppl) {
            F8 f = unpack8(__ldcs(src + px * c8));
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float y = fmaf(f.v[e], a[e], b[e]);
                f.v[e] = act ? silu_f(y) : y;
            }
            dst[px * c8] = pack8(f);
        }
    }
}

// Convolution with few input channels (the network's first convolution): a warp takes four consecutive output pixels of
// a row, each lane eight consecutive output channels per round; the weights sit in shared memory as [tap * C + c][Cout] and
// every weight read serves the four pixels.
template <typename InT>
__global__ void __launch_bounds__(256) conv_small_cin_kernel(const InT* x, const float* w, const float* bias,
                                                             __nv_bfloat16* out, int Nb, int H, int W, int C, int Cout,
                                                             int R, int stride, int pad, int Ho, int Wo) {
    extern __shared__ float sw[];                      // [R*R*C][Cout]
    const int taps = R * R * C;
    for (int i = threadIdx.x; i < taps * Cout; i += blockDim.x) {
        const int co = i / taps, k = i - co * taps;   // global layout [Cout][R][R][C]
        sw[k * Cout + co] = w[i];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int wq = (Wo + 3) / 4;                       // groups of four pixels per output row
    const int64_t groups = int64_t(Nb) * Ho * wq;
    for (int64_t g = int64_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); g < groups;
         g += int64_t(gridDim.x) * (blockDim.x >> 5)) {
        const int wo0 = int(g % wq) * 4;
        const int ho = int((g / wq) % Ho);
        const int n = int(g / (int64_t(wq) * Ho));
        for (int co0 = lane * 8; co0 < Cout; co0 += 256) {
            float acc[4][8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float b = bias != nullptr ? __ldg(bias + co0 + e) : 0.f;
#pragma unroll
                for (int pp = 0; pp < 4; ++pp) acc[pp][e] = b;
            }
            for (int r = 0; r < R; ++r) {
                const int hi = ho * stride + r - pad;
                if (hi < 0 || hi >= H) continue;
                for (int sx = 0; sx < R; ++sx) {
                    for (int c = 0; c < C; ++c) {
                        float xv[4];
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp) {
                            const int wi = (wo0 + pp) * stride + sx - pad;
                            xv[pp] = 0.f;
                            if (wi >= 0 && wi < W && wo0 + pp < Wo) {
                                const InT* px = x + ((int64_t(n) * H + hi) * W + wi) * C + c;
                                if (sizeof(InT) == 4) xv[pp] = __ldg(reinterpret_cast<const float*>(px));
                                else xv[pp] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(px));
                            }
                        }
                        const float4* wr = reinterpret_cast<const float4*>(sw + ((r * R + sx) * C + c) * Cout + co0);
                        const float4 w0 = wr[0], w1 = wr[1];
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp) {
                            acc[pp][0] = fmaf(xv[pp], w0.x, acc[pp][0]); acc[pp][1] = fmaf(xv[pp], w0.y, acc[pp][1]);
                            acc[pp][2] = fmaf(xv[pp], w0.z, acc[pp][2]); acc[pp][3] = fmaf(xv[pp], w0.w, acc[pp][3]);
                            acc[pp][4] = fmaf(xv[pp], w1.x, acc[pp][4]); acc[pp][5] = fmaf(xv[pp], w1.y, acc[pp][5]);
                            acc[pp][6] = fmaf(xv[pp], w1.z, acc[pp][6]); acc[pp][7] = fmaf(xv[pp], w1.w, acc[pp][7]);
                        }
                    }
                }
            }
#pragma unroll
            for (int pp = 0; pp < 4; ++pp) {
                if (wo0 + pp >= Wo) continue;
                F8 f;
#pragma unroll
                for (int e = 0; e < 8; ++e) f.v[e] = acc[pp][e];
                *reinterpret_cast<uint4*>(out + ((int64_t(n) * Ho + ho) * Wo + wo0 + pp) * Cout + co0) = pack8(f);
            }
        }
    }
}

// Convolution with few output channels (the network's last convolution): a warp takes four consecutive output pixels of a
// row, each lane eight input channels per round of 256 for every filter tap (coalesced 512-byte reads); the weights
// [Cout][R][R][C] sit in shared memory as they are and every weight read serves the four pixels; the partial sums of the
// warp are added up by shuffles.  Output fp32.
template <int COUT>
__global__ void __launch_bounds__(256) conv_small_cout_kernel(const __nv_bfloat16* x, const float* w, const float* bias,
                                                              float* out, int Nb, int H, int W, int C, int R, int stride,
                                                              int pad, int Ho, int Wo) {
    extern __shared__ float sw[];                      // [COUT][R*R][C]
    const int wsize = COUT * R * R * C;
    for (int i = threadIdx.x; i < wsize; i += blockDim.x) sw[i] = w[i];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int wq = (Wo + 3) / 4;
    const int64_t groups = int64_t(Nb) * Ho * wq;
    for (int64_t g = int64_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); g < groups;
         g += int64_t(gridDim.x) * (blockDim.x >> 5)) {
        const int wo0 = int(g % wq) * 4;
        const int ho = int((g / wq) % Ho);
        const int n = int(g / (int64_t(wq) * Ho));
        float acc[4][COUT];
#pragma unroll
        for (int pp = 0; pp < 4; ++pp)
#pragma unroll
            for (int o = 0; o < COUT; ++o) acc[pp][o] = 0.f;
        for (int r = 0; r < R; ++r) {
            const int hi = ho * stride + r - pad;
            if (hi < 0 || hi >= H) continue;
            for (int sx = 0; sx < R; ++sx) {
                for (int c0 = lane * 8; c0 < C; c0 += 256) {
                    F8 f[4];
#pragma unroll
                    for (int pp = 0; pp < 4; ++pp) {
                        const int wi = (wo0 + pp) * stride + sx - pad;
                        uint4 raw = make_uint4(0u, 0u, 0u, 0u);
                        if (wi >= 0 && wi < W && wo0 + pp < Wo)
                            raw = __ldg(reinterpret_cast<const uint4*>(x + ((int64_t(n) * H + hi) * W + wi) * C + c0));
                        f[pp] = unpack8(raw);
                    }
#pragma unroll
                    for (int o = 0; o < COUT; ++o) {
                        const float4* wr = reinterpret_cast<const float4*>(sw + (o * R * R + r * R + sx) * C + c0);
                        const float4 w0 = wr[0], w1 = wr[1];
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp) {
                            acc[pp][o] = fmaf(f[pp].v[0], w0.x, fmaf(f[pp].v[1], w0.y, fmaf(f[pp].v[2], w0.z, fmaf(f[pp].v[3], w0.w, acc[pp][o]))));
                            acc[pp][o] = fmaf(f[pp].v[4], w1.x, fmaf(f[pp].v[5], w1.y, fmaf(f[pp].v[6], w1.z, fmaf(f[pp].v[7], w1.w, acc[pp][o]))));
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int pp = 0; pp < 4; ++pp)
#pragma unroll
            for (int o = 0; o < COUT; ++o) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc[pp][o] += __shfl_xor_sync(0xffffffffu, acc[pp][o], off);
            }
        // lane pp * COUT + o writes output o of pixel pp
#pragma unroll
        for (int pp = 0; pp < 4; ++pp)
#pragma unroll
            for (int o = 0; o < COUT; ++o)
                if (lane == pp * COUT + o && wo0 + pp < Wo)
                    out[((int64_t(n) * Ho + ho) * Wo + wo0 + pp) * COUT + o] = acc[pp][o] + (bias != nullptr ? __ldg(bias + o) : 0.f);
    }
}

// The 3x3, stride 1, pad 1 shapes of the network's first and last convolution.  What bounds them is the shared-memory
// traffic of the weights (a warp-wide 16-byte read costs four wavefronts), so a warp of the first convolution takes EIGHT consecutive output
// pixels of a row per weight read (the last one four), the input columns they touch in one filter row are fetched once per row (not once per
// tap), the weights are laid out so that the 32 lanes of a 16-byte read touch consecutive addresses (a lane's eight
// channels as two quads half a round apart: no bank conflicts), and the multiply-adds run two wide (`fma.f32x2`: an
// input value is paired with itself or, for the last convolution, with its channel neighbour).
constexpr int kConvPx = 8;      // first convolution (few registers per pixel)
constexpr int kConvPxOut = 4;   // last convolution (ten input-column pieces of eight channels per row are already 40 registers)

// Position of channel ch (of a round of up to 256 channels, eight per lane) in the conflict-free order.
__device__ __forceinline__ int conv_slot(int ch, int half_stride) {
    const int rnd = ch >> 8, cl = ch & 255;
    return rnd * 256 + ((cl >> 2) & 1) * half_stride + (cl >> 3) * 4 + (cl & 3);
}

template <typename InT, int CIN>
__global__ void __launch_bounds__(256) conv3x3_small_cin_kernel(const InT* x, const float* w, const float* bias,
                                                                __nv_bfloat16* out, int Nb, int H, int W, int Cout) {
    extern __shared__ float sw[];                      // [9 * CIN][Cout], channels in conflict-free order
    constexpr int taps = 9 * CIN;
    const int hs = (Cout < 256 ? Cout : 256) / 2;
    for (int i = threadIdx.x; i < taps * Cout; i += blockDim.x) {
        const int co = i / taps, k = i - co * taps;   // global layout [Cout][3][3][CIN]
        sw[k * Cout + conv_slot(co, hs)] = w[i];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int wq = (W + kConvPx - 1) / kConvPx;        // groups of eight pixels per output row
    const int64_t groups = int64_t(Nb) * H * wq;
    for (int64_t g = int64_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); g < groups;
         g += int64_t(gridDim.x) * (blockDim.x >> 5)) {
        const int wo0 = int(g % wq) * kConvPx;
        const int ho = int((g / wq) % H);
        const int n = int(g / (int64_t(wq) * H));
        for (int co0 = lane * 8; co0 < Cout; co0 += 256) {
            f32x2 acc[kConvPx][4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float b0 = bias != nullptr ? __ldg(bias + co0 + 2 * j) : 0.f;
                const float b1 = bias != nullptr ? __ldg(bias + co0 + 2 * j + 1) : 0.f;
#pragma unroll
                for (int pp = 0; pp < kConvPx; ++pp) acc[pp][j] = pk2(b0, b1);
            }
            const float* wbase = sw + (co0 & ~255) + lane * 4;
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const int hi = ho + r - 1;
                if (hi < 0 || hi >= H) continue;
                float xin[kConvPx + 2][CIN];
                const InT* row = x + (int64_t(n) * H + hi) * W * CIN;
#pragma unroll
                for (int j = 0; j < kConvPx + 2; ++j) {
                    const int wi = wo0 - 1 + j;
                    const bool in = wi >= 0 && wi < W;
#pragma unroll
                    for (int c = 0; c < CIN; ++c) {
                        float v = 0.f;
                        if (in) {
                            if (sizeof(InT) == 4) v = __ldg(reinterpret_cast<const float*>(row + wi * CIN + c));
                            else v = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(row + wi * CIN + c));
                        }
                        xin[j][c] = v;
                    }
                }
#pragma unroll
                for (int sx = 0; sx < 3; ++sx) {
#pragma unroll
                    for (int c = 0; c < CIN; ++c) {
                        const float* wr = wbase + ((r * 3 + sx) * CIN + c) * Cout;
                        const ulonglong2 w0 = *reinterpret_cast<const ulonglong2*>(wr);
                        const ulonglong2 w1 = *reinterpret_cast<const ulonglong2*>(wr + hs);
#pragma unroll
                        for (int pp = 0; pp < kConvPx; ++pp) {
                            const f32x2 xv = pk2(xin[pp + sx][c], xin[pp + sx][c]);
                            acc[pp][0] = fma2(w0.x, xv, acc[pp][0]);
                            acc[pp][1] = fma2(w0.y, xv, acc[pp][1]);
                            acc[pp][2] = fma2(w1.x, xv, acc[pp][2]);
                            acc[pp][3] = fma2(w1.y, xv, acc[pp][3]);
                        }
                    }
                }
            }
#pragma unroll
            for (int pp = 0; pp < kConvPx; ++pp) {
                if (wo0 + pp >= W) continue;
                F8 f;
#pragma unroll
                for (int j = 0; j < 4; ++j) upk2(acc[pp][j], f.v[2 * j], f.v[2 * j + 1]);
                *reinterpret_cast<uint4*>(out + ((int64_t(n) * H + ho) * W + wo0 + pp) * Cout + co0) = pack8(f);
            }
        }
    }
}

template <int COUT>
__global__ void __launch_bounds__(256) conv3x3_small_cout_kernel(const __nv_bfloat16* x, const float* w, const float* bias,
                                                                 float* out, int Nb, int H, int W, int C) {
    extern __shared__ float sw[];                      // [COUT][9][C], channels in conflict-free order
    const int wsize = COUT * 9 * C;
    const int hs = (C < 256 ? C : 256) / 2;
    for (int i = threadIdx.x; i < wsize; i += blockDim.x) {
        const int ot = i / C, c = i - ot * C;
        sw[ot * C + conv_slot(c, hs)] = w[i];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int wq = (W + kConvPxOut - 1) / kConvPxOut;
    const int64_t groups = int64_t(Nb) * H * wq;
    for (int64_t g = int64_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); g < groups;
         g += int64_t(gridDim.x) * (blockDim.x >> 5)) {
        const int wo0 = int(g % wq) * kConvPxOut;
        const int ho = int((g / wq) % H);
        const int n = int(g / (int64_t(wq) * H));
        f32x2 acc[kConvPxOut][COUT];                      // even and odd input channels side by side
#pragma unroll
        for (int pp = 0; pp < kConvPxOut; ++pp)
#pragma unroll
            for (int o = 0; o < COUT; ++o) acc[pp][o] = pk2(0.f, 0.f);
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int hi = ho + r - 1;
            if (hi < 0 || hi >= H) continue;
            const __nv_bfloat16* row = x + (int64_t(n) * H + hi) * W * C;
            for (int c0 = lane * 8; c0 < C; c0 += 256) {
                f32x2 xin[kConvPxOut + 2][4];
#pragma unroll
                for (int j = 0; j < kConvPxOut + 2; ++j) {
                    const int wi = wo0 - 1 + j;
                    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
                    if (wi >= 0 && wi < W) raw = __ldg(reinterpret_cast<const uint4*>(row + int64_t(wi) * C + c0));
                    xin[j][0] = pk2(bf16_lo(raw.x), bf16_hi(raw.x));
                    xin[j][1] = pk2(bf16_lo(raw.y), bf16_hi(raw.y));
                    xin[j][2] = pk2(bf16_lo(raw.z), bf16_hi(raw.z));
                    xin[j][3] = pk2(bf16_lo(raw.w), bf16_hi(raw.w));
                }
                const float* wbase = sw + (c0 & ~255) + lane * 4;
#pragma unroll
                for (int sx = 0; sx < 3; ++sx) {
#pragma unroll
                    for (int o = 0; o < COUT; ++o) {
                        const float* wr = wbase + (o * 9 + r * 3 + sx) * C;
                        const ulonglong2 w0 = *reinterpret_cast<const ulonglong2*>(wr);
                        const ulonglong2 w1 = *reinterpret_cast<const ulonglong2*>(wr + hs);
#pragma unroll
                        for (int pp = 0; pp < kConvPxOut; ++pp)
                            acc[pp][o] = fma2(xin[pp + sx][0], w0.x, fma2(xin[pp + sx][1], w0.y,
                                         fma2(xin[pp + sx][2], w1.x, fma2(xin[pp + sx][3], w1.y, acc[pp][o]))));
                    }
                }
            }
        }
        float red[kConvPxOut][COUT];
#pragma unroll
        for (int pp = 0; pp < kConvPxOut; ++pp)
#pragma unroll
            for (int o = 0; o < COUT; ++o) {
                float a, b;
                upk2(acc[pp][o], a, b);
                red[pp][o] = a + b;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) red[pp][o] += __shfl_xor_sync(0xffffffffu, red[pp][o], off);
            }
        // lane pp * COUT + o writes output o of pixel pp
#pragma unroll
        for (int pp = 0; pp < kConvPxOut; ++pp)
#pragma unroll
            for (int o = 0; o < COUT; ++o)
                if (lane == pp * COUT + o && wo0 + pp < W)
                    out[((int64_t(n) * H + ho) * W + wo0 + pp) * COUT + o] = red[pp][o] + (bias != nullptr ? __ldg(bias + o) : 0.f);
    }
}

inline int blocks_for(int64_t n, int threads) { return int((n + threads - 1) / threads); }

}  // namespace
}  // namespace hq

using namespace hq;

extern "C" hq_status hq_silu(const void* x, int64_t count, void* out, void* stream) {
    if (count < 0) return HQ_ERR_SHAPE;
    if (count == 0) return HQ_OK;
    if (x == nullptr || out == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(out) || count % 8 != 0) return HQ_ERR_ALIGNMENT;
    const int64_t n8 = count / 8;
    silu_kernel<<<blocks_for(n8, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(x), static_cast<uint4*>(out), n8);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_add(const void* a, const void* b, int64_t count, void* out, void* stream) {
    if (count < 0) return HQ_ERR_SHAPE;
    if (count == 0) return HQ_OK;
    if (a == nullptr || b == nullptr || out == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(b) || !aligned16(out) || count % 8 != 0) return HQ_ERR_ALIGNMENT;
    const int64_t n8 = count / 8;
    add_kernel<<<blocks_for(n8, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(a), static_cast<const uint4*>(b), static_cast<uint4*>(out), n8);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_add_rows_bcast(void* h, const void* e, int64_t Nb, int64_t rows_per_sample, int64_t C,
                                       void* stream) {
    if (Nb < 0 || rows_per_sample < 0 || C <= 0) return HQ_ERR_SHAPE;
    if (Nb == 0 || rows_per_sample == 0) return HQ_OK;
    if (h == nullptr || e == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(h) || !aligned16(e) || C % 8 != 0) return HQ_ERR_ALIGNMENT;
    const int64_t n8 = Nb * rows_per_sample * (C / 8);
    add_rows_bcast_kernel<<<blocks_for(n8, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<uint4*>(h), static_cast<const uint4*>(e), n8, int(C / 8), rows_per_sample * (C / 8));
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_class_embed_add(void* emb, const void* table, const int32_t* labels, int64_t Nb, int64_t dim,
                                        int64_t classes, void* stream) {
    if (Nb < 0 || dim <= 0 || classes <= 0 || Nb * dim > 0x7FFFFFFF) return HQ_ERR_SHAPE;
    if (Nb == 0) return HQ_OK;
    if (emb == nullptr || table == nullptr || labels == nullptr) return HQ_ERR_INVALID_ARG;
    class_embed_add_kernel<<<blocks_for(Nb * dim, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<__nv_bfloat16*>(emb), static_cast<const __nv_bfloat16*>(table), labels, int(Nb), int(dim), int(classes));
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_timestep_embedding(const float* t, int64_t Nb, int64_t dim, float max_period, void* out,
                                           void* stream) {
    if (Nb < 0 || dim <= 0 || (dim & 1) || !(max_period > 1.0f) || Nb * dim > 0x7FFFFFFF) return HQ_ERR_SHAPE;
    if (Nb == 0) return HQ_OK;
    if (t == nullptr || out == nullptr) return HQ_ERR_INVALID_ARG;
    timestep_embedding_kernel<<<blocks_for(Nb * (dim / 2), 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        t, int(Nb), int(dim), max_period, static_cast<__nv_bfloat16*>(out));
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_upsample_nearest2x(const void* x, int64_t Nb, int64_t H, int64_t W, int64_t C, void* out,
                                           void* stream) {
    if (Nb < 0 || H <= 0 || W <= 0 || C <= 0 || H > 0x3FFFFFFF || W > 0x3FFFFFFF) return HQ_ERR_SHAPE;
    if (Nb == 0) return HQ_OK;
    if (x == nullptr || out == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(out) || C % 8 != 0) return HQ_ERR_ALIGNMENT;
    const int64_t n8 = Nb * H * W * (C / 8);
    upsample2x_kernel<<<blocks_for(n8, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(x), static_cast<uint4*>(out), n8, int(C / 8), int(W), int(H));
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_concat_channels(const void* a, int64_t Ca, const void* b, int64_t Cb, int64_t rows, void* out,
                                        void* stream) {
    if (rows < 0 || Ca <= 0 || Cb <= 0) return HQ_ERR_SHAPE;
    if (rows == 0) return HQ_OK;
    if (a == nullptr || b == nullptr || out == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(b) || !aligned16(out) || Ca % 8 != 0 || Cb % 8 != 0) return HQ_ERR_ALIGNMENT;
    const int64_t n8 = rows * ((Ca + Cb) / 8);
    concat_kernel<<<blocks_for(n8, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(a), int(Ca / 8), static_cast<const uint4*>(b), int(Cb / 8), static_cast<uint4*>(out), n8);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_groupnorm_act(const void* x, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups,
                                      const float* gamma, const float* beta, float eps, int silu, void* out,
                                      void* scratch, size_t scratch_bytes, void* stream) {
    if (x == nullptr || out == nullptr || gamma == nullptr || beta == nullptr || scratch == nullptr) return HQ_ERR_INVALID_ARG;
    if (Nb <= 0 || H <= 0 || W <= 0 || C <= 0 || groups <= 0 || C % groups != 0) return HQ_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(out) || C % 8 != 0) return HQ_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float* stats = nullptr;
    hq_status s = launch_gn_stats(x, HQ_BF16, Nb, H * W, C, groups, eps, scratch, scratch_bytes, &stats, st, nullptr, nullptr, 0);
    if (s != HQ_OK) return s;
    if (Nb > 65535) return HQ_ERR_UNSUPPORTED;
    const int c8 = int(C / 8);
    const int64_t hw = H * W;
    const int64_t ppl = c8 < 256 ? 256 / c8 : 1;
    int64_t chunks = hw / (ppl * 8);                   // about 8 pixels per thread
    chunks = chunks < 1 ? 1 : (chunks > 2048 ? 2048 : chunks);
    gn_apply_kernel<<<dim3(unsigned(chunks), unsigned(Nb)), 256, 0, st>>>(static_cast<const uint4*>(x), static_cast<uint4*>(out),
                                                                         c8, hw, int(chunks), stats, gamma, beta, groups,
                                                                         int(C / groups), silu != 0);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

extern "C" hq_status hq_conv2d_direct(const void* x, hq_dtype xdt, const float* w, const float* bias, int64_t Nb,
                                      int64_t H, int64_t W, int64_t C, int64_t Cout, int R, int stride, int pad, void* y,
                                      hq_dtype ydt, void* stream) {
    if (x == nullptr || w == nullptr || y == nullptr) return HQ_ERR_INVALID_ARG;
    if ((xdt != HQ_F32 && xdt != HQ_BF16) || (ydt != HQ_F32 && ydt != HQ_BF16)) return HQ_ERR_INVALID_ARG;
    if (Nb <= 0 || H <= 0 || W <= 0 || C <= 0 || Cout <= 0) return HQ_ERR_SHAPE;
    if ((R != 1 && R != 3) || (stride != 1 && stride != 2) || pad < 0 || pad > 1) return HQ_ERR_UNSUPPORTED;
    const int64_t Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - R) / stride + 1;
    if (Ho <= 0 || Wo <= 0) return HQ_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = size_t(R) * R * C * Cout * sizeof(float);
    if (smem > 160 * 1024) return HQ_ERR_UNSUPPORTED;
    const int64_t pixel_groups = Nb * Ho * ((Wo + 3) / 4);                    // a warp takes four pixels at a time
    const int grid = int(pixel_groups / 8 < 148 * 16 ? (pixel_groups + 7) / 8 : 148 * 16);
    const bool same3x3 = R == 3 && stride == 1 && pad == 1;
    const int64_t groups8 = Nb * Ho * ((Wo + 7) / 8);                          // the first 3x3 convolution: eight pixels per warp
    const int grid8 = int(groups8 / 8 < 148 * 16 ? (groups8 + 7) / 8 : 148 * 16);
    if (ydt == HQ_BF16 && C <= 16 && Cout % 8 == 0) {                          // few input channels
        if (!aligned16(y)) return HQ_ERR_ALIGNMENT;
        if (same3x3 && (C == 3 || C == 4) && (Cout <= 256 || Cout % 256 == 0)) {
#define HQ_CIN_CASE(T, N)                                                                                           \
            HQ_CUDA_OK(cudaFuncSetAttribute(conv3x3_small_cin_kernel<T, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem))); \
            conv3x3_small_cin_kernel<T, N><<<grid8, 256, smem, st>>>(static_cast<const T*>(x), w, bias,              \
                static_cast<__nv_bfloat16*>(y), int(Nb), int(H), int(W), int(Cout));
            if (xdt == HQ_F32) { if (C == 3) { HQ_CIN_CASE(float, 3) } else { HQ_CIN_CASE(float, 4) } }
            else { if (C == 3) { HQ_CIN_CASE(__nv_bfloat16, 3) } else { HQ_CIN_CASE(__nv_bfloat16, 4) } }
#undef HQ_CIN_CASE
            return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
        }
        if (xdt == HQ_F32) {
            HQ_CUDA_OK(cudaFuncSetAttribute(conv_small_cin_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
            conv_small_cin_kernel<float><<<grid, 256, smem, st>>>(static_cast<const float*>(x), w, bias,
                static_cast<__nv_bfloat16*>(y), int(Nb), int(H), int(W), int(C), int(Cout), R, stride, pad, int(Ho), int(Wo));
        } else {
            HQ_CUDA_OK(cudaFuncSetAttribute(conv_small_cin_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
            conv_small_cin_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(x), w, bias,
                static_cast<__nv_bfloat16*>(y), int(Nb), int(H), int(W), int(C), int(Cout), R, stride, pad, int(Ho), int(Wo));
        }
        return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
    }
    if (ydt == HQ_F32 && xdt == HQ_BF16 && Cout <= 4 && C % 8 == 0) {          // few output channels
        if (!aligned16(x)) return HQ_ERR_ALIGNMENT;
        if (same3x3 && (C <= 256 || C % 256 == 0)) {
#define HQ_COUT3_CASE(N)                                                                                            \
            case N:                                                                                                 \
                HQ_CUDA_OK(cudaFuncSetAttribute(conv3x3_small_cout_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem))); \
                conv3x3_small_cout_kernel<N><<<grid, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(x), w, bias, \
                    static_cast<float*>(y), int(Nb), int(H), int(W), int(C));                                       \
                break;
            switch (int(Cout)) {
                HQ_COUT3_CASE(1) HQ_COUT3_CASE(2) HQ_COUT3_CASE(3) HQ_COUT3_CASE(4)
                default: return HQ_ERR_UNSUPPORTED;
            }
#undef HQ_COUT3_CASE
            return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
        }
#define HQ_COUT_CASE(N)                                                                                             \
        case N:                                                                                                     \
            HQ_CUDA_OK(cudaFuncSetAttribute(conv_small_cout_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem))); \
            conv_small_cout_kernel<N><<<grid, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(x), w, bias,       \
                static_cast<float*>(y), int(Nb), int(H), int(W), int(C), R, stride, pad, int(Ho), int(Wo));         \
            break;
        switch (int(Cout)) {
            HQ_COUT_CASE(1) HQ_COUT_CASE(2) HQ_COUT_CASE(3) HQ_COUT_CASE(4)
            default: return HQ_ERR_UNSUPPORTED;
        }
#undef HQ_COUT_CASE
        return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
    }
    return HQ_ERR_UNSUPPORTED;
}
