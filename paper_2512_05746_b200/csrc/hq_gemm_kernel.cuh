// Device side of the integer GEMM / implicit-GEMM convolution (Eq. 12, Eq. 14): tile geometry, shared-memory layout,
// the persistent kernel and the per-instantiation launcher.  Included by the translation units that instantiate the
// kernel (one per container and problem kind, so that they compile in parallel) and by the host-side launcher.
#pragma once
#include <cuda.h>

#include "hq_common.cuh"

namespace hq {
namespace gemm {


constexpr int kBM = 128;             // rows per tile (TMEM lanes)
constexpr int kBN = 256;             // operand-B rows per tile (TMEM columns)
constexpr int kBK = 128;             // bytes of K per stage (one 128-byte swizzle row)
constexpr int kMaxStages = 6;
constexpr int kResidentKb = 4;       // largest number of K blocks a resident weight tile may have
constexpr int kABytes = kBM * kBK;           // 16 KB
constexpr int kBBytes = kBN * kBK;           // 32 KB
constexpr int kRawBytes = kBM * kBK / 2;     // 8 KB packed activation tile (lands in the upper half of its A stage)
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 8;            // two per TMEM lane quarter, each taking half of the tile's columns
constexpr int kStagingBytes = 2048;          // per epilogue warp: 32 rows x 64 bytes
constexpr int kParamBytes = kEpiWarps * 2 * (kBN / 2) * 4;   // per epilogue warp: [scale_w | bias][its columns]
constexpr int kSmemLimit = 232448;           // 227 KB
enum : int { kModeFast = 0, kModeGeneric = 1, kModePerTap = 2 };
// warps: producer, MMA issuer, 8 epilogue, then 4 unpack warps (nibble container) or a second MMA issuer (fast mode
// with one code per byte)
__host__ __device__ constexpr int cta_threads(bool nibble, bool frag) { return nibble ? 448 : (frag ? 352 : 320); }
// Whether the fragment-layout epilogue with its second MMA issuer is used (fast mode, one code per byte): for K_pad
// <= 256, and for one weight limb with resident weights (K_pad <= 512).  Measured there 10-22 % faster; with two limbs
// and K_pad >= 512 it is level, and with streamed weights 2-4 % slower on most shapes.
inline bool use_frag(bool nibble, bool fast, int limbs, int num_kb) {
    return !nibble && fast && (num_kb <= 2 || (limbs == 1 && num_kb <= kResidentKb));
}

struct GemmParams {
    int64_t M;            // GEMM rows (unused for conv)
    int N;                // output channels
    int limbs;
    int a_shift;          // 4 when activation bytes are q<<4 (nibble container), else 0
    int combine_fast;     // 256*hi + lo of the raw (shifted) accumulators fits int32
    int kb_per_tap;       // 128-byte K blocks per filter tap
    int taps;
    int tiles_m, tiles_n;
    int stages;           // ring depth
    int b_resident;       // weight tile stays in shared memory; tiles are walked n-major in contiguous ranges
    uint32_t a_box_bytes; // bytes one activation TMA box delivers
    // convolution geometry (conv != 0)
    int conv, Nb, H, W, Ho, Wo, R, S, stride, pad;
    int bw, bh, bn, tiles_w, tiles_h;
    // epilogue
    const float* scale_a; int sa_scalar;
    const float* scale_w; const float* bias; float alpha;
    int32_t* acc_out; void* y; int y_bf16; int64_t ldy;
    int y_vec_ok, acc_vec_ok;
    int per_tap;          // convolution with one activation scale per input pixel: the accumulator is drained per filter tap
    int col_pass;         // per_tap with one weight limb: which 64 of a warp's 128 columns this launch produces
    int pdl;              // launched ahead of the completion of the kernel that produces the codes and scale_a
    int frag;             // fragment-layout epilogue + second MMA issuer (see use_frag)
    int tma_store;        // bf16 output goes out through bulk tensor stores (rows of a tile are consecutive output rows)
    int32_t* dev_status;
};

struct SharedCtl {
    uint64_t full[kMaxStages];
    uint64_t full2[kMaxStages];       // the same stages when filled for the second MMA issuer (see the kernel)
    uint64_t empty[kMaxStages];
    uint64_t rawread[kMaxStages];     // all unpack threads hold their share of the packed tile in registers
    uint64_t unpacked[kMaxStages];
    uint64_t bfull[kResidentKb];
    uint64_t bfree;
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

// Shared-memory carve-up (all offsets from a 1024-byte aligned base).
struct SmemLayout { int b_off, a_off, staging_off, param_off, ctl_off, total; };
// `frag`: the fragment-layout fast epilogue (two staging buffers per warp, column parameters in registers).
__host__ __device__ inline SmemLayout smem_layout(int stages, bool resident, int num_kb, bool frag) {
    SmemLayout L;
    L.b_off = 0;
    L.a_off = (resident ? num_kb : stages) * kBBytes;
    L.staging_off = L.a_off + stages * kABytes;
    L.param_off = L.staging_off + kEpiWarps * kStagingBytes * (frag ? 2 : 1);
    L.ctl_off = L.param_off + (frag ? 0 : kParamBytes);
    L.total = L.ctl_off + int(sizeof(SharedCtl)) + 1024;      // + slack for the base alignment
    return L;
}

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SharedCtl* ctl, int32_t* dev_status,
                                              int32_t code) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000000LL) {           // each poll parks the thread for up to a millisecond
        if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
    }
    ctl->abort_flag = 1;
    if (dev_status) atomicExch(dev_status, code);
    return false;
}

struct TileCoord {
    int m_tile, n_tile;
    int n0, h0, w0;      // conv: first image / output row / output column of the tile
};

// Tiles of one CTA, walked without divisions: `count` tiles starting at (m_tile, n_tile).  With resident weights a
// CTA owns a contiguous range of the n-major tile order; otherwise tile c, c + G, c + 2G, ... of the m-major order.
struct TileCursor { int m_tile, n_tile, count, dm, dn; };
__device__ __forceinline__ TileCursor tile_begin(const GemmParams& p, bool resident) {
    const int T = p.tiles_m * p.tiles_n, G = gridDim.x, c = blockIdx.x;
    TileCursor t;
    if (resident) {
        const int first = int(int64_t(c) * T / G);
        t.count = int(int64_t(c + 1) * T / G) - first;
        t.n_tile = first / p.tiles_m; t.m_tile = first - t.n_tile * p.tiles_m;
        t.dm = t.dn = 0;
    } else {
        t.count = c < T ? (T - c + G - 1) / G : 0;
        t.m_tile = c / p.tiles_n; t.n_tile = c - t.m_tile * p.tiles_n;
        t.dm = G / p.tiles_n; t.dn = G - t.dm * p.tiles_n;
    }
    return t;
}
__device__ __forceinline__ void tile_next(const GemmParams& p, TileCursor& t, bool resident) {
    if (resident) {
        if (++t.m_tile == p.tiles_m) { t.m_tile = 0; ++t.n_tile; }
    } else {
        t.n_tile += t.dn; t.m_tile += t.dm;
        if (t.n_tile >= p.tiles_n) { t.n_tile -= p.tiles_n; ++t.m_tile; }
    }
}

template <bool CONV>
__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, const TileCursor& cur) {
    TileCoord t;
    t.m_tile = cur.m_tile; t.n_tile = cur.n_tile;
    t.n0 = t.h0 = t.w0 = 0;
    if (CONV) {
        const int tw = t.m_tile % p.tiles_w;
        const int th = (t.m_tile / p.tiles_w) % p.tiles_h;
        const int tn = t.m_tile / (p.tiles_w * p.tiles_h);
        t.w0 = tw * p.bw; t.h0 = th * p.bh; t.n0 = tn * p.bn;
    }
    return t;
}

// Output row (index into [M] / flattened NHWC pixels) of row `r` of a tile, or -1 if that row does not exist.
template <bool CONV>
__device__ __forceinline__ int out_row_of(const GemmParams& p, const TileCoord& tc, int r) {
    if (CONV) {
        const int iw = r % p.bw;
        const int ih = (r / p.bw) % p.bh;
        const int in = r / (p.bw * p.bh);
        const int n = tc.n0 + in, ho = tc.h0 + ih, wo = tc.w0 + iw;
        if (in >= p.bn || n >= p.Nb || ho >= p.Ho || wo >= p.Wo) return -1;
        return (n * p.Ho + ho) * p.Wo + wo;
    }
    const int64_t row = int64_t(tc.m_tile) * kBM + r;
    return row < p.M ? int(row) : -1;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// Staging buffer of one epilogue warp: 32 rows x 64 bytes, so that global stores are row-contiguous 16-byte
// pieces.  A lane holds one output row and hands in 16 columns at a time.  ELT = 2: float bit patterns stored as
// bf16, a staging row is 32 columns filled by two calls (`half` = 0, 1); ELT = 4: 32-bit words as they are, a
// staging row is the 16 columns of one call.  The piece index is XOR-swizzled so that both the row-per-lane
// writes and the row-contiguous reads are free of bank conflicts.
template <int ELT>
__device__ __forceinline__ void stage_put(unsigned char* stg, const uint32_t (&v)[16], int lane, int half) {
    const int wsw = (lane >> 1) & 3;
    if (ELT == 2) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(v[8 * j + 0]), __uint_as_float(v[8 * j + 1]));
            w.y = pack_bf16x2(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
            w.z = pack_bf16x2(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
            w.w = pack_bf16x2(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
            *reinterpret_cast<uint4*>(stg + lane * 64 + (((2 * half + j) ^ wsw) << 4)) = w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            *reinterpret_cast<uint4*>(stg + lane * 64 + ((j ^ wsw) << 4)) =
                make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    }
}

// Reads the staged rows back row-contiguously (4 lanes per row, 8 rows per pass) and stores them.
// rows[i] is the output row of staging row (8 i + lane / 4), or -1; col0 is the column of piece 0.
template <int ELT>
__device__ __forceinline__ void stage_flush(unsigned char* stg, int lane, void* out, int64_t ld, int N, int col0,
                                            const int (&rows)[4], bool vec_ok) {
    constexpr int EPP = 16 / ELT;                  // elements per 16-byte piece
    __syncwarp();
    const int pc = lane & 3;
    const int col = col0 + pc * EPP;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int srow = i * 8 + (lane >> 2);
        const uint4 w = *reinterpret_cast<const uint4*>(stg + srow * 64 + ((pc ^ ((srow >> 1) & 3)) << 4));
        const int grow = rows[i];
        if (grow < 0 || col >= N) continue;
        unsigned char* dst = static_cast<unsigned char*>(out) + (int64_t(grow) * ld + col) * ELT;
        if (vec_ok && col + EPP <= N) {
            *reinterpret_cast<uint4*>(dst) = w;
        } else {
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < EPP; ++e) {
                if (col + e < N) {
                    if (ELT == 2) reinterpret_cast<uint16_t*>(dst)[e] = uint16_t(ww[e >> 1] >> ((e & 1) * 16));
                    else reinterpret_cast<uint32_t*>(dst)[e] = ww[e];
                }
            }
        }
    }
    __syncwarp();
}

// A lane's 16 consecutive output values (one row) stored straight to global memory, with bounds checks.
// ELT = 2: float bit patterns stored as bf16; ELT = 4: 32-bit words as they are.
template <int ELT>
__device__ __forceinline__ void store_row16(void* out_row, const uint32_t (&v)[16], int col, int N, bool vec_ok) {
    if (ELT == 2) {
        __nv_bfloat16* d = static_cast<__nv_bfloat16*>(out_row) + col;
        if (vec_ok && col + 16 <= N) {
#pragma unroll
            for (int j = 0; j < 2; ++j)
                reinterpret_cast<uint4*>(d)[j] = make_uint4(
                    pack_bf16x2(__uint_as_float(v[8 * j + 0]), __uint_as_float(v[8 * j + 1])),
                    pack_bf16x2(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3])),
                    pack_bf16x2(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5])),
                    pack_bf16x2(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7])));
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) if (col + j < N) d[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
        }
    } else {
        uint32_t* d = static_cast<uint32_t*>(out_row) + col;
        if (vec_ok && col + 16 <= N) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                reinterpret_cast<uint4*>(d)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) if (col + j < N) d[j] = v[j];
        }
    }
}

// Epilogue of one warp for the common case: bf16 output written by bulk tensor stores, limbs recombined as
// 256*hi + lo without overflow.  Per 16 columns: two TMEM loads, one integer multiply-add, int->float, two float
// operations per value, bf16 packing and two 16-byte stores into the warp's staging buffer (32 rows x 64 bytes, laid
// out in the 64-byte swizzle of the output tensor map); every 32 columns one lane hands the buffer to the copy
// engine, which clips rows and columns beyond the output, and the warp carries on with the next columns.  Before
// the buffer is written again the lane waits until the engine has read it.
template <int LIMBS, bool EARLY = false>
__device__ __forceinline__ void epilogue_fast(uint32_t t_row, unsigned char* stg, int lane, const float* prm_sw,
                                              const float* prm_b, float sa_eff, const CUtensorMap* tmY, int col0,
                                              int row0, uint64_t* tempty_bar) {
    constexpr int NSTEPS = LIMBS == 2 ? kBN / 2 / 2 / 16 : kBN / 2 / 16;
    const uint32_t wsw = (lane >> 1) & 3;
    unsigned char* wr = stg + lane * 64;
    if constexpr (EARLY) {
        // All of this warp's accumulator columns are requested at once (128 registers) and the accumulator is handed
        // back to the MMA warp as soon as they have arrived, before any of the arithmetic and stores below.
        constexpr int NL = LIMBS == 2 ? 2 * NSTEPS : NSTEPS;
        uint32_t acc[NL][16];
#pragma unroll
        for (int st = 0; st < NSTEPS; ++st) {
            tmem_ld_32x16(t_row + uint32_t(st * 16), acc[st]);
            if (LIMBS == 2) tmem_ld_32x16(t_row + uint32_t(kBN / 2 + st * 16), acc[NSTEPS + st]);
        }
#pragma unroll
        for (int l = 0; l < NL; ++l) tmem_ld_wait_16(acc[l]);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar);
#pragma unroll
        for (int st = 0; st < NSTEPS; ++st) {
            int32_t w[16];
#pragma unroll
            for (int j = 0; j < 16; ++j)
                w[j] = LIMBS == 2 ? int32_t(acc[st][j]) * 256 + int32_t(acc[NSTEPS + st][j]) : int32_t(acc[st][j]);
            if ((st & 1) == 0) {                           // the copy engine must be done reading the staging buffer
                if (lane == 0) bulk_wait_read_all();
                __syncwarp();
            }
            const float4* sw4 = reinterpret_cast<const float4*>(prm_sw + st * 16);
            const float4* b4 = reinterpret_cast<const float4*>(prm_b + st * 16);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float4 s0 = sw4[2 * j], s1 = sw4[2 * j + 1], c0 = b4[2 * j], c1 = b4[2 * j + 1];
                uint4 o;
                o.x = pack_bf16x2(fmaf(float(w[8 * j + 0]) * s0.x, sa_eff, c0.x), fmaf(float(w[8 * j + 1]) * s0.y, sa_eff, c0.y));
                o.y = pack_bf16x2(fmaf(float(w[8 * j + 2]) * s0.z, sa_eff, c0.z), fmaf(float(w[8 * j + 3]) * s0.w, sa_eff, c0.w));
                o.z = pack_bf16x2(fmaf(float(w[8 * j + 4]) * s1.x, sa_eff, c1.x), fmaf(float(w[8 * j + 5]) * s1.y, sa_eff, c1.y));
                o.w = pack_bf16x2(fmaf(float(w[8 * j + 6]) * s1.z, sa_eff, c1.z), fmaf(float(w[8 * j + 7]) * s1.w, sa_eff, c1.w));
                *reinterpret_cast<uint4*>(wr + (((2 * (st & 1) + j) ^ wsw) << 4)) = o;
            }
            if (st & 1) {
                fence_proxy_async_smem();                  // the lanes' writes become visible to the copy engine
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(tmY, stg, col0 + (st >> 1) * 32, row0);
                    bulk_commit_group();
                }
            }
        }
        return;
    }
    uint32_t hi[16], lo[16];
    tmem_ld_32x16(t_row, hi);
    if (LIMBS == 2) tmem_ld_32x16(t_row + uint32_t(kBN / 2), lo);
#pragma unroll
    for (int st = 0; st < NSTEPS; ++st) {
        int32_t w[16];
        tmem_ld_wait_16(hi);
        if (LIMBS == 2) {
            tmem_ld_wait_16(lo);
#pragma unroll
            for (int j = 0; j < 16; ++j) w[j] = int32_t(hi[j]) * 256 + int32_t(lo[j]);
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) w[j] = int32_t(hi[j]);
        }
        if (st + 1 < NSTEPS) {
            tmem_ld_32x16(t_row + uint32_t((st + 1) * 16), hi);
            if (LIMBS == 2) tmem_ld_32x16(t_row + uint32_t(kBN / 2 + (st + 1) * 16), lo);
        } else {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);
        }
        if ((st & 1) == 0) {                           // the copy engine must be done reading the staging buffer
            if (lane == 0) bulk_wait_read_all();
            __syncwarp();
        }
        const float4* sw4 = reinterpret_cast<const float4*>(prm_sw + st * 16);
        const float4* b4 = reinterpret_cast<const float4*>(prm_b + st * 16);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float4 s0 = sw4[2 * j], s1 = sw4[2 * j + 1], c0 = b4[2 * j], c1 = b4[2 * j + 1];
            uint4 o;
            o.x = pack_bf16x2(fmaf(float(w[8 * j + 0]) * s0.x, sa_eff, c0.x), fmaf(float(w[8 * j + 1]) * s0.y, sa_eff, c0.y));
            o.y = pack_bf16x2(fmaf(float(w[8 * j + 2]) * s0.z, sa_eff, c0.z), fmaf(float(w[8 * j + 3]) * s0.w, sa_eff, c0.w));
            o.z = pack_bf16x2(fmaf(float(w[8 * j + 4]) * s1.x, sa_eff, c1.x), fmaf(float(w[8 * j + 5]) * s1.y, sa_eff, c1.y));
            o.w = pack_bf16x2(fmaf(float(w[8 * j + 6]) * s1.z, sa_eff, c1.z), fmaf(float(w[8 * j + 7]) * s1.w, sa_eff, c1.w));
            *reinterpret_cast<uint4*>(wr + (((2 * (st & 1) + j) ^ wsw) << 4)) = o;
        }
        if (st & 1) {
            fence_proxy_async_smem();                  // the lanes' writes become visible to the copy engine
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(tmY, stg, col0 + (st >> 1) * 32, row0);
                bulk_commit_group();
            }
        }
    }
}

// Epilogue warp of the fast output mode with accumulators read in the 16x256b fragment layout: a lane holds, for its
// four rows (lane/4 + 8 j of the warp's 32), the column pairs 8 n + 2 (lane%4) + {0, 1}.  So the scale_w / bias of a
// lane's columns are 1/4 of the warp's and stay in registers while the weight tile stays (no shared-memory reads at
// all), and a bf16 pair goes to the staging buffer as one 32-bit store that is free of bank conflicts in the 64-byte
// swizzle of the output tensor map.  The shared-memory data pipe, which also feeds the tensor core its operands, is
// the busiest unit of this kernel: with row-per-lane loads the broadcast reads of the column parameters and the 16-byte
// staging stores took more of it than the MMAs themselves.
// Per 32 columns: four TMEM loads (two 16-lane slabs x two limbs), recombination, rescale, 16 stores, one bulk store.
template <bool CONV, int LIMBS>
__device__ __forceinline__ void fast_epilogue_warp(const GemmParams& p, const TileCursor& walk, bool resident,
                                                   SharedCtl* ctl, uint32_t tmem_base, unsigned char* stg,
                                                   const CUtensorMap* tmY, int warp, int lane) {
    constexpr int CPT = LIMBS == 2 ? kBN / 2 : kBN;      // output columns per tile
    constexpr int CPW = CPT / 2;                         // ... per warp
    constexpr int NCH = CPW / 32;                        // 32-column chunks: one staging buffer and one bulk store each
    const int q = warp & 3;                              // TMEM lane quarter this warp may read
    const int wc0 = ((warp - 2) >> 2) * CPW;             // first column (in the tile) of this warp
    const int tq = lane & 3, tr = lane >> 2;
    const uint32_t rsw = uint32_t(tr >> 1) & 3u;         // swizzle term of this lane's staging rows (same for all four)
    const int64_t total_rows = CONV ? int64_t(p.Nb) * p.Ho * p.Wo : p.M;
    const float a_eff = p.alpha / float(1 << p.a_shift); // the accumulators carry the container's shift
    float sw[CPW / 4], bb[CPW / 4];
    float sa[4] = {0.f, 0.f, 0.f, 0.f};
    griddep_wait();                                      // scale_a comes from the kernel before this one
    TileCursor cur = walk;
    int last_n = -1;
    for (int i = 0; i < walk.count; ++i, tile_next(p, cur, resident)) {
        const int as = i & 1;
        const TileCoord tc = tile_coord<CONV>(p, cur);
        const int col_base = tc.n_tile * CPT + wc0;
        if (tc.n_tile != last_n) {                       // consecutive tiles under resident weights share their columns
            last_n = tc.n_tile;
#pragma unroll
            for (int c = 0; c < CPW / 4; ++c) {
                const int col = col_base + 8 * (c >> 1) + 2 * tq + (c & 1);
                sw[c] = col < p.N ? __ldg(p.scale_w + col) : 0.f;
                bb[c] = (p.bias != nullptr && col < p.N) ? __ldg(p.bias + col) : 0.f;
            }
        }
        // rows of the tile are consecutive output rows (checked on the host); this warp owns 32 of them
        const int row0 = out_row_of<CONV>(p, tc, 0) + q * 32;
        if (i == 0) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t row = int64_t(row0) + tr + 8 * j;
                sa[j] = p.sa_scalar ? __ldg(p.scale_a) : (row < total_rows ? __ldg(p.scale_a + row) : 0.f);
            }
        }
        int row0_next = -1;
        if (i + 1 < walk.count && !p.sa_scalar) {
            TileCursor nx = cur;
            tile_next(p, nx, resident);
            row0_next = out_row_of<CONV>(p, tile_coord<CONV>(p, nx), 0) + q * 32;
        }
        if (!wait_or_abort(&ctl->tfull[as], uint32_t(i >> 1) & 1u, ctl, p.dev_status, kStatusAccumWait)) break;
        tc_fence_after();
        float sa_eff[4], sa_nx[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            sa_eff[j] = a_eff * sa[j];
            sa_nx[j] = sa[j];
            if (row0_next >= 0) {                        // the next tile's row scales fly while this tile is processed
                const int64_t row = int64_t(row0_next) + tr + 8 * j;
                sa_nx[j] = row < total_rows ? __ldg(p.scale_a + row) : 0.f;
            }
        }
        const uint32_t t0 = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN + wc0);
        const uint32_t t1 = t0 + (16u << 16);            // the second 16-lane slab
        uint32_t h0[16], h1[16], l0[16], l1[16];
        tmem_ld_16x256_x4(t0, h0);
        tmem_ld_16x256_x4(t1, h1);
        if (LIMBS == 2) { tmem_ld_16x256_x4(t0 + uint32_t(kBN / 2), l0); tmem_ld_16x256_x4(t1 + uint32_t(kBN / 2), l1); }
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            float f0[16], f1[16];
            tmem_ld_wait_16(h0);
            tmem_ld_wait_16(h1);
            if (LIMBS == 2) {
                tmem_ld_wait_16(l0);
                tmem_ld_wait_16(l1);
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    f0[e] = float(int32_t(h0[e]) * 256 + int32_t(l0[e]));
                    f1[e] = float(int32_t(h1[e]) * 256 + int32_t(l1[e]));
                }
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) { f0[e] = float(int32_t(h0[e])); f1[e] = float(int32_t(h1[e])); }
            }
            if (ch + 1 < NCH) {                          // the next chunk's loads fly while this one is processed
                const uint32_t c = uint32_t((ch + 1) * 32);
                tmem_ld_16x256_x4(t0 + c, h0);
                tmem_ld_16x256_x4(t1 + c, h1);
                if (LIMBS == 2) { tmem_ld_16x256_x4(t0 + c + uint32_t(kBN / 2), l0); tmem_ld_16x256_x4(t1 + c + uint32_t(kBN / 2), l1); }
            } else {                                     // accumulator fully read: hand it back to the MMA warp
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->tempty[as]);
            }
            // two staging buffers, used in turn: the copy engine must be done reading the one written two chunks ago
            unsigned char* buf = stg + ((i * NCH + ch) & 1) * kStagingBytes;
            if (lane == 0) bulk_wait_read_1();
            __syncwarp();
#pragma unroll
            for (int n = 0; n < 4; ++n) {
                const int c = 2 * (ch * 4 + n);          // index of this repeat's column pair in sw / bb
                unsigned char* wr = buf + tr * 64 + ((uint32_t(n) ^ rsw) << 4) + 4 * tq;
                // slab 0: rows tr, tr + 8; slab 1: rows tr + 16, tr + 24
                *reinterpret_cast<uint32_t*>(wr) = pack_bf16x2(fmaf(f0[4 * n + 0] * sw[c], sa_eff[0], bb[c]),
                                                               fmaf(f0[4 * n + 1] * sw[c + 1], sa_eff[0], bb[c + 1]));
                *reinterpret_cast<uint32_t*>(wr + 8 * 64) = pack_bf16x2(fmaf(f0[4 * n + 2] * sw[c], sa_eff[1], bb[c]),
                                                                        fmaf(f0[4 * n + 3] * sw[c + 1], sa_eff[1], bb[c + 1]));
                *reinterpret_cast<uint32_t*>(wr + 16 * 64) = pack_bf16x2(fmaf(f1[4 * n + 0] * sw[c], sa_eff[2], bb[c]),
                                                                         fmaf(f1[4 * n + 1] * sw[c + 1], sa_eff[2], bb[c + 1]));
                *reinterpret_cast<uint32_t*>(wr + 24 * 64) = pack_bf16x2(fmaf(f1[4 * n + 2] * sw[c], sa_eff[3], bb[c]),
                                                                         fmaf(f1[4 * n + 3] * sw[c + 1], sa_eff[3], bb[c + 1]));
            }
            fence_proxy_async_smem();                    // the lanes' writes become visible to the copy engine
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(tmY, buf, col_base + ch * 32, row0);
                bulk_commit_group();
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) sa[j] = sa_nx[j];
    }
    if (lane == 0) bulk_wait_read_all();                 // shared memory must outlive the copy engine's reads
}

// The kernel is compiled once per combination of
//   NIBBLE   container of the activation codes (the nibble container adds the four unpack warps),
//   MODE     kModeFast: bf16 output through bulk tensor stores, limbs recombined as 256*hi + lo without overflow (the
//            host checks the conditions); kModeGeneric: every other output form; kModePerTap: the per-filter-tap drain
//            of the accumulator (one activation scale per input pixel),
//   CONV     implicit-GEMM convolution (4-D activation boxes, pixel geometry) or plain GEMM,
//   LIMBS_T  weight limbs (1 or 2), or 0 = read at run time,
//   RES_T    weights resident (1) / streamed (0), or -1 = read at run time,
//   FRAG     fragment-layout epilogue and a second MMA issuer (fast mode with one code per byte only; see use_frag),
// because the hot loop of each role is short and runs once per tile: run-time branches over these choices and the
// code of the paths not taken cost 10-15 % on the K <= 512 shapes (instruction fetch and bookkeeping per tile).
template <bool NIBBLE, int MODE, bool CONV, int LIMBS_T, int RES_T, bool FRAG>
__global__ void __launch_bounds__(cta_threads(NIBBLE, FRAG), 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const __grid_constant__ CUtensorMap tmY, const GemmParams p) {
    constexpr bool PERTAP = MODE == kModePerTap;
    static_assert(!FRAG || (MODE == kModeFast && !NIBBLE), "the fragment-layout epilogue exists for the fast mode with one code per byte");
    // MMA-issuing warps: two (warp 1 and the CTA's last warp) together with the fragment-layout epilogue, else one
    constexpr int ISSUERS = FRAG ? 2 : 1;
    constexpr int kIssuer2 = 2 + kEpiWarps;
    const int limbs = LIMBS_T != 0 ? LIMBS_T : p.limbs;
    const bool resident = RES_T >= 0 ? (RES_T != 0) : (p.b_resident != 0);
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int num_kb = p.kb_per_tap * p.taps;
    const SmemLayout L = smem_layout(p.stages, resident, num_kb, FRAG);
    unsigned char* sB = smem + L.b_off;
    unsigned char* sA = smem + L.a_off;
    unsigned char* sStage = smem + L.staging_off;
    float* sParam = reinterpret_cast<float*>(smem + L.param_off);
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + L.ctl_off);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const TileCursor walk = tile_begin(p, resident);
    const int nstages = p.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->full2[s], 1);
            mbar_init(&ctl->empty[s], 1);
            mbar_init(&ctl->rawread[s], 128);
            mbar_init(&ctl->unpacked[s], 128);
        }
        for (int k = 0; k < kResidentKb; ++k) mbar_init(&ctl->bfull[k], 1);
        mbar_init(&ctl->bfree, ISSUERS);
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], kEpiWarps); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        if (p.tma_store) tma_prefetch_desc(&tmY);
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
            int cur_n = -1, reloads = 0;
            long long armed = 0;
            uint32_t par_a = 0, par_b = 0;     // per stage: parity of the next phase of full[] / full2[]
            uint32_t last_fill = 0;            // per stage: which of the two barriers its latest fill was armed on
            bool ok = true;
            TileCursor cur = walk;
            for (int i = 0; i < walk.count && ok; ++i, tile_next(p, cur, resident)) {
                const TileCoord tc = tile_coord<CONV>(p, cur);
                if (resident && tc.n_tile != cur_n) {
                    // the previous weight tile must have been read by its last MMA before it is overwritten
                    if (reloads > 0 &&
                        !wait_or_abort(&ctl->bfree, uint32_t(reloads - 1) & 1u, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    for (int kb = 0; kb < num_kb; ++kb) {
                        mbar_expect_tx(&ctl->bfull[kb], kBBytes);
                        tma_load_2d(sB + kb * kBBytes, &tmB, &ctl->bfull[kb], kb * kBK, tc.n_tile * kBN);
                    }
                    cur_n = tc.n_tile; ++reloads;
                }
                // Weights do not depend on the kernel before this one, activation codes do: with a programmatic
                // dependent launch the first weight tile is on its way while that kernel finishes.
                if (i == 0) griddep_wait();
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!wait_or_abort(&ctl->empty[stage], phase ^ 1, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    // the stage's arrival is signalled on the barrier of the issuer that takes this tile
                    uint64_t* fbar = (ISSUERS == 2 && (i & 1)) ? &ctl->full2[stage] : &ctl->full[stage];
                    if (ISSUERS == 2 && (i & 1)) { last_fill |= 1u << stage; par_b ^= 1u << stage; }
                    else { last_fill &= ~(1u << stage); par_a ^= 1u << stage; }
                    mbar_expect_tx(fbar, p.a_box_bytes + (resident ? 0u : uint32_t(kBBytes)));
                    unsigned char* a_dst = sA + stage * kABytes + (NIBBLE ? kABytes - kRawBytes : 0);
                    const int a_k = (NIBBLE ? kBK / 2 : kBK);
                    if (CONV) {
                        const int tap = kb / p.kb_per_tap, kc = kb - tap * p.kb_per_tap;
                        const int r = tap / p.S, s = tap - r * p.S;
                        tma_load_4d(a_dst, &tmA, fbar, kc * a_k, tc.w0 * p.stride + s - p.pad,
                                    tc.h0 * p.stride + r - p.pad, tc.n0);
                    } else {
                        tma_load_2d(a_dst, &tmA, fbar, kb * a_k, tc.m_tile * kBM);
                    }
                    if (!resident) tma_load_2d(sB + stage * kBBytes, &tmB, fbar, kb * kBK, tc.n_tile * kBN);
                    ++armed;
                    if (++stage == nstages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // Abort path: wait (bounded) for the copies this thread started so none lands after the CTA exits.
                if (reloads > 0)
                    for (int kb = 0; kb < num_kb; ++kb) mbar_wait(&ctl->bfull[kb], uint32_t(reloads - 1) & 1u, nullptr, 0);
                const int back = armed < nstages ? int(armed) : nstages;
                for (int j = 0; j < back; ++j) {
                    if (--stage < 0) stage = nstages - 1;
                    const bool second = (last_fill >> stage) & 1u;
                    const uint32_t armed_parity = (((second ? par_b : par_a) >> stage) & 1u) ^ 1u;   // the phase armed last
                    mbar_wait(second ? &ctl->full2[stage] : &ctl->full[stage], armed_parity, nullptr, 0);
                }
            }
        }
    } else if (warp == 1 || (ISSUERS == 2 && warp == kIssuer2)) {
        // ------------------------------------------------------------------ MMA issuer(s)
        // One lane needs about as long to get a K block issued (barrier wait, fence, four MMAs, commit) as the tensor
        // pipe needs to run it, so with a single issuer every wait at a tile change leaves the pipe idle.  With two,
        // warp 1 takes the even tiles (accumulator 0) and the CTA's last warp the odd ones (accumulator 1).  They share
        // the ring of operand stages; the producer signals a stage on full[] or full2[] according to the tile it
        // belongs to, so each barrier has one waiter who sees all of its phases in order.
        if (lane == 0) {
            const int me = warp == 1 ? 0 : 1;
            uint64_t* fullbar = me ? ctl->full2 : ctl->full;
            const uint32_t idesc = make_idesc_i8(kBM, kBN);
            int stage = 0; uint32_t phase = 0;            // position in the ring (phase: the unpack barriers' parity)
            uint32_t par = 0;                             // per stage: parity of the next phase of this issuer's barrier
            int cur_n = -1, reloads = 0;
            bool ok = true, pending_b = false;
            TileCursor cur = walk;
            // One accumulator per tile, or (per-tap mode) one per filter tap of a tile; they alternate between the
            // two TMEM buffers in the order they are produced.
            const int groups = PERTAP ? p.taps : 1;
            const int kb_per_group = num_kb / groups;
            int seq = 0;
            for (int i = 0; i < walk.count && ok; ++i, tile_next(p, cur, resident)) {
                if (resident && cur.n_tile != cur_n) { cur_n = cur.n_tile; ++reloads; pending_b = true; }
                const bool mine = ISSUERS == 1 || (i & 1) == me;
                if (!mine) {
                    // The other issuer's tile: step over its stages.  New weights are waited for here all the same, so
                    // that this lane sees every phase of the weight barriers (a parity wait cannot tell phase r from r+2).
                    if (pending_b) {
                        for (int kb = 0; kb < num_kb && ok; ++kb)
                            if (!wait_or_abort(&ctl->bfull[kb], uint32_t(reloads - 1) & 1u, ctl, p.dev_status, kStatusTmaWait)) ok = false;
                        pending_b = false;
                    }
                    stage += num_kb;
                    while (stage >= nstages) { stage -= nstages; phase ^= 1; }
                } else {
                    const bool new_b = pending_b;          // first use of these weights: wait per K block before its MMAs
                    pending_b = false;
                    for (int g = 0; g < groups && ok; ++g, ++seq) {
                        const int as = ISSUERS == 2 ? me : (seq & 1);
                        const uint32_t aphase = ISSUERS == 2 ? uint32_t(i >> 1) & 1u : uint32_t(seq >> 1) & 1u;
                        if (!wait_or_abort(&ctl->tempty[as], aphase ^ 1, ctl, p.dev_status, kStatusAccumFree)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + uint32_t(as * kBN);
                        for (int kk = 0; kk < kb_per_group; ++kk) {
                            const int kb = g * kb_per_group + kk;
                            if (new_b && !wait_or_abort(&ctl->bfull[kb], uint32_t(reloads - 1) & 1u, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                            if (!wait_or_abort(&fullbar[stage], (par >> stage) & 1u, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                            par ^= 1u << stage;
                            if (NIBBLE) {
                                if (!wait_or_abort(&ctl->unpacked[stage], phase, ctl, p.dev_status, kStatusUnpackWait)) { ok = false; break; }
                            }
                            tc_fence_after();
                            const uint64_t a_desc = make_sw128_kmajor_desc(smem_u32(sA + stage * kABytes));
                            const uint64_t b_desc = make_sw128_kmajor_desc(smem_u32(sB + (resident ? kb : stage) * kBBytes));
#pragma unroll
                            for (int k = 0; k < kBK / 32; ++k)
                                mma_i8(d_tmem, a_desc + uint64_t(k * 2), b_desc + uint64_t(k * 2), idesc, (kk | k) != 0 ? 1u : 0u);
                            mma_commit(&ctl->empty[stage]);
                            if (++stage == nstages) { stage = 0; phase ^= 1; }
                        }
                        if (ok) mma_commit(&ctl->tfull[as]);
                    }
                }
                // The next tile of the range starts a new weight tile: tell the producer when this issuer's MMAs on the
                // old one are done (the barrier counts one arrival per issuer; an issuer with nothing in flight
                // arrives at once).
                if (ok && resident && i + 1 < walk.count && cur.m_tile + 1 == p.tiles_m) mma_commit(&ctl->bfree);
            }
        }
    } else if (FRAG && warp < 2 + kEpiWarps) {
        // ------------------------------------------------------------------ epilogue (warps 2-9), fragment layout
        if constexpr (FRAG)
            fast_epilogue_warp<CONV, LIMBS_T>(p, walk, resident, ctl, tmem_base, sStage + (warp - 2) * 2 * kStagingBytes, &tmY,
                                              warp, lane);
    } else if (warp < 2 + kEpiWarps) {
        // ------------------------------------------------------------------ epilogue (warps 2-9)
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int chalf = (warp - 2) >> 2;            // which half of the tile's columns this warp takes
        unsigned char* stg = sStage + (warp - 2) * kStagingBytes;
        float* prm_sw = sParam + (warp - 2) * 2 * (kBN / 2);
        float* prm_b = prm_sw + kBN / 2;
        const int cols_per_tile = limbs == 2 ? kBN / 2 : kBN;
        const int cols_per_warp = cols_per_tile / 2;
        const bool want_y = MODE == kModeFast ? true : p.y != nullptr;
        const bool want_acc = MODE == kModeFast ? false : p.acc_out != nullptr;
        bool ok = true;
        TileCursor cur = walk;
        int last_n = -1;
        float sa_next = 0.f;
        griddep_wait();                               // scale_a comes from the kernel before this one
        for (int i = 0; i < walk.count && ok; ++i, tile_next(p, cur, resident)) {
            const int as = i & 1;
            const uint32_t aphase = (i >> 1) & 1;
            const TileCoord tc = tile_coord<CONV>(p, cur);
            const int col_base = tc.n_tile * cols_per_tile;
            // This warp's columns [wc0, wc0 + cols_per_warp) of the tile; their scale_w / bias go to the warp's own
            // slice of shared memory (read back as broadcasts), so no CTA-wide barrier is needed.
            const int wc0 = chalf * cols_per_warp;
            if (want_y && tc.n_tile != last_n) {       // consecutive tiles under resident weights share their columns
                last_n = tc.n_tile;
                __syncwarp();
                for (int c = lane; c < cols_per_warp; c += 32) {
                    const int col = col_base + wc0 + c;
                    prm_sw[c] = col < p.N ? __ldg(p.scale_w + col) : 0.f;
                    prm_b[c] = (p.bias != nullptr && col < p.N) ? __ldg(p.bias + col) : 0.f;
                }
                __syncwarp();
            }
            if (PERTAP) {
                // One scale per INPUT pixel: every filter tap's integer sum is drained on its own, multiplied by the
                // scale of the pixel that tap read for this output pixel, and added up in fp32 registers (64 columns
                // per warp and launch).  y = alpha * S_w[o] * sum_taps S_a[pix(tap)] * acc_tap + bias[o].
                const int pc0 = limbs == 2 ? wc0 : wc0 + p.col_pass * 64;   // first column (in the tile) handled here
                const int r_tile = q * 32 + lane;
                const int iw = r_tile % p.bw, ih = (r_tile / p.bw) % p.bh, in_ = r_tile / (p.bw * p.bh);
                const int n = tc.n0 + in_, ho = tc.h0 + ih, wo = tc.w0 + iw;
                const bool row_ok = in_ < p.bn && n < p.Nb && ho < p.Ho && wo < p.Wo;
                const int my_out = row_ok ? (n * p.Ho + ho) * p.Wo + wo : -1;
                auto tap_scale = [&](int g) -> float {
                    const int r = g / p.S, sx = g - r * p.S;
                    const int hi_ = ho * p.stride + r - p.pad, wi_ = wo * p.stride + sx - p.pad;
                    if (!row_ok || hi_ < 0 || hi_ >= p.H || wi_ < 0 || wi_ >= p.W) return 0.f;
                    return __ldg(p.scale_a + (int64_t(n) * p.H + hi_) * p.W + wi_);
                };
                float run[64];
#pragma unroll
                for (int j = 0; j < 64; ++j) run[j] = 0.f;
                float s_next = tap_scale(0);
                for (int g = 0; g < p.taps && ok; ++g) {
                    const int seq = i * p.taps + g;
                    const int as2 = seq & 1;
                    const float s_g = s_next;
                    if (g + 1 < p.taps) s_next = tap_scale(g + 1);
                    if (!wait_or_abort(&ctl->tfull[as2], uint32_t(seq >> 1) & 1u, ctl, p.dev_status, kStatusAccumWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t t_tap = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as2 * kBN + pc0);
                    uint32_t hi[16], lo[16];
                    tmem_ld_32x16(t_tap, hi);
                    if (limbs == 2) tmem_ld_32x16(t_tap + uint32_t(kBN / 2), lo);
#pragma unroll
                    for (int st = 0; st < 4; ++st) {
                        int32_t w[16];
                        tmem_ld_wait_16(hi);
                        if (limbs == 2) {
                            tmem_ld_wait_16(lo);
                            if (p.combine_fast) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) w[j] = int32_t(hi[j]) * 256 + int32_t(lo[j]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    w[j] = ((int32_t(hi[j]) >> p.a_shift) << 8) + (int32_t(lo[j]) >> p.a_shift);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j) w[j] = p.combine_fast ? int32_t(hi[j]) : (int32_t(hi[j]) >> p.a_shift);
                        }
                        if (st < 3) {
                            tmem_ld_32x16(t_tap + uint32_t((st + 1) * 16), hi);
                            if (limbs == 2) tmem_ld_32x16(t_tap + uint32_t(kBN / 2 + (st + 1) * 16), lo);
                        } else {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&ctl->tempty[as2]);
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) run[st * 16 + j] = fmaf(float(w[j]), s_g, run[st * 16 + j]);
                    }
                }
                if (!ok) break;
                if (my_out >= 0) {
                    const float a_eff = p.combine_fast ? p.alpha / float(1 << p.a_shift) : p.alpha;
                    const int prm0 = pc0 - wc0;                    // offset into the warp's staged column parameters
                    unsigned char* y_row = static_cast<unsigned char*>(p.y) + int64_t(my_out) * p.ldy * (p.y_bf16 ? 2 : 4);
#pragma unroll
                    for (int st = 0; st < 4; ++st) {
                        uint32_t f[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            f[j] = __float_as_uint(fmaf(run[st * 16 + j] * prm_sw[prm0 + st * 16 + j], a_eff, prm_b[prm0 + st * 16 + j]));
                        const int col = col_base + pc0 + st * 16;
                        if (col < p.N) {
                            if (p.y_bf16) store_row16<2>(y_row, f, col, p.N, p.y_vec_ok != 0);
                            else store_row16<4>(y_row, f, col, p.N, p.y_vec_ok != 0);
                        }
                    }
                }
                continue;
            }
            const int my_row = out_row_of<CONV>(p, tc, q * 32 + lane);
            // the row scale of this tile was requested while the previous tile was processed
            float sa_raw = sa_next;
            if (i == 0 && want_y) {
                if (p.sa_scalar) sa_raw = __ldg(p.scale_a);
                else if (my_row >= 0) sa_raw = __ldg(p.scale_a + my_row);
            }
            int next_row = -1;
            if (i + 1 < walk.count && want_y && !p.sa_scalar) {
                TileCursor nx = cur;
                tile_next(p, nx, resident);
                next_row = out_row_of<CONV>(p, tile_coord<CONV>(p, nx), q * 32 + lane);
            }
            int rows[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) rows[j] = out_row_of<CONV>(p, tc, q * 32 + j * 8 + (lane >> 2));
            if (!wait_or_abort(&ctl->tfull[as], aphase, ctl, p.dev_status, kStatusAccumWait)) { ok = false; break; }
            tc_fence_after();
            if (next_row >= 0) sa_next = __ldg(p.scale_a + next_row);
            else if (p.sa_scalar) sa_next = sa_raw;
            float sa_eff = 0.f;
            if (want_y && my_row >= 0) {
                sa_eff = p.alpha * sa_raw;
                if (p.combine_fast) sa_eff *= 1.0f / float(1 << p.a_shift);
            }
            if constexpr (MODE == kModeFast) {
                // rows of the tile are consecutive output rows (checked on the host); this warp owns 32 of them
                const int row0 = out_row_of<CONV>(p, tc, 0) + q * 32;
                const uint32_t t_fast = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN + wc0);
                epilogue_fast<LIMBS_T, !NIBBLE>(t_fast, stg, lane, prm_sw, prm_b, sa_eff, &tmY, col_base + wc0, row0, &ctl->tempty[as]);
                continue;
            }

            // walk the warp's columns in steps of 16
            int nsteps = cols_per_warp / 16;
            if (col_base + wc0 + nsteps * 16 > p.N) {
                const int left = p.N - (col_base + wc0);
                nsteps = left > 0 ? (left + 15) / 16 : 0;
            }
            const uint32_t t_row = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN + wc0);
            uint32_t hi[16], lo[16];
            if (nsteps > 0) {
                tmem_ld_32x16(t_row, hi);
                if (limbs == 2) tmem_ld_32x16(t_row + uint32_t(kBN / 2), lo);
            }
            for (int st = 0; st < nsteps; ++st) {
                const int tcol = wc0 + st * 16;        // column inside the tile
                uint32_t val[16];
                tmem_ld_wait_16(hi);
                if (limbs == 2) {
                    tmem_ld_wait_16(lo);
                    if (p.combine_fast) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) val[j] = uint32_t(int32_t(hi[j]) * 256 + int32_t(lo[j]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            val[j] = uint32_t(((int32_t(hi[j]) >> p.a_shift) << 8) + (int32_t(lo[j]) >> p.a_shift));
                    }
                } else if (p.combine_fast) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) val[j] = hi[j];
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) val[j] = uint32_t(int32_t(hi[j]) >> p.a_shift);
                }
                if (st + 1 < nsteps) {                 // the next step's loads fly while this one is processed
                    tmem_ld_32x16(t_row + uint32_t((st + 1) * 16), hi);
                    if (limbs == 2) tmem_ld_32x16(t_row + uint32_t(kBN / 2 + (st + 1) * 16), lo);
                } else {                               // accumulator fully read: hand it back to the MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->tempty[as]);
                }
                if (want_acc && my_row >= 0) {         // each lane stores 64 contiguous bytes of its own row
                    int32_t* dst = p.acc_out + int64_t(my_row) * p.N + col_base + tcol;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        int32_t a4[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            a4[e] = p.combine_fast ? (int32_t(val[j + e]) >> p.a_shift) : int32_t(val[j + e]);
                        if (p.acc_vec_ok && col_base + tcol + j + 4 <= p.N) {
                            *reinterpret_cast<int4*>(dst + j) = make_int4(a4[0], a4[1], a4[2], a4[3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) if (col_base + tcol + j + e < p.N) dst[j + e] = a4[e];
                        }
                    }
                }
                if (want_y) {
                    const float4* sw4 = reinterpret_cast<const float4*>(prm_sw + st * 16);
                    const float4* b4 = reinterpret_cast<const float4*>(prm_b + st * 16);
                    uint32_t f[16];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float4 sw = sw4[j], bb = b4[j];
                        f[4 * j + 0] = __float_as_uint(fmaf(float(int32_t(val[4 * j + 0])) * sw.x, sa_eff, bb.x));
                        f[4 * j + 1] = __float_as_uint(fmaf(float(int32_t(val[4 * j + 1])) * sw.y, sa_eff, bb.y));
                        f[4 * j + 2] = __float_as_uint(fmaf(float(int32_t(val[4 * j + 2])) * sw.z, sa_eff, bb.z));
                        f[4 * j + 3] = __float_as_uint(fmaf(float(int32_t(val[4 * j + 3])) * sw.w, sa_eff, bb.w));
                    }
                    if (p.y_bf16) {
                        stage_put<2>(stg, f, lane, st & 1);
                        if ((st & 1) || st + 1 == nsteps)
                            stage_flush<2>(stg, lane, p.y, p.ldy, p.N, col_base + wc0 + (st & ~1) * 16, rows,
                                           p.y_vec_ok != 0);
                    } else {
                        stage_put<4>(stg, f, lane, 0);
                        stage_flush<4>(stg, lane, p.y, p.ldy, p.N, col_base + tcol, rows, p.y_vec_ok != 0);
                    }
                }
            }
            if (nsteps == 0) {                         // this warp's columns lie beyond N: nothing to read
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->tempty[as]);
            }
        }
        if (lane == 0) bulk_wait_read_all();           // shared memory must outlive the copy engine's reads
    } else if (NIBBLE) {
        // ------------------------------------------------------------------ nibble -> int8 unpack (warps 10-13)
        // The packed tile (128 rows x 64 bytes) lands in the upper half of the 16 KB operand stage; every thread
        // first takes its share into registers, then (after a barrier of the four warps) the stage is rewritten
        // in place as 128 rows x 128 bytes with the 128-byte swizzle the MMA descriptor expects.
        const int t = threadIdx.x - (2 + kEpiWarps) * 32;    // 0..127
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        for (int i = 0; i < walk.count && ok; ++i) {
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!wait_or_abort(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                unsigned char* dstA = sA + stage * kABytes;
                const uint4* raw = reinterpret_cast<const uint4*>(dstA + kABytes - kRawBytes);
                uint4 w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) w[j] = raw[j * 128 + t];
                mbar_arrive(&ctl->rawread[stage]);     // the stage may be overwritten once all 128 threads got here
                if (!wait_or_abort(&ctl->rawread[stage], phase, ctl, p.dev_status, kStatusUnpackWait)) { ok = false; break; }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int id = j * 128 + t;           // 16-byte chunk of the packed tile: row = id/4, part = id%4
                    const int row = id >> 2, part = id & 3;
                    uint4 o0, o1;
                    o0.x = (w[j].x << 4) & 0xF0F0F0F0u; o0.y = w[j].x & 0xF0F0F0F0u;
                    o0.z = (w[j].y << 4) & 0xF0F0F0F0u; o0.w = w[j].y & 0xF0F0F0F0u;
                    o1.x = (w[j].z << 4) & 0xF0F0F0F0u; o1.y = w[j].z & 0xF0F0F0F0u;
                    o1.z = (w[j].w << 4) & 0xF0F0F0F0u; o1.w = w[j].w & 0xF0F0F0F0u;
                    unsigned char* rowp = dstA + row * 128;
                    *reinterpret_cast<uint4*>(rowp + (((2 * part) ^ (row & 7)) << 4)) = o0;
                    *reinterpret_cast<uint4*>(rowp + (((2 * part + 1) ^ (row & 7)) << 4)) = o1;
                }
                fence_proxy_async_smem();
                mbar_arrive(&ctl->unpacked[stage]);
                if (++stage == nstages) { stage = 0; phase ^= 1; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}


// Launches one instantiation; the first launch per device raises its dynamic shared-memory limit.
template <bool NIBBLE, int MODE, bool CONV, int LIMBS_T, int RES_T, bool FRAG = false>
cudaError_t launch_one(int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA, const CUtensorMap& tmB,
                       const CUtensorMap& tmY, const GemmParams& p) {
    static bool attr_set[64] = {};
    auto kern = qgemm_kernel<NIBBLE, MODE, CONV, LIMBS_T, RES_T, FRAG>;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    if (p.pdl) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(unsigned(grid)); cfg.blockDim = dim3(unsigned(cta_threads(NIBBLE, FRAG)));
        cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, p);
    }
    kern<<<grid, cta_threads(NIBBLE, FRAG), smem, st>>>(tmA, tmB, tmY, p);
    return cudaGetLastError();
}

// Picks the instantiation for (mode, limbs, resident) of one container and problem kind.
template <bool NIBBLE, bool CONV>
cudaError_t dispatch(int mode, int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA, const CUtensorMap& tmB,
                     const CUtensorMap& tmY, const GemmParams& p) {
    if (mode == kModeFast) {
        if constexpr (!NIBBLE) {
            if (p.frag) {
                if (!p.b_resident) return cudaErrorInvalidValue;       // chosen for resident weights only
                return p.limbs == 1 ? launch_one<NIBBLE, kModeFast, CONV, 1, 1, true>(grid, smem, st, tmA, tmB, tmY, p)
                                    : launch_one<NIBBLE, kModeFast, CONV, 2, 1, true>(grid, smem, st, tmA, tmB, tmY, p);
            }
        }
        if (p.limbs == 2)
            return p.b_resident ? launch_one<NIBBLE, kModeFast, CONV, 2, 1>(grid, smem, st, tmA, tmB, tmY, p)
                                : launch_one<NIBBLE, kModeFast, CONV, 2, 0>(grid, smem, st, tmA, tmB, tmY, p);
        return p.b_resident ? launch_one<NIBBLE, kModeFast, CONV, 1, 1>(grid, smem, st, tmA, tmB, tmY, p)
                            : launch_one<NIBBLE, kModeFast, CONV, 1, 0>(grid, smem, st, tmA, tmB, tmY, p);
    }
    if (mode == kModePerTap) {
        if constexpr (CONV) return launch_one<NIBBLE, kModePerTap, true, 0, -1>(grid, smem, st, tmA, tmB, tmY, p);
        else return cudaErrorInvalidValue;
    }
    return launch_one<NIBBLE, kModeGeneric, CONV, 0, -1>(grid, smem, st, tmA, tmB, tmY, p);
}

// One definition each in hq_gemm_inst_*.cu.
cudaError_t launch_i8_gemm(int mode, int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA,
                           const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p);
cudaError_t launch_i8_conv(int mode, int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA,
                           const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p);
cudaError_t launch_nibble_gemm(int mode, int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA,
                               const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p);
cudaError_t launch_nibble_conv(int mode, int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA,
                               const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p);

}  // namespace gemm

// Host helpers defined in hq_gemm.cu: tensor-map encoders (byte matrices with an optional 128-byte swizzle; the bf16
// output map with 32 x 32 boxes in the 64-byte swizzle) and the SM count of the current device.
bool encode_2d(CUtensorMap* tm, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
               uint32_t box_inner, uint32_t box_rows, bool swizzle128);
bool encode_y(CUtensorMap* tm, const void* y, uint64_t N, uint64_t rows, uint64_t ldy);
int sm_count();
}  // namespace hq
