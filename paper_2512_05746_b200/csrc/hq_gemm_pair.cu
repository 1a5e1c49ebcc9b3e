// Integer GEMM with the rescale epilogue (Eq. 12) on PAIRS of SMs: tcgen05.mma.cta_group::2.
//
// Two CTAs of a cluster share one 256 x 256 x K tile: each holds its own 128 activation rows and HALF of the 256
// operand-B rows in its shared memory (with two weight limbs: one CTA the "hi" rows, the other the "lo" rows), one lane of
// the leader CTA issues every MMA for both tensor cores, and each CTA's tensor memory receives the 128 x 256 accumulator of
// its own rows.  Per SM and MMA the tensor core reads 8 KB of operands from its shared memory instead of 12 KB -- the
// shared-memory data pipe is the busiest unit of the one-CTA kernel on short reductions -- and the resident weight tile
// shrinks to 64 KB, which leaves room for an activation ring of eight 16 KB stages, or of three 32 KB stages (two K blocks
// each, K_pad 256 / 512: half the barrier rounds for the issuing lane).
//
// Covered: plain GEMM, one code per byte, K_pad <= 512 (weights resident), bf16 output through bulk tensor stores; below
// this kernel, the same protocol with streamed weights for longer reductions and convolutions.
// Every CTA issues its own TMA loads (no multicast); the loads of the second CTA signal the leader's barriers; MMA
// completion is committed to both CTAs' barriers; the second CTA's epilogue warps release the accumulators with remote
// barrier arrivals.  Every wait is bounded.
#include <cuda.h>

#include "hq_gemm_kernel.cuh"

namespace hq {
namespace {
using namespace gemm;

// 16-column epilogue steps whose column parameters stay in registers in the kernels with two K blocks per ring stage
// (two of a two-limb warp's four: 64 registers; with three the kernel spills and measured slower).
constexpr int kPairRegSteps = 2;
constexpr int kPairThreads = 320;              // producer warp, MMA warp, eight epilogue warps
constexpr int kPairMaxStages = 8;
constexpr int kPairBBytes = 128 * kBK;         // this CTA's half of a weight K block: 128 rows x 128 bytes
constexpr int kPairParamBytes = kEpiWarps * 2 * (kBN / 2) * 4;

struct PairParams {
    int64_t M; int N, limbs, num_kb, tiles_m2, tiles_n, stages;
    const float* scale_a; int sa_scalar;
    const float* scale_w; const float* bias; float alpha;
    int pdl;
    int32_t* dev_status;
};

struct PairCtl {
    uint64_t full[kPairMaxStages];     // leader: both CTAs' activation stages have landed
    uint64_t empty[kPairMaxStages];    // each CTA: the MMAs that read the stage have completed
    uint64_t bfull[kResidentKb];       // leader: both halves of a weight K block have landed
    uint64_t bfree;                    // each CTA: the MMAs on the old weight tile have completed
    uint64_t tfull[2];                 // each CTA: an accumulator is complete
    uint64_t tempty[2];                // leader: both CTAs' epilogue warps have read an accumulator
    uint32_t tmem_base;
    volatile int abort_flag;
};

struct PairLayout { int b_off, a_off, staging_off, param_off, ctl_off, total; };
// kps: K blocks of a tile's activations per ring stage
__host__ __device__ inline PairLayout pair_layout(int num_kb, int stages, int kps = 1) {
    PairLayout L;
    L.b_off = 0;
    L.a_off = num_kb * kPairBBytes;
    L.staging_off = L.a_off + stages * kps * kABytes;
    L.param_off = L.staging_off + kEpiWarps * 2 * kStagingBytes;       // two staging buffers per epilogue warp
    L.ctl_off = L.param_off + kPairParamBytes;
    L.total = L.ctl_off + int(sizeof(PairCtl)) + 1024;
    return L;
}

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The address of the same shared-memory object in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_u32(p)), "r"(rank));
    return a;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    // default (CTA-scope release) semantics: what the arrival orders are this warp's tensor-memory reads, which the
    // tcgen05 fence in front of it covers; a cluster-scope release here drains the thread's whole memory pipeline
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion bytes are credited to the barrier at `bar_cluster_addr` (this CTA's or the leader's).
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the shared-memory descriptors given as (low word, high word): only the address field in the low word
// varies within a kernel, so the issuing lane advances a descriptor with one 32-bit addition.  ACC is a constant.
template <bool ACC>
__device__ __forceinline__ void mma_i8_pair_lh(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "n"(ACC ? 1 : 0)
        : "memory");
}
// Arrive on the barrier at the same offset in both CTAs of the pair once all MMAs issued so far have completed.
__device__ __forceinline__ void mma_commit_pair(uint64_t* bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask)
                 : "memory");
}

// One poll with a short suspend-time hint: barriers of this kernel are completed from the other CTA (remote arrivals,
// multicast commits, the peer's TMA bytes), and a thread parked for long on such a barrier is not resumed promptly.
#ifndef HQ_PAIR_WAIT_NS
#define HQ_PAIR_WAIT_NS 64
#endif
__device__ __forceinline__ bool pair_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(uint32_t(HQ_PAIR_WAIT_NS))
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool wait_pair(uint64_t* bar, uint32_t parity, PairCtl* ctl, int32_t* dev_status, int32_t code) {
    if (pair_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000000LL) {
        if (pair_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
    }
    ctl->abort_flag = 1;
    if (dev_status) atomicExch(dev_status, code);
    return false;
}

// The row-per-lane bulk-store epilogue of the one-CTA kernel (16 columns at a time: two tensor-memory loads, 256 * hi + lo,
// rescale, bf16 into a staging buffer in the 64-byte swizzle of the output tensor map, one bulk tensor store per 32
// columns), with the accumulator handed back by an arrival on the LEADER's barrier (a cluster address).
// PREG > 0: the column parameters of the warp's first PREG 16-column steps are in registers (`rsw`, `rb`; the caller
// loads them once per column tile).  Every lane needs all of them, so from shared memory they arrive as broadcast reads,
// 128 wavefronts per warp and tile, 1024 per tile on the data pipe that also feeds the tensor core its operands (1024 per
// tile) and takes the staging stores and the bulk stores' reads (520): together more than the 2144 cycles of a tile's MMAs.
// NBUF: the warp's staging buffers (two used in turn, or one).
template <int LIMBS, int PREG = 0, int NBUF = 2>
__device__ __forceinline__ void epilogue_pair(uint32_t t_row, unsigned char* stg, int lane, const float* prm_sw,
                                              const float* prm_b, float sa_eff, const CUtensorMap* tmY, int col0, int row0,
                                              uint32_t tempty_leader, const float (&rsw)[PREG > 0 ? PREG * 16 : 1] = {0.f},
                                              const float (&rb)[PREG > 0 ? PREG * 16 : 1] = {0.f}) {
    constexpr int NSTEPS = LIMBS == 2 ? kBN / 2 / 2 / 16 : kBN / 2 / 16;
    const uint32_t wsw = (lane >> 1) & 3;
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
            if (lane == 0) mbar_arrive_cluster(tempty_leader);
        }
        // two staging buffers, used in turn: the copy engine must be done reading the one written two stores ago
        unsigned char* buf = NBUF == 2 ? stg + ((st >> 1) & 1) * kStagingBytes : stg;
        unsigned char* wr = buf + lane * 64;
        if ((st & 1) == 0) {
            if (lane == 0) { if (NBUF == 2) bulk_wait_read_1(); else bulk_wait_read_all(); }
            __syncwarp();
        }
        const float4* sw4 = reinterpret_cast<const float4*>(prm_sw + st * 16);
        const float4* b4 = reinterpret_cast<const float4*>(prm_b + st * 16);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float4 s0, s1, c0, c1;
            if (st < PREG) {
                const int e = st * 16 + 8 * j;
                s0 = make_float4(rsw[e], rsw[e + 1], rsw[e + 2], rsw[e + 3]); s1 = make_float4(rsw[e + 4], rsw[e + 5], rsw[e + 6], rsw[e + 7]);
                c0 = make_float4(rb[e], rb[e + 1], rb[e + 2], rb[e + 3]); c1 = make_float4(rb[e + 4], rb[e + 5], rb[e + 6], rb[e + 7]);
            } else {
                s0 = sw4[2 * j]; s1 = sw4[2 * j + 1]; c0 = b4[2 * j]; c1 = b4[2 * j + 1];
            }
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
                tma_store_2d(tmY, buf, col0 + (st >> 1) * 32, row0);
                bulk_commit_group();
            }
        }
    }
}

// NKB > 0: the reduction has exactly NKB K blocks (compile-time loops) and a ring stage holds KPS = 2 of them (32 KB):
// one barrier round and one commit per two K blocks.  The issuing lane needs about 70 cycles per MMA and about 180 per
// barrier round, which for one K block per stage is as long as the tensor pipe runs the block (536 cycles); with two the
// lane is ahead of the pipe.  Three 32 KB stages fit beside the 64 KB weight half of K_pad = 512 (the pair halves the
// weights; the one-CTA kernel has 64 KB for all its stages).
template <int LIMBS, int NKB, int KPS>
__global__ void __launch_bounds__(kPairThreads, 1)
qgemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmY, const PairParams p) {
    constexpr bool WHOLE = NKB > 0;
    static_assert(NKB == 0 ? KPS == 1 : (KPS > 1 && NKB % KPS == 0), "a stage holds a whole fraction of the tile's K blocks");
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const PairLayout L = pair_layout(p.num_kb, p.stages, KPS);
    unsigned char* sB = smem + L.b_off;
    unsigned char* sA = smem + L.a_off;
    unsigned char* sStage = smem + L.staging_off;
    float* sParam = reinterpret_cast<float*>(smem + L.param_off);
    PairCtl* ctl = reinterpret_cast<PairCtl*>(smem + L.ctl_off);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                 // 0: leader (issues the MMAs), 1: its peer
    const int nstages = p.stages, num_kb = p.num_kb;
    // the pair's contiguous range of 256-row tiles in column-tile-major order (consecutive tiles share their weights).
    // A change of weight tile inside a range stalls the pair for about one tile (the old tile's MMAs drain, then 64 KB
    // per CTA arrive), and the slowest pair sets the kernel's time: the ranges are cut in units of cost, a column tile
    // costing its row tiles plus one, so that a pair that changes weights gets one tile fewer.
    const int G = gridDim.x >> 1, c = blockIdx.x >> 1;
    const int W = p.tiles_m2 + 1;
    const int64_t C = int64_t(p.tiles_n) * W;
    auto first_tile = [&](int pair) {
        const int64_t lo = (int64_t(pair) * C + G - 1) / G;        // first cost position of the pair
        int n = int(lo / W), m = int(lo - int64_t(n) * W);
        if (m == p.tiles_m2) { ++n; m = 0; }                        // the slot that stands for the weight change
        return n * p.tiles_m2 + m;
    };
    const int first = first_tile(c);
    const int count = first_tile(c + 1) - first;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairMaxStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int k = 0; k < kResidentKb; ++k) mbar_init(&ctl->bfull[k], 1);
        mbar_init(&ctl->bfree, 1);
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], 2 * kEpiWarps); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmY);
    }
    if (warp == 1) { __syncwarp(); tmem_alloc_pair(&ctl->tmem_base, kTmemCols); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised and both tensor memories allocated
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per CTA, its own halves)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            int cur_n = -1, reloads = 0;
            bool ok = true;
            for (int i = 0; i < count && ok; ++i) {
                const int u = first + i;
                const int n_tile = u / p.tiles_m2, m2 = u - n_tile * p.tiles_m2;
                if (n_tile != cur_n) {
                    // the previous weight tile must have been read by its last MMA before it is overwritten
                    if (reloads > 0 && !wait_pair(&ctl->bfree, uint32_t(reloads - 1) & 1u, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    for (int kb = 0; kb < num_kb; ++kb) {
                        if (rank == 0) mbar_expect_tx(&ctl->bfull[kb], 2u * uint32_t(kPairBBytes));
                        tma_load_2d_pair(sB + kb * kPairBBytes, &tmB, map_to_cta(&ctl->bfull[kb], 0), kb * kBK,
                                         n_tile * kBN + int(rank) * 128);
                    }
                    cur_n = n_tile; ++reloads;
                }
                if (i == 0 && p.pdl) griddep_wait();       // the codes come from the kernel before this one
                if constexpr (WHOLE) {
#pragma unroll
                    for (int h = 0; h < NKB / KPS; ++h) {
                        if (!wait_pair(&ctl->empty[stage], phase ^ 1, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                        if (rank == 0) mbar_expect_tx(&ctl->full[stage], 2u * uint32_t(KPS * kABytes));
                        const uint32_t fbar = map_to_cta(&ctl->full[stage], 0);
#pragma unroll
                        for (int k = 0; k < KPS; ++k)
                            tma_load_2d_pair(sA + (stage * KPS + k) * kABytes, &tmA, fbar, (h * KPS + k) * kBK,
                                             m2 * 256 + int(rank) * 128);
                        if (++stage == nstages) { stage = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                } else {
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!wait_pair(&ctl->empty[stage], phase ^ 1, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    if (rank == 0) mbar_expect_tx(&ctl->full[stage], 2u * uint32_t(kABytes));
                    tma_load_2d_pair(sA + stage * kABytes, &tmA, map_to_cta(&ctl->full[stage], 0), kb * kBK,
                                     m2 * 256 + int(rank) * 128);
                    if (++stage == nstages) { stage = 0; phase ^= 1; }
                }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_idesc_i8(256, kBN);
            int stage = 0; uint32_t phase = 0;
            int cur_n = -1, reloads = 0;
            bool ok = true;
            if constexpr (WHOLE) {
                // A lone lane runs its instructions one dependent step at a time (about five cycles each), so this loop is
                // kept to the instructions the tile needs: tile coordinates advance by counting, descriptors by one
                // 32-bit addition, the weight-tile barriers are visited only on the first tile of a column tile.
                const uint64_t dsc = make_sw128_kmajor_desc(smem_u32(sA));
                const uint32_t desc_hi = uint32_t(dsc >> 32), a_lo0 = uint32_t(dsc);
                const uint32_t b_lo0 = uint32_t(make_sw128_kmajor_desc(smem_u32(sB)));
                constexpr uint32_t kStageUnits = uint32_t(KPS * kABytes) >> 4;
                uint32_t a_lo = a_lo0;
                int m2 = first % p.tiles_m2;
                bool new_b = true;
                for (int i = 0; i < count; ++i) {
                    const int as = i & 1;
                    if (!wait_pair(&ctl->tempty[as], (uint32_t(i >> 1) & 1u) ^ 1u, ctl, p.dev_status, kStatusAccumFree)) break;
                    if (new_b) {
                        ++reloads;
                        bool okb = true;
#pragma unroll
                        for (int kb = 0; kb < NKB; ++kb)
                            okb = okb && wait_pair(&ctl->bfull[kb], uint32_t(reloads - 1) & 1u, ctl, p.dev_status, kStatusTmaWait);
                        if (!okb) break;
                        new_b = false;
                    }
                    const uint32_t d_tmem = tmem_base + uint32_t(as * kBN);
                    bool okt = true;
#pragma unroll
                    for (int h = 0; h < NKB / KPS; ++h) {
                        if (!wait_pair(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { okt = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int kk = 0; kk < KPS; ++kk) {
                            constexpr uint32_t kAUnits = uint32_t(kABytes) >> 4, kBUnits = uint32_t(kPairBBytes) >> 4;
                            const uint32_t al = a_lo + uint32_t(kk) * kAUnits, bl = b_lo0 + uint32_t(h * KPS + kk) * kBUnits;
                            if (h == 0 && kk == 0) mma_i8_pair_lh<false>(d_tmem, al, bl, desc_hi, idesc);
                            else mma_i8_pair_lh<true>(d_tmem, al, bl, desc_hi, idesc);
                            mma_i8_pair_lh<true>(d_tmem, al + 2, bl + 2, desc_hi, idesc);
                            mma_i8_pair_lh<true>(d_tmem, al + 4, bl + 4, desc_hi, idesc);
                            mma_i8_pair_lh<true>(d_tmem, al + 6, bl + 6, desc_hi, idesc);
                        }
                        mma_commit_pair(&ctl->empty[stage]);
                        a_lo += kStageUnits;
                        if (++stage == nstages) { stage = 0; phase ^= 1; a_lo = a_lo0; }
                    }
                    if (!okt) break;
                    mma_commit_pair(&ctl->tfull[as]);
                    // the next tile of the range starts a new weight tile: tell both producers when the MMAs on the old one are done
                    if (++m2 == p.tiles_m2) {
                        m2 = 0; new_b = true;
                        if (i + 1 < count) mma_commit_pair(&ctl->bfree);
                    }
                }
            } else
            for (int i = 0; i < count && ok; ++i) {
                const int u = first + i;
                const int n_tile = u / p.tiles_m2, m2 = u - n_tile * p.tiles_m2;
                bool new_b = false;
                if (n_tile != cur_n) { cur_n = n_tile; ++reloads; new_b = true; }
                const int as = i & 1;
                if (!wait_pair(&ctl->tempty[as], (uint32_t(i >> 1) & 1u) ^ 1u, ctl, p.dev_status, kStatusAccumFree)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + uint32_t(as * kBN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (new_b && !wait_pair(&ctl->bfull[kb], uint32_t(reloads - 1) & 1u, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                    if (!wait_pair(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_sw128_kmajor_desc(smem_u32(sA + stage * kABytes));
                    const uint64_t b_desc = make_sw128_kmajor_desc(smem_u32(sB + kb * kPairBBytes));
#pragma unroll
                    for (int k = 0; k < kBK / 32; ++k)
                        mma_i8_pair(d_tmem, a_desc + uint64_t(k * 2), b_desc + uint64_t(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
                    mma_commit_pair(&ctl->empty[stage]);
                    if (++stage == nstages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit_pair(&ctl->tfull[as]);
                // the next tile of the range starts a new weight tile: tell both producers when the MMAs on the old one are done
                if (i + 1 < count && m2 + 1 == p.tiles_m2) mma_commit_pair(&ctl->bfree);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2-9 of both CTAs)
        const int ew = warp - 2;
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int chalf = ew >> 2;                    // which half of the tile's columns this warp takes
        unsigned char* stg = sStage + ew * 2 * kStagingBytes;
        float* prm_sw = sParam + ew * 2 * (kBN / 2);
        float* prm_b = prm_sw + kBN / 2;
        constexpr int cols_per_tile = LIMBS == 2 ? kBN / 2 : kBN;
        constexpr int cols_per_warp = cols_per_tile / 2;
        const int wc0 = chalf * cols_per_warp;
        const uint32_t tempty_leader[2] = {map_to_cta(&ctl->tempty[0], 0), map_to_cta(&ctl->tempty[1], 0)};
        int last_n = -1;
        bool ok = true;
        float sa_next = 0.f;
        constexpr int PREG = WHOLE ? kPairRegSteps : 0;
        float rsw[PREG > 0 ? PREG * 16 : 1], rb[PREG > 0 ? PREG * 16 : 1];
        if (p.pdl) griddep_wait();                    // scale_a comes from the kernel before this one
        for (int i = 0; i < count && ok; ++i) {
            const int u = first + i;
            const int n_tile = u / p.tiles_m2, m2 = u - n_tile * p.tiles_m2;
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
                if constexpr (PREG > 0) {
#pragma unroll
                    for (int e = 0; e < PREG * 16; ++e) { rsw[e] = prm_sw[e]; rb[e] = prm_b[e]; }
                }
            }
            // the row scale of this tile was requested while the previous tile was processed
            float sa = sa_next;
            if (i == 0) {
                const int64_t my_row = int64_t(m2) * 256 + int(rank) * 128 + q * 32 + lane;
                sa = p.sa_scalar ? __ldg(p.scale_a) : (my_row < p.M ? __ldg(p.scale_a + my_row) : 0.f);
            }
            if (!wait_pair(&ctl->tfull[as], uint32_t(i >> 1) & 1u, ctl, p.dev_status, kStatusAccumWait)) { ok = false; break; }
            tc_fence_after();
            sa_next = sa;
            if (i + 1 < count && !p.sa_scalar) {
                const int u2 = u + 1;
                const int n2 = u2 / p.tiles_m2, m2n = u2 - n2 * p.tiles_m2;
                const int64_t row2 = int64_t(m2n) * 256 + int(rank) * 128 + q * 32 + lane;
                sa_next = row2 < p.M ? __ldg(p.scale_a + row2) : 0.f;
            }
            const float sa_eff = p.alpha * sa;
            const int row0 = m2 * 256 + int(rank) * 128 + q * 32;
            const uint32_t t_fast = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN + wc0);
            epilogue_pair<LIMBS, PREG>(t_fast, stg, lane, prm_sw, prm_b, sa_eff, &tmY, col_base + wc0, row0, tempty_leader[as], rsw, rb);
        }
        if (lane == 0) bulk_wait_read_all();           // shared memory must outlive the copy engine's reads
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // neither CTA leaves while its peer may still signal its barriers or read its operands
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

// ---- long reductions and convolutions on pairs of SMs: weights streamed --------------------------------------------
// Where the reduction does not fit a resident weight tile (K_pad > 512, every 3x3 convolution), the one-CTA kernel's
// issuing lane needs about as long per 128-byte K block (barrier wait, four MMAs, commit: ~600 cycles) as the tensor
// pipe needs to run it (536), and its ring holds four 48 KB stages.  On a pair of SMs one lane issues a K block for
// both tensor cores, each CTA brings its own 128 activation rows and HALF of the 256 weight rows of the block (32 KB
// per stage and CTA: six stages), and the same MMA count serves twice the rows.  Tiles are taken in row-major order,
// pair c the tiles c, c + G, ..., so that the pairs working side by side share their activation rows in L2.
// Convolution: a tile's 128 rows are 128 consecutive output pixels (whole output rows; checked by the host), fetched per
// filter tap by a 4-D bulk tensor load whose out-of-range coordinates supply the zero padding.
struct PairStreamParams {
    int64_t M; int N, limbs, num_kb, tiles_m2, tiles_n, stages;
    const float* scale_a; int sa_scalar;
    const float* scale_w; const float* bias; float alpha;
    int pdl;
    int32_t* dev_status;
    // convolution geometry (CONV instantiations)
    int kb_per_tap, S, stride, pad, bw, bh, bn, tiles_w, tiles_h;
};

constexpr int kPairStageBytes = kABytes + kPairBBytes;      // 32 KB: this CTA's activation rows and its half of the weights

struct PairStreamLayout { int ring_off, staging_off, param_off, ctl_off, total; };
// kps: K blocks per ring stage; with two, 64 KB stages, the epilogue warps have one staging buffer each instead of two
__host__ __device__ inline PairStreamLayout pair_stream_layout(int stages, int kps = 1) {
    PairStreamLayout L;
    L.ring_off = 0;
    L.staging_off = stages * kps * kPairStageBytes;
    L.param_off = L.staging_off + kEpiWarps * (kps == 2 ? 1 : 2) * kStagingBytes;
    L.ctl_off = L.param_off + kPairParamBytes;
    L.total = L.ctl_off + int(sizeof(PairCtl)) + 1024;
    return L;
}

__device__ __forceinline__ void tma_load_4d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr, int c0, int c1,
                                                 int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2),
          "r"(c3)
        : "memory");
}

// KPS = 2 (even K block counts): two K blocks per ring stage, laid out [A0 | B0 | A1 | B1]: the issuing lane's barrier
// rounds halve (a wait, a fence, eight MMAs and a commit per 64 KB stage); three stages fit.
template <int LIMBS, bool CONV, int KPS>
__global__ void __launch_bounds__(kPairThreads, 1)
qgemm_pair_stream_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const __grid_constant__ CUtensorMap tmY, const PairStreamParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const PairStreamLayout L = pair_stream_layout(p.stages, KPS);
    unsigned char* sRing = smem + L.ring_off;
    unsigned char* sStage = smem + L.staging_off;
    float* sParam = reinterpret_cast<float*>(smem + L.param_off);
    PairCtl* ctl = reinterpret_cast<PairCtl*>(smem + L.ctl_off);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                 // 0: leader (issues the MMAs), 1: its peer
    const int nstages = p.stages, num_kb = p.num_kb;
    const int T = p.tiles_m2 * p.tiles_n, G = gridDim.x >> 1, c = blockIdx.x >> 1;
    const int count = c < T ? (T - c + G - 1) / G : 0;    // tiles c, c + G, ... of the row-major order

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairMaxStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], 2 * kEpiWarps); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmY);
    }
    if (warp == 1) { __syncwarp(); tmem_alloc_pair(&ctl->tmem_base, kTmemCols); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised and both tensor memories allocated
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per CTA, its own halves)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            if (p.pdl) griddep_wait();                     // the codes come from the kernel before this one
            for (int i = 0; i < count && ok; ++i) {
                const int u = c + i * G;
                const int m2 = u / p.tiles_n, n_tile = u - m2 * p.tiles_n;
                const int m_tile = m2 * 2 + int(rank);     // this CTA's 128 rows
                int w0 = 0, h0 = 0, n0 = 0;
                if (CONV) {
                    const int tw = m_tile % p.tiles_w;
                    const int th = (m_tile / p.tiles_w) % p.tiles_h;
                    const int tn = m_tile / (p.tiles_w * p.tiles_h);
                    w0 = tw * p.bw; h0 = th * p.bh; n0 = tn * p.bn;      // past the last image: the load delivers zeros
                }
                for (int kb0 = 0; kb0 < num_kb; kb0 += KPS) {
                    if (!wait_pair(&ctl->empty[stage], phase ^ 1, ctl, p.dev_status, kStatusEmptyWait)) { ok = false; break; }
                    const uint32_t fbar = map_to_cta(&ctl->full[stage], 0);
                    if (rank == 0) mbar_expect_tx(&ctl->full[stage], 2u * uint32_t(KPS * kPairStageBytes));
#pragma unroll
                    for (int k = 0; k < KPS; ++k) {
                        const int kb = kb0 + k;
                        unsigned char* dst = sRing + (stage * KPS + k) * kPairStageBytes;
                        if (CONV) {
                            const int tap = kb / p.kb_per_tap, kc = kb - tap * p.kb_per_tap;
                            const int r = tap / p.S, s = tap - r * p.S;
                            tma_load_4d_pair(dst, &tmA, fbar, kc * kBK, w0 * p.stride + s - p.pad, h0 * p.stride + r - p.pad, n0);
                        } else {
                            tma_load_2d_pair(dst, &tmA, fbar, kb * kBK, m_tile * kBM);
                        }
                        tma_load_2d_pair(dst + kABytes, &tmB, fbar, kb * kBK, n_tile * kBN + int(rank) * 128);
                    }
                    if (++stage == nstages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            // A lone lane spends several cycles per instruction, and this lane's path per K block is what paces the
            // kernel: the operand descriptors advance by constants (a stage is 32 KB = 2048 descriptor units on, the
            // weights 1024 units behind the activations), and only the very first MMA of a tile overwrites.
            const uint32_t idesc = make_idesc_i8(256, kBN);
            const uint64_t desc0 = make_sw128_kmajor_desc(smem_u32(sRing));
            constexpr uint64_t kBlockUnits = kPairStageBytes >> 4, kStageUnits = KPS * kBlockUnits, kBUnits = kABytes >> 4;
            uint64_t a_desc = desc0;
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int i = 0; i < count && ok; ++i) {
                const int as = i & 1;
                if (!wait_pair(&ctl->tempty[as], (uint32_t(i >> 1) & 1u) ^ 1u, ctl, p.dev_status, kStatusAccumFree)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + uint32_t(as * kBN);
                uint32_t acc = 0;                          // 0 for the first MMA of the tile only
                for (int kb = 0; kb < num_kb; kb += KPS) {
                    if (!wait_pair(&ctl->full[stage], phase, ctl, p.dev_status, kStatusTmaWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t b_desc = a_desc + kBUnits;
                    mma_i8_pair(d_tmem, a_desc, b_desc, idesc, acc);
                    mma_i8_pair(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
                    mma_i8_pair(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
                    mma_i8_pair(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
                    if (KPS == 2) {
                        mma_i8_pair(d_tmem, a_desc + kBlockUnits, b_desc + kBlockUnits, idesc, 1u);
                        mma_i8_pair(d_tmem, a_desc + (kBlockUnits + 2), b_desc + (kBlockUnits + 2), idesc, 1u);
                        mma_i8_pair(d_tmem, a_desc + (kBlockUnits + 4), b_desc + (kBlockUnits + 4), idesc, 1u);
                        mma_i8_pair(d_tmem, a_desc + (kBlockUnits + 6), b_desc + (kBlockUnits + 6), idesc, 1u);
                    }
                    acc = 1u;
                    mma_commit_pair(&ctl->empty[stage]);
                    a_desc += kStageUnits;
                    if (++stage == nstages) { stage = 0; phase ^= 1; a_desc = desc0; }
                }
                if (!ok) break;
                mma_commit_pair(&ctl->tfull[as]);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2-9 of both CTAs)
        const int ew = warp - 2;
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int chalf = ew >> 2;                    // which half of the tile's columns this warp takes
        constexpr int NBUF = KPS == 2 ? 1 : 2;
        unsigned char* stg = sStage + ew * NBUF * kStagingBytes;
        float* prm_sw = sParam + ew * 2 * (kBN / 2);
        float* prm_b = prm_sw + kBN / 2;
        constexpr int cols_per_tile = LIMBS == 2 ? kBN / 2 : kBN;
        constexpr int cols_per_warp = cols_per_tile / 2;
        const int wc0 = chalf * cols_per_warp;
        const uint32_t tempty_leader[2] = {map_to_cta(&ctl->tempty[0], 0), map_to_cta(&ctl->tempty[1], 0)};
        int last_n = -1;
        bool ok = true;
        if (p.pdl) griddep_wait();                    // scale_a comes from the kernel before this one
        for (int i = 0; i < count && ok; ++i) {
            const int u = c + i * G;
            const int m2 = u / p.tiles_n, n_tile = u - m2 * p.tiles_n;
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
            const int64_t my_row = int64_t(m2) * 256 + int(rank) * 128 + q * 32 + lane;
            const float sa = p.sa_scalar ? __ldg(p.scale_a) : (my_row < p.M ? __ldg(p.scale_a + my_row) : 0.f);
            if (!wait_pair(&ctl->tfull[as], uint32_t(i >> 1) & 1u, ctl, p.dev_status, kStatusAccumWait)) { ok = false; break; }
            tc_fence_after();
            const float sa_eff = p.alpha * sa;
            const int row0 = m2 * 256 + int(rank) * 128 + q * 32;
            const uint32_t t_fast = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(as * kBN + wc0);
            epilogue_pair<LIMBS, 0, NBUF>(t_fast, stg, lane, prm_sw, prm_b, sa_eff, &tmY, col_base + wc0, row0, tempty_leader[as]);
        }
        if (lane == 0) bulk_wait_read_all();           // shared memory must outlive the copy engine's reads
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // neither CTA leaves while its peer may still signal its barriers or read its operands
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

// Issue-rate probe of the paired int8 MMA: back-to-back 256 x 256 x 32 MMAs of a 2-CTA cluster on resident tiles.
__global__ void __launch_bounds__(128, 1) mma_pair_probe_kernel(int iters, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t done_bar;
    __shared__ uint32_t tmem_slot;
    const uint32_t rank = cluster_rank();
    for (int i = threadIdx.x; i < (kABytes + kPairBBytes) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u;
    if (threadIdx.x == 0) { mbar_init(&done_bar, 1); fence_barrier_init(); }
    fence_proxy_async_smem();
    if (threadIdx.x >= 32 && threadIdx.x < 64) { __syncwarp(); tmem_alloc_pair(&tmem_slot, 256); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    if (threadIdx.x == 0) {
        if (rank == 0) {
            const uint32_t idesc = make_idesc_i8(256, kBN);
            const uint64_t a_desc = make_sw128_kmajor_desc(smem_u32(smem));
            const uint64_t b_desc = make_sw128_kmajor_desc(smem_u32(smem + kABytes));
            for (int i = 0; i < iters; ++i)
                mma_i8_pair(tmem_base, a_desc + uint64_t((i & 3) * 2), b_desc + uint64_t((i & 3) * 2), idesc, i != 0 ? 1u : 0u);
            mma_commit_pair(&done_bar);
        }
        mbar_wait(&done_bar, 0, dev_status, kStatusAccumWait);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (threadIdx.x >= 32 && threadIdx.x < 64) tmem_dealloc_pair(tmem_base, 256);
}

template <int LIMBS, int NKB, int KPS>
cudaError_t launch_pair(int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA, const CUtensorMap& tmB,
                        const CUtensorMap& tmY, const PairParams& p) {
    auto kern = qgemm_pair_kernel<LIMBS, NKB, KPS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid)); cfg.blockDim = dim3(unsigned(kPairThreads));
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    int na = 1;
    if (p.pdl) {
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        na = 2;
    }
    cfg.attrs = attr; cfg.numAttrs = unsigned(na);
    return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, p);
}

// How many 2-CTA clusters of this kernel the device runs at once (the SM count of a GPC need not be even).
template <int LIMBS, int NKB, int KPS>
int max_pairs(size_t smem) {
    static int cached[64][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return sm_count() / 2;
    int& slot = cached[dev][LIMBS - 1];
    if (slot == 0) {
        auto kern = qgemm_pair_kernel<LIMBS, NKB, KPS>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(unsigned(sm_count() / 2 * 2)); cfg.blockDim = dim3(unsigned(kPairThreads));
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0)
            n = sm_count() / 2 - 2;
        slot = n < sm_count() / 2 ? n : sm_count() / 2;
    }
    return slot;
}

template <int LIMBS, bool CONV, int KPS>
cudaError_t launch_pair_stream(int pairs_wanted, size_t smem, cudaStream_t st, const CUtensorMap& tmA, const CUtensorMap& tmB,
                               const CUtensorMap& tmY, const PairStreamParams& p) {
    auto kern = qgemm_pair_stream_kernel<LIMBS, CONV, KPS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(unsigned(kPairThreads));
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    // how many 2-CTA clusters the device runs at once (the SM count of a GPC need not be even), once per device
    static int cached[64] = {};
    int dev = 0, pairs_max = sm_count() / 2 - 2;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        if (cached[dev] == 0) {
            int n = 0;
            cfg.gridDim = dim3(unsigned(sm_count() / 2 * 2));
            if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0)
                cached[dev] = n < sm_count() / 2 ? n : sm_count() / 2;
            else
                cached[dev] = pairs_max;
        }
        pairs_max = cached[dev];
    }
    const int pairs = pairs_wanted < pairs_max ? pairs_wanted : pairs_max;
    cfg.gridDim = dim3(unsigned(2 * pairs));
    int na = 1;
    if (p.pdl) {
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        na = 2;
    }
    cfg.numAttrs = unsigned(na);
    return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, p);
}

bool pair_stream_stages(PairStreamParams& p, size_t& smem, int kps) {
    for (int stages = kPairMaxStages; stages >= 3; --stages) {
        const PairStreamLayout L = pair_stream_layout(stages, kps);
        if (L.total <= kSmemLimit) { p.stages = stages; smem = size_t(L.total); return true; }
    }
    return false;
}

}  // namespace

// Whether the streamed pair kernel covers a plain GEMM / a convolution planned by the one-CTA path (`g`: that plan).
bool pair_stream_covers_gemm(hq_container cont, const hq_weight_desc* desc, int64_t M, const void* y, hq_dtype ydt, int64_t ldy,
                             const int32_t* acc_out, bool combine_fast) {
    return cont == HQ_CODES_INT8 && desc->RS == 1 && desc->C_pad > int64_t(kResidentKb) * kBK && y != nullptr &&
           acc_out == nullptr && ydt == HQ_BF16 && aligned16(y) && (ldy * 2) % 16 == 0 && combine_fast && M >= 256;
}
bool pair_stream_covers_conv(hq_container cont, const gemm::GemmParams& g) {
    // one static scale, or one scale per output pixel of a 1x1 convolution (per_tap marks per-pixel scales under a window)
    return cont == HQ_CODES_INT8 && g.conv && g.tma_store && !g.per_tap && g.bw * g.bh * g.bn == kBM &&
           g.kb_per_tap * g.taps > kResidentKb && int64_t(g.tiles_m) >= 2;
}

hq_status launch_qgemm_pair_stream(const void* a_codes, int64_t M, int64_t K, int64_t lda, const hq_weight_desc* desc,
                                   const void* w_dev, const float* scale_a, int scale_a_is_scalar, const float* scale_w,
                                   const float* bias, float alpha, void* y, int64_t ldy, int32_t* dev_status, cudaStream_t st,
                                   bool after_quant) {
    PairStreamParams p{};
    p.M = M; p.N = int(desc->N); p.limbs = desc->limbs;
    p.num_kb = int(desc->C_pad / kBK);
    p.tiles_m2 = int((M + 255) / 256);
    p.tiles_n = int(desc->limbs == 2 ? desc->N_pad / 128 : (desc->N_pad + 255) / 256);
    p.scale_a = scale_a; p.sa_scalar = scale_a_is_scalar; p.scale_w = scale_w; p.bias = bias; p.alpha = alpha;
    p.pdl = after_quant ? 1 : 0; p.dev_status = dev_status;
    size_t smem = 0;
    if (!pair_stream_stages(p, smem, 1)) return HQ_ERR_UNSUPPORTED;    // two K blocks per stage measured 2 % slower here
    CUtensorMap tmA, tmB, tmY;
    if (!encode_2d(&tmA, a_codes, uint64_t(K), uint64_t(M), uint64_t(lda), kBK, kBM, true)) return HQ_ERR_CUDA;
    const uint64_t Kp = uint64_t(desc->C_pad);
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, 128, true)) return HQ_ERR_CUDA;
    if (!encode_y(&tmY, y, uint64_t(desc->N), uint64_t(M), uint64_t(ldy))) return HQ_ERR_CUDA;
    const int tiles = p.tiles_m2 * p.tiles_n;
    cudaError_t e = desc->limbs == 2 ? launch_pair_stream<2, false, 1>(tiles, smem, st, tmA, tmB, tmY, p)
                                     : launch_pair_stream<1, false, 1>(tiles, smem, st, tmA, tmB, tmY, p);
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

// The convolution the one-CTA path has planned in `g` (tile geometry, epilogue parameters) on pairs of SMs; tmA and tmY are
// that plan's tensor maps (the activation boxes are the same 128 pixels), the weight map is rebuilt with 128-row boxes.
hq_status launch_qconv_pair(const gemm::GemmParams& g, const CUtensorMap& tmA, const CUtensorMap& tmY,
                            const hq_weight_desc* desc, const void* w_dev, cudaStream_t st) {
    PairStreamParams p{};
    p.M = int64_t(g.Nb) * g.Ho * g.Wo; p.N = g.N; p.limbs = g.limbs;
    p.num_kb = g.kb_per_tap * g.taps;
    p.tiles_m2 = (g.tiles_m + 1) / 2;
    p.tiles_n = g.tiles_n;
    p.scale_a = g.scale_a; p.sa_scalar = g.sa_scalar; p.scale_w = g.scale_w; p.bias = g.bias; p.alpha = g.alpha;
    p.pdl = g.pdl; p.dev_status = g.dev_status;
    p.kb_per_tap = g.kb_per_tap; p.S = g.S; p.stride = g.stride; p.pad = g.pad;
    p.bw = g.bw; p.bh = g.bh; p.bn = g.bn; p.tiles_w = g.tiles_w; p.tiles_h = g.tiles_h;
    size_t smem = 0;
    const int kps = p.num_kb % 2 == 0 ? 2 : 1;      // two K blocks per ring stage: 6 % faster on the 3x3 convolutions
    if (!pair_stream_stages(p, smem, kps)) return HQ_ERR_UNSUPPORTED;
    CUtensorMap tmB;
    const uint64_t Kp = uint64_t(desc->C_pad) * desc->RS;
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, 128, true)) return HQ_ERR_CUDA;
    const int tiles = p.tiles_m2 * p.tiles_n;
    cudaError_t e;
    if (kps == 2) e = desc->limbs == 2 ? launch_pair_stream<2, true, 2>(tiles, smem, st, tmA, tmB, tmY, p)
                                       : launch_pair_stream<1, true, 2>(tiles, smem, st, tmA, tmB, tmY, p);
    else e = desc->limbs == 2 ? launch_pair_stream<2, true, 1>(tiles, smem, st, tmA, tmB, tmY, p)
                              : launch_pair_stream<1, true, 1>(tiles, smem, st, tmA, tmB, tmY, p);
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

// Whether the pair kernel covers a problem (see the top of this file); the caller has validated the arguments.
bool pair_kernel_covers(hq_container cont, const hq_weight_desc* desc, int64_t M, const void* y, hq_dtype ydt, int64_t ldy,
                        const int32_t* acc_out, bool combine_fast) {
    return cont == HQ_CODES_INT8 && desc->RS == 1 && desc->C_pad <= int64_t(kResidentKb) * kBK && y != nullptr &&
           acc_out == nullptr && ydt == HQ_BF16 && aligned16(y) && (ldy * 2) % 16 == 0 && combine_fast && M >= 256;
}

// Where the pair kernel is also the faster one: two-limb weights at K_pad = 512 (the epilogue's share of a tile is
// smallest there) on problems with at least one 256-row tile per SM.  With one limb or at K_pad = 256 a tile has as much
// epilogue as MMA work and the shape sweep measured the one-CTA kernel level or up to 15 % faster.
bool pair_kernel_pays(const hq_weight_desc* desc, int64_t M) {
    const int num_kb = int(desc->C_pad / kBK);
    const int64_t tiles = ((M + 255) / 256) * (desc->N_pad / 128);
    return desc->limbs == 2 && num_kb == 4 && tiles >= int64_t(sm_count());
}

hq_status launch_qgemm_pair(const void* a_codes, int64_t M, int64_t K, int64_t lda, const hq_weight_desc* desc,
                            const void* w_dev, const float* scale_a, int scale_a_is_scalar, const float* scale_w,
                            const float* bias, float alpha, void* y, int64_t ldy, int32_t* dev_status, cudaStream_t st,
                            bool after_quant) {
    PairParams p{};
    p.M = M; p.N = int(desc->N); p.limbs = desc->limbs;
    p.num_kb = int(desc->C_pad / kBK);
    p.tiles_m2 = int((M + 255) / 256);
    p.tiles_n = int(desc->limbs == 2 ? desc->N_pad / 128 : (desc->N_pad + 255) / 256);
    p.scale_a = scale_a; p.sa_scalar = scale_a_is_scalar; p.scale_w = scale_w; p.bias = bias; p.alpha = alpha;
    p.pdl = after_quant ? 1 : 0; p.dev_status = dev_status;
    const bool whole = p.num_kb == 4 || p.num_kb == 2;     // two K blocks per ring stage (see the kernel)
    size_t smem = 0;
    for (int stages = kPairMaxStages; stages >= 2; --stages) {
        const PairLayout L = pair_layout(p.num_kb, stages, whole ? 2 : 1);
        if (L.total <= kSmemLimit) { p.stages = stages; smem = size_t(L.total); break; }
    }
    if (smem == 0) return HQ_ERR_UNSUPPORTED;
    CUtensorMap tmA, tmB, tmY;
    if (!encode_2d(&tmA, a_codes, uint64_t(K), uint64_t(M), uint64_t(lda), kBK, kBM, true)) return HQ_ERR_CUDA;
    const uint64_t Kp = uint64_t(desc->C_pad);
    if (!encode_2d(&tmB, w_dev, Kp, uint64_t(desc->N_pad) * desc->limbs, Kp, kBK, 128, true)) return HQ_ERR_CUDA;
    if (!encode_y(&tmY, y, uint64_t(desc->N), uint64_t(M), uint64_t(ldy))) return HQ_ERR_CUDA;
    const int tiles = p.tiles_m2 * p.tiles_n;
    const int nkb = whole ? p.num_kb : 0;
    const bool two = desc->limbs == 2;
    const int pairs_max = nkb == 4 ? (two ? max_pairs<2, 4, 2>(smem) : max_pairs<1, 4, 2>(smem))
                        : nkb == 2 ? (two ? max_pairs<2, 2, 2>(smem) : max_pairs<1, 2, 2>(smem))
                                   : (two ? max_pairs<2, 0, 1>(smem) : max_pairs<1, 0, 1>(smem));
    const int pairs = tiles < pairs_max ? tiles : pairs_max;
    const int grid = 2 * pairs;
    cudaError_t e;
#define HQ_PAIR_GO(L, N, K) launch_pair<L, N, K>(grid, smem, st, tmA, tmB, tmY, p)
    if (nkb == 4) e = two ? HQ_PAIR_GO(2, 4, 2) : HQ_PAIR_GO(1, 4, 2);
    else if (nkb == 2) e = two ? HQ_PAIR_GO(2, 2, 2) : HQ_PAIR_GO(1, 2, 2);
    else e = two ? HQ_PAIR_GO(2, 0, 1) : HQ_PAIR_GO(1, 0, 1);
#undef HQ_PAIR_GO
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

}  // namespace hq

extern "C" hq_status hq_mma_i8_probe_pair(int pairs, int iters, int32_t* dev_status, void* stream) {
    using namespace hq;
    if (pairs <= 0 || iters <= 0) return HQ_ERR_INVALID_ARG;
    const size_t smem = 1024 + hq::gemm::kABytes + kPairBBytes;
    HQ_CUDA_OK(cudaFuncSetAttribute(mma_pair_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(2 * pairs)); cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem; cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, mma_pair_probe_kernel, iters, dev_status) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
