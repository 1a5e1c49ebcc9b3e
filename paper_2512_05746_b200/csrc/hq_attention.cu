// Self-attention core of the network's attention blocks (between the quantized QKV projection and the quantized output
// projection; not one of the paper's equations): per sample and head, out = softmax(q k^T / sqrt(dh)) v.
//
// One CTA of 128 threads takes 128 queries of one (sample, head) and walks the keys in blocks of 128:
//   S = Q K_j^T      tcgen05.mma kind::f16 (bf16 operands from shared memory, fp32 accumulator in tensor memory)
//   row softmax      thread t owns query row t = lane t of tensor memory: running maximum and sum (online softmax),
//                    P = exp2(c (S - m)) rounded to bf16 into shared memory (the sum runs over the unrounded values: the
//                    roundings of 128 weights average out), the output accumulator rescaled in tensor
//                    memory when the running maximum moved
//   O += P V_j       tcgen05.mma again, V read as an MN-major operand so that it needs no transpose
// and finally O / sum goes out as bf16.  Operands are staged by plain 16-byte loads into the unswizzled canonical
// layout of the tensor core (8 x 16-byte core matrices).  Several CTAs are resident per SM and overlap one another's
// load, tensor and softmax phases; every wait is bounded.
#include <cuda.h>

#include "hq_common.cuh"
#include "hq_fwht.cuh"

namespace hq {
// hq_gemm.cu: bf16 [rows][cols] with a row pitch, boxes of box_rows x 64 columns in the 128-byte swizzle
bool encode_2d_bf16_sw128(CUtensorMap* tm, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                          uint32_t box_rows);

namespace {

constexpr int kQTile = 128;      // queries per CTA (tensor-memory lanes)
constexpr int kKeyBlock = 64;    // keys per step: S (64 columns) and O (dh columns) fit 128 columns of tensor memory up to
                                 // dh = 64, and a CTA's tiles 48 KB of shared memory, so that four CTAs share an SM
__host__ __device__ constexpr int attn_tmem_cols(int dh) { return kKeyBlock + dh <= 128 ? 128 : 256; }
constexpr int32_t kStatusAttnWait = 0x600;

struct AttnParams {
    const __nv_bfloat16* qkv;    // [Nb * L][3 C]
    __nv_bfloat16* out;          // [Nb * L][C]
    int L, C, heads;
    float scale_log2;            // log2(e) / sqrt(dh)
    int32_t* dev_status;
};

// Shared-memory matrix descriptor without swizzle: 8 x 16-byte core matrices; `lbo` / `sbo` are the byte distances between
// core matrices along K and along M/N for a K-major operand, and along K and along N (groups of 8) for an MN-major one.
__device__ __forceinline__ uint64_t make_desc_noswizzle(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= uint64_t((smem_addr & 0x3FFFFu) >> 4);
    d |= uint64_t((lbo >> 4) & 0x3FFFu) << 16;
    d |= uint64_t((sbo >> 4) & 0x3FFFu) << 32;
    d |= uint64_t(1) << 46;
    return d;
}

// Instruction descriptor for kind::f16 with bf16 operands and an fp32 accumulator, tile M x N; B MN-major when asked.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | (uint32_t(N >> 3) << 17) |
           (uint32_t(M >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// Copies `rows_valid` rows (of 128) x DH bf16 from global memory (row pitch `pitch` elements) into the canonical
// core-matrix layout: the 16-byte piece (row, v) lands at (row / 8) * group_stride + v * 128 + (row % 8) * 16.  Rows beyond
// rows_valid are zero.  Consecutive lanes take consecutive rows of a group, so the shared-memory stores of a warp fall
// into four 128-byte runs.
template <int DH, int ROWS>
__device__ __forceinline__ void fetch_tile(uint4 (&reg)[ROWS * DH / 1024], const __nv_bfloat16* src, int64_t pitch, int rows_valid,
                                           int tid) {
    static_assert((ROWS * DH / 8) % 128 == 0, "the tile's 16-byte pieces are dealt to 128 threads");
#pragma unroll
    for (int i = 0; i < ROWS * DH / 1024; ++i) {
        const int f = tid + 128 * i;
        const int rg = f / DH, within = f - rg * DH;
        const int row = rg * 8 + (within & 7), v = within >> 3;
        reg[i] = make_uint4(0u, 0u, 0u, 0u);
        if (row < rows_valid) reg[i] = __ldg(reinterpret_cast<const uint4*>(src + int64_t(row) * pitch + v * 8));
    }
}
template <int DH, int ROWS>
__device__ __forceinline__ void put_tile(unsigned char* dst, const uint4 (&reg)[ROWS * DH / 1024], int tid) {
    constexpr int group_stride = (DH / 8) * 128;
#pragma unroll
    for (int i = 0; i < ROWS * DH / 1024; ++i) {
        const int f = tid + 128 * i;
        const int rg = f / DH, within = f - rg * DH;
        *reinterpret_cast<uint4*>(dst + rg * group_stride + (within >> 3) * 128 + (within & 7) * 16) = reg[i];
    }
}
template <int DH, int ROWS>
__device__ __forceinline__ void stage_tile(unsigned char* dst, const __nv_bfloat16* src, int64_t pitch, int rows_valid,
                                           int tid) {
    uint4 reg[ROWS * DH / 1024];
    fetch_tile<DH, ROWS>(reg, src, pitch, rows_valid, tid);
    put_tile<DH, ROWS>(dst, reg, tid);
}

template <int DH>
__global__ void __launch_bounds__(128, (DH <= 64 ? 4 : 2)) attention_kernel(const AttnParams p) {
    extern __shared__ __align__(128) unsigned char smem_attn[];
    constexpr int KB = kKeyBlock;
    constexpr int kQBytes = kQTile * DH * 2, kKVBytes = KB * DH * 2;
    constexpr int kTmemCols = attn_tmem_cols(DH);
    unsigned char* sQ = smem_attn;
    unsigned char* sK = sQ + kQBytes;
    unsigned char* sV = sK + kKVBytes;
    unsigned char* sP = sV + kKVBytes;                         // 128 x KB bf16
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int q0 = blockIdx.x * kQTile, head = blockIdx.y, n = blockIdx.z;
    const int L = p.L, C = p.C;
    const int64_t pitch = 3 * int64_t(C);
    const __nv_bfloat16* base = p.qkv + int64_t(n) * L * pitch + head * DH;

    if (tid == 0) { mbar_init(&bar, 1); fence_barrier_init(); }
    // the allocation is a warp-wide (.sync.aligned) instruction: it runs in a warp none of whose lanes took another path
    if (warp == 1) { __syncwarp(); tmem_alloc(&tmem_slot, kTmemCols); tmem_relinquish(); }
    stage_tile<DH, kQTile>(sQ, base + int64_t(q0) * pitch, pitch, L - q0 < kQTile ? L - q0 : kQTile, tid);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t t_s = tmem_base + (uint32_t(warp * 32) << 16);          // this warp's lanes, S at columns 0..KB-1
    const uint32_t t_o = t_s + uint32_t(KB);                               // O at columns KB..KB+DH-1

    constexpr uint32_t kGroup = (DH / 8) * 128;                            // bytes of one 8-row group of a DH-wide tile
    constexpr uint32_t kPGroup = (KB / 8) * 128;                           // bytes of one 8-row group of P
    const uint32_t idesc_s = make_idesc_bf16(kQTile, KB, false);
    const uint32_t idesc_o = make_idesc_bf16(kQTile, DH, true);

    float m_run = -INFINITY, l_run = 0.f;
    uint32_t phase = 0;
    bool ok = true;
    const int nblocks = (L + KB - 1) / KB;
    // The next key block's K and V pieces are requested into registers while the current block's softmax runs, so that
    // their latency is not on the block's critical path.
    constexpr int NR = KB * DH / 1024;
    uint4 kreg[NR], vreg[NR];
    fetch_tile<DH, KB>(kreg, base + C, pitch, L < KB ? L : KB, tid);
    fetch_tile<DH, KB>(vreg, base + 2 * C, pitch, L < KB ? L : KB, tid);
    for (int j = 0; j < nblocks && ok; ++j) {
        const int k0 = j * KB;
        const int kvalid = L - k0 < KB ? L - k0 : KB;
        put_tile<DH, KB>(sK, kreg, tid);
        put_tile<DH, KB>(sV, vreg, tid);
        fence_proxy_async_smem();
        __syncthreads();
        if (j + 1 < nblocks) {
            const int k1 = k0 + KB;
            const int kv1 = L - k1 < KB ? L - k1 : KB;
            fetch_tile<DH, KB>(kreg, base + C + int64_t(k1) * pitch, pitch, kv1, tid);
            fetch_tile<DH, KB>(vreg, base + 2 * C + int64_t(k1) * pitch, pitch, kv1, tid);
        }
        // One lane issues; its warp-mates wait for it at the warp barrier instead of polling beside it (a polling loop
        // on the other side of a divergent branch can keep the issuing lane from being scheduled).
        if (warp == 0) {
            if (tid == 0) {
                tc_fence_after();
                // K-major operands: core matrices of a row group are contiguous along K (lbo 128), groups kGroup apart
                const uint64_t a = make_desc_noswizzle(smem_u32(sQ), 128, kGroup);
                const uint64_t b = make_desc_noswizzle(smem_u32(sK), 128, kGroup);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)
                    mma_bf16(tmem_base, a + uint64_t(k * 16), b + uint64_t(k * 16), idesc_s, k != 0 ? 1u : 0u);
                mma_commit(&bar);
            }
            __syncwarp();
        }
        ok = mbar_wait(&bar, phase, p.dev_status, kStatusAttnWait);
        phase ^= 1;
        ok = __syncthreads_and(ok);
        if (!ok) break;
        tc_fence_after();

        // ---- the row's KB scores come into registers once: maximum, then P = exp2(c (S - m)), the row sum, and P as bf16
        // into shared memory (K-major: KB / 8 key groups of 128 bytes per row group)
        const bool full = kvalid == KB;
        uint32_t sreg[KB];
#pragma unroll
        for (int c = 0; c < KB / 32; ++c) tmem_ld_32x32(t_s + uint32_t(c * 32), *reinterpret_cast<uint32_t (*)[32]>(&sreg[32 * c]));
#pragma unroll
        for (int c = 0; c < KB / 32; ++c) tmem_ld_wait_32(*reinterpret_cast<uint32_t (*)[32]>(&sreg[32 * c]));
        if (!full) {
#pragma unroll
            for (int e = 0; e < KB; ++e)
                if (e >= kvalid) sreg[e] = 0xFF800000u;                   // -inf: no part in the maximum, weight 0
        }
        float mx = -INFINITY;
#pragma unroll
        for (int e = 0; e < KB; e += 2) mx = max3(mx, __uint_as_float(sreg[e]), __uint_as_float(sreg[e + 1]));
        const float m_new = fmaxf(m_run, mx);
        const float mc = m_new * p.scale_log2;
        const float alpha = ex2(m_run * p.scale_log2 - mc);              // 0 on the first block (m_run = -inf)
        f32x2 sum2 = pk2(0.f, 0.f);
        const f32x2 sc2 = pk2(p.scale_log2, p.scale_log2), nmc2 = pk2(-mc, -mc);
        unsigned char* prow = sP + (tid >> 3) * kPGroup + (tid & 7) * 16;
#pragma unroll
        for (int g = 0; g < KB / 8; ++g) {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                float z0, z1;
                upk2(fma2(pk2(__uint_as_float(sreg[8 * g + 2 * h]), __uint_as_float(sreg[8 * g + 2 * h + 1])), sc2, nmc2), z0, z1);
                const float p0 = ex2(z0), p1 = ex2(z1);
                sum2 = add2(sum2, pk2(p0, p1));
                w[h] = pack_bf16(p0, p1);
            }
            *reinterpret_cast<uint4*>(prow + g * 128) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        float sum_lo, sum_hi;
        upk2(sum2, sum_lo, sum_hi);
        l_run = fmaf(l_run, alpha, sum_lo + sum_hi);
        m_run = m_new;
        // ---- the output accumulator follows the running maximum (skipped when no row of the warp moved)
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
            for (int c = 0; c < DH / 16; ++c) {
                uint32_t r[16];
                tmem_ld_32x16(t_o + uint32_t(c * 16), r);
                tmem_ld_wait_16(r);
#pragma unroll
                for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st_32x16(t_o + uint32_t(c * 16), r);
            }
            tmem_st_wait();
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (warp == 0) {
            if (tid == 0) {
                tc_fence_after();
                // P: K-major, row groups kPGroup bytes apart.  V: MN-major, key groups kGroup apart (lbo), dh groups 128 (sbo).
                const uint64_t a = make_desc_noswizzle(smem_u32(sP), 128, kPGroup);
                const uint64_t b = make_desc_noswizzle(smem_u32(sV), kGroup, 128);
#pragma unroll
                for (int k = 0; k < KB / 16; ++k)
                    mma_bf16(tmem_base + uint32_t(KB), a + uint64_t(k * 16), b + uint64_t(k * 2 * (kGroup >> 4)), idesc_o,
                             (j | k) != 0 ? 1u : 0u);
                mma_commit(&bar);
            }
            __syncwarp();
        }
        ok = mbar_wait(&bar, phase, p.dev_status, kStatusAttnWait);
        phase ^= 1;
        ok = __syncthreads_and(ok);
        if (!ok) break;
        tc_fence_after();
    }

    if (ok) {
        // every lane takes part in the tensor-memory loads (warp-wide instructions); only existing rows are stored
        const bool row_ok = q0 + tid < L;
        const float inv = 1.0f / l_run;
        __nv_bfloat16* dst = p.out + (int64_t(n) * L + (row_ok ? q0 + tid : 0)) * C + head * DH;
#pragma unroll
        for (int c = 0; c < DH / 16; ++c) {
            uint32_t r[16];
            tmem_ld_32x16(t_o + uint32_t(c * 16), r);
            tmem_ld_wait_16(r);
            uint4 w0, w1;
            w0.x = pack_bf16(__uint_as_float(r[0]) * inv, __uint_as_float(r[1]) * inv);
            w0.y = pack_bf16(__uint_as_float(r[2]) * inv, __uint_as_float(r[3]) * inv);
            w0.z = pack_bf16(__uint_as_float(r[4]) * inv, __uint_as_float(r[5]) * inv);
            w0.w = pack_bf16(__uint_as_float(r[6]) * inv, __uint_as_float(r[7]) * inv);
            w1.x = pack_bf16(__uint_as_float(r[8]) * inv, __uint_as_float(r[9]) * inv);
            w1.y = pack_bf16(__uint_as_float(r[10]) * inv, __uint_as_float(r[11]) * inv);
            w1.z = pack_bf16(__uint_as_float(r[12]) * inv, __uint_as_float(r[13]) * inv);
            w1.w = pack_bf16(__uint_as_float(r[14]) * inv, __uint_as_float(r[15]) * inv);
            if (row_ok) {
                reinterpret_cast<uint4*>(dst + c * 16)[0] = w0;
                reinterpret_cast<uint4*>(dst + c * 16)[1] = w1;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ---- head widths of 64 and 128: operands by TMA -----------------------------------------------------------------
// Q, K and V tiles come in by bulk tensor loads in the 128-byte swizzle (rows of 64 head channels = 128 bytes; a width
// of 128 takes two such column halves per tile), issued by one thread as soon as the MMAs that read the buffer have
// completed: the next K block lands during the softmax, the next V block during the next S product, no registers or
// shared-memory stores are spent on staging, and a CTA needs 48 KB of shared memory and 128 columns of tensor memory at
// width 64, so that four share an SM.  Q and K are K-major operands (8-row groups 1024 bytes apart); V is read as an
// MN-major operand (8-key groups 1024 bytes apart, the two 64-channel halves one tile apart).
// The running maximum of a row moves only when a block's maximum exceeds it by more than 2^8 in the exponent: the
// weights then stay below 2^8 (exact in bf16's range), the normalisation by the row sum at the end is unchanged, and
// the read-modify-write of the output accumulator in tensor memory is almost never needed after the first block.
constexpr int32_t kStatusAttnTma = 0x601;

__device__ __forceinline__ uint64_t make_sw128_mnmajor_desc(uint32_t smem_addr, uint32_t atom_stride_bytes) {
    uint64_t d = 0;
    d |= uint64_t((smem_addr & 0x3FFFFu) >> 4);
    d |= uint64_t((atom_stride_bytes >> 4) & 0x3FFFu) << 16;   // between 64-element groups along N
    d |= uint64_t(1024 >> 4) << 32;                            // between 8-row groups along K
    d |= uint64_t(1) << 46;
    d |= uint64_t(2) << 61;
    return d;
}

template <int DH>
__global__ void __launch_bounds__(128, (DH <= 64 ? 4 : 2))
attention_tma_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV, const AttnParams p) {
    extern __shared__ __align__(1024) unsigned char smem_attn_tma[];
    constexpr int KB = kKeyBlock, NH = DH / 64;                // column halves per tile
    constexpr int kQHalf = kQTile * 128, kKVHalf = KB * 128;   // bytes of one 64-channel half of a tile
    constexpr int kTmemCols = attn_tmem_cols(DH);
    unsigned char* sQ = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_attn_tma) + 1023) & ~uintptr_t(1023));
    unsigned char* sK = sQ + NH * kQHalf;
    unsigned char* sV = sK + NH * kKVHalf;
    unsigned char* sP = sV + NH * kKVHalf;                     // 128 x KB bf16, unswizzled core matrices
    __shared__ uint64_t bar_mma, bar_q, bar_k, bar_v;
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int q0 = blockIdx.x * kQTile, head = blockIdx.y, n = blockIdx.z;
    const int L = p.L, C = p.C;
    const int row0 = n * L;                                    // the sample's first row of the [Nb L][3 C] matrix
    const int nblocks = (L + KB - 1) / KB;

    if (tid == 0) {
        mbar_init(&bar_mma, 1); mbar_init(&bar_q, 1); mbar_init(&bar_k, 1); mbar_init(&bar_v, 1);
        fence_barrier_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmKV);
    }
    if (warp == 1) { __syncwarp(); tmem_alloc(&tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    bool q_flying = false, k_flying = false, v_flying = false;  // thread 0: a load into the buffer is outstanding
    uint32_t k_par = 0, v_par = 0;                              // ... and the barrier phase it completes
    if (tid == 0) {
        mbar_expect_tx(&bar_q, NH * kQHalf);
#pragma unroll
        for (int h = 0; h < NH; ++h) tma_load_2d(sQ + h * kQHalf, &tmQ, &bar_q, head * DH + 64 * h, row0 + q0);
        mbar_expect_tx(&bar_k, NH * kKVHalf);
#pragma unroll
        for (int h = 0; h < NH; ++h) tma_load_2d(sK + h * kKVHalf, &tmKV, &bar_k, C + head * DH + 64 * h, row0);
        mbar_expect_tx(&bar_v, NH * kKVHalf);
#pragma unroll
        for (int h = 0; h < NH; ++h) tma_load_2d(sV + h * kKVHalf, &tmKV, &bar_v, 2 * C + head * DH + 64 * h, row0);
        q_flying = k_flying = v_flying = true;
    }
    const uint32_t tmem_base = tmem_slot;
    const uint32_t t_s = tmem_base + (uint32_t(warp * 32) << 16);
    const uint32_t t_o = t_s + uint32_t(KB);
    constexpr uint32_t kPGroup = (KB / 8) * 128;
    const uint32_t idesc_s = make_idesc_bf16(kQTile, KB, false);
    const uint32_t idesc_o = make_idesc_bf16(kQTile, DH, true);

    float m_run = -INFINITY, l_run = 0.f;
    uint32_t ph_mma = 0;
    bool ok = true;
    // S of block 0
    if (warp == 0) {
        if (tid == 0) {
            bool ready = mbar_wait(&bar_q, 0, p.dev_status, kStatusAttnTma);
            if (ready) q_flying = false;
            ready = ready && mbar_wait(&bar_k, 0, p.dev_status, kStatusAttnTma);
            if (ready) {
                k_flying = false;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < DH / 16; ++k) {
                    const uint64_t a = make_sw128_kmajor_desc(smem_u32(sQ + (k / 4) * kQHalf)) + uint64_t(2 * (k & 3));
                    const uint64_t b = make_sw128_kmajor_desc(smem_u32(sK + (k / 4) * kKVHalf)) + uint64_t(2 * (k & 3));
                    mma_bf16(tmem_base, a, b, idesc_s, k != 0 ? 1u : 0u);
                }
                mma_commit(&bar_mma);
            }
        }
        __syncwarp();
    }
    // Block j: wait for S(j) (and O += P V of block j - 1, issued in the same batch), refill the buffers those MMAs have
    // read, softmax from registers, then one batch of MMAs again: O += P(j) V(j) and S(j + 1) -- the S columns are free as
    // soon as every thread holds its row in registers, so the two products share one trip to the tensor core.
    for (int j = 0; j < nblocks && ok; ++j) {
        const int k0 = j * KB;
        const int kvalid = L - k0 < KB ? L - k0 : KB;
        ok = mbar_wait(&bar_mma, ph_mma, p.dev_status, kStatusAttnWait);
        ph_mma ^= 1;
        ok = __syncthreads_and(ok);
        if (!ok) break;
        tc_fence_after();
        if (tid == 0) {
            if (j + 1 < nblocks) {                             // the K buffer is free: the next block's keys
                mbar_expect_tx(&bar_k, NH * kKVHalf);
#pragma unroll
                for (int h = 0; h < NH; ++h)
                    tma_load_2d(sK + h * kKVHalf, &tmKV, &bar_k, C + head * DH + 64 * h, row0 + k0 + KB);
                k_flying = true;
                k_par = uint32_t(j + 1) & 1u;
            }
            if (j > 0) {                                       // the V buffer is free: this block's values
                mbar_expect_tx(&bar_v, NH * kKVHalf);
#pragma unroll
                for (int h = 0; h < NH; ++h)
                    tma_load_2d(sV + h * kKVHalf, &tmKV, &bar_v, 2 * C + head * DH + 64 * h, row0 + k0);
                v_flying = true;
                v_par = uint32_t(j) & 1u;
            }
        }
        // ---- the row's KB scores come into registers once: maximum, P = exp2(c (S - m)), row sum, P as bf16 to smem
        const bool full = kvalid == KB;
        uint32_t sreg[KB];
#pragma unroll
        for (int c = 0; c < KB / 32; ++c) tmem_ld_32x32(t_s + uint32_t(c * 32), *reinterpret_cast<uint32_t (*)[32]>(&sreg[32 * c]));
#pragma unroll
        for (int c = 0; c < KB / 32; ++c) tmem_ld_wait_32(*reinterpret_cast<uint32_t (*)[32]>(&sreg[32 * c]));
        if (!full) {
#pragma unroll
            for (int e = 0; e < KB; ++e)
                if (e >= kvalid) sreg[e] = 0xFF800000u;                   // -inf: no part in the maximum, weight 0
        }
        float mx = -INFINITY;
#pragma unroll
        for (int e = 0; e < KB; e += 2) mx = max3(mx, __uint_as_float(sreg[e]), __uint_as_float(sreg[e + 1]));
        const float m_new = (mx - m_run) * p.scale_log2 > 8.0f ? mx : m_run;     // first block: inf > 8
        const float mc = m_new * p.scale_log2;
        const float alpha = ex2(m_run * p.scale_log2 - mc);              // 1 when the maximum stays, 0 on the first block
        f32x2 sum2 = pk2(0.f, 0.f);
        const f32x2 sc2 = pk2(p.scale_log2, p.scale_log2), nmc2 = pk2(-mc, -mc);
        unsigned char* prow = sP + (tid >> 3) * kPGroup + (tid & 7) * 16;
#pragma unroll
        for (int g = 0; g < KB / 8; ++g) {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                float z0, z1;
                upk2(fma2(pk2(__uint_as_float(sreg[8 * g + 2 * h]), __uint_as_float(sreg[8 * g + 2 * h + 1])), sc2, nmc2), z0, z1);
                const float p0 = ex2(z0), p1 = ex2(z1);
                sum2 = add2(sum2, pk2(p0, p1));
                w[h] = pack_bf16(p0, p1);
            }
            *reinterpret_cast<uint4*>(prow + g * 128) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        float sum_lo, sum_hi;
        upk2(sum2, sum_lo, sum_hi);
        l_run = fmaf(l_run, alpha, sum_lo + sum_hi);
        m_run = m_new;
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
            for (int c = 0; c < DH / 16; ++c) {
                uint32_t r[16];
                tmem_ld_32x16(t_o + uint32_t(c * 16), r);
                tmem_ld_wait_16(r);
#pragma unroll
                for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st_32x16(t_o + uint32_t(c * 16), r);
            }
            tmem_st_wait();
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (warp == 0) {
            if (tid == 0) {
                bool ready = mbar_wait(&bar_v, uint32_t(j) & 1u, p.dev_status, kStatusAttnTma);
                if (ready) v_flying = false;
                if (ready && j + 1 < nblocks) {
                    ready = mbar_wait(&bar_k, uint32_t(j + 1) & 1u, p.dev_status, kStatusAttnTma);
                    if (ready) k_flying = false;
                }
                if (ready) {
                    tc_fence_after();
                    const uint64_t a = make_desc_noswizzle(smem_u32(sP), 128, kPGroup);
                    const uint64_t b = make_sw128_mnmajor_desc(smem_u32(sV), kKVHalf);
#pragma unroll
                    for (int k = 0; k < KB / 16; ++k)        // 16 keys on: two core-matrix columns of P, 16 rows of V
                        mma_bf16(tmem_base + uint32_t(KB), a + uint64_t(k * 16), b + uint64_t(k * 128), idesc_o,
                                 (j | k) != 0 ? 1u : 0u);
                    if (j + 1 < nblocks) {
#pragma unroll
                        for (int k = 0; k < DH / 16; ++k) {
                            const uint64_t qa = make_sw128_kmajor_desc(smem_u32(sQ + (k / 4) * kQHalf)) + uint64_t(2 * (k & 3));
                            const uint64_t kb = make_sw128_kmajor_desc(smem_u32(sK + (k / 4) * kKVHalf)) + uint64_t(2 * (k & 3));
                            mma_bf16(tmem_base, qa, kb, idesc_s, k != 0 ? 1u : 0u);
                        }
                    }
                    mma_commit(&bar_mma);
                }
            }
            __syncwarp();
        }
    }
    if (ok) {                                                  // the last O += P V
        ok = mbar_wait(&bar_mma, ph_mma, p.dev_status, kStatusAttnWait);
        ok = __syncthreads_and(ok);
        tc_fence_after();
    }
    if (!ok && tid == 0) {
        // a wait ran out: the loads still on their way must land before the CTA's shared memory is given up
        if (q_flying) mbar_wait(&bar_q, 0, nullptr, 0);
        if (k_flying) mbar_wait(&bar_k, k_par, nullptr, 0);
        if (v_flying) mbar_wait(&bar_v, v_par, nullptr, 0);
    }

    if (ok) {
        const bool row_ok = q0 + tid < L;
        const float inv = 1.0f / l_run;
        __nv_bfloat16* dst = p.out + (int64_t(n) * L + (row_ok ? q0 + tid : 0)) * C + head * DH;
#pragma unroll
        for (int c = 0; c < DH / 16; ++c) {
            uint32_t r[16];
            tmem_ld_32x16(t_o + uint32_t(c * 16), r);
            tmem_ld_wait_16(r);
            uint4 w0, w1;
            w0.x = pack_bf16(__uint_as_float(r[0]) * inv, __uint_as_float(r[1]) * inv);
            w0.y = pack_bf16(__uint_as_float(r[2]) * inv, __uint_as_float(r[3]) * inv);
            w0.z = pack_bf16(__uint_as_float(r[4]) * inv, __uint_as_float(r[5]) * inv);
            w0.w = pack_bf16(__uint_as_float(r[6]) * inv, __uint_as_float(r[7]) * inv);
            w1.x = pack_bf16(__uint_as_float(r[8]) * inv, __uint_as_float(r[9]) * inv);
            w1.y = pack_bf16(__uint_as_float(r[10]) * inv, __uint_as_float(r[11]) * inv);
            w1.z = pack_bf16(__uint_as_float(r[12]) * inv, __uint_as_float(r[13]) * inv);
            w1.w = pack_bf16(__uint_as_float(r[14]) * inv, __uint_as_float(r[15]) * inv);
            if (row_ok) {
                reinterpret_cast<uint4*>(dst + c * 16)[0] = w0;
                reinterpret_cast<uint4*>(dst + c * 16)[1] = w1;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

template <int DH>
hq_status launch_attention_tma(const AttnParams& p, int Nb, cudaStream_t st) {
    CUtensorMap tmQ, tmKV;
    const uint64_t rows = uint64_t(Nb) * p.L, cols = 3 * uint64_t(p.C);
    if (!encode_2d_bf16_sw128(&tmQ, p.qkv, cols, rows, cols * 2, kQTile)) return HQ_ERR_CUDA;
    if (!encode_2d_bf16_sw128(&tmKV, p.qkv, cols, rows, cols * 2, kKeyBlock)) return HQ_ERR_CUDA;
    const size_t smem = size_t(DH / 64) * (kQTile + 2 * kKeyBlock) * 128 + size_t(kQTile) * kKeyBlock * 2 + 1024;
    if (cudaFuncSetAttribute(attention_tma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
        return HQ_ERR_CUDA;
    const dim3 grid(unsigned((p.L + kQTile - 1) / kQTile), unsigned(p.heads), unsigned(Nb));
    attention_tma_kernel<DH><<<grid, 128, smem, st>>>(tmQ, tmKV, p);
    return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

template <int DH>
cudaError_t launch_attention(const AttnParams& p, int Nb, cudaStream_t st) {
    const size_t smem = size_t(kQTile + 2 * kKeyBlock) * DH * 2 + size_t(kQTile) * kKeyBlock * 2 + 128;
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    const dim3 grid(unsigned((p.L + kQTile - 1) / kQTile), unsigned(p.heads), unsigned(Nb));
    attention_kernel<DH><<<grid, 128, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace
}  // namespace hq

extern "C" hq_status hq_attention(const void* qkv, int64_t Nb, int64_t L, int64_t C, int heads, void* out,
                                  int32_t* dev_status, void* stream) {
    using namespace hq;
    if (Nb < 0 || L <= 0 || C <= 0 || heads <= 0 || C % heads != 0) return HQ_ERR_SHAPE;
    if (Nb == 0) return HQ_OK;
    if (qkv == nullptr || out == nullptr) return HQ_ERR_INVALID_ARG;
    if (!aligned16(qkv) || !aligned16(out) || C % 8 != 0) return HQ_ERR_ALIGNMENT;
    if (Nb > 65535 || heads > 65535 || L > (1 << 24) || Nb * L > 0x7fffffff) return HQ_ERR_UNSUPPORTED;
    const int dh = int(C / heads);
    AttnParams p{};
    p.qkv = static_cast<const __nv_bfloat16*>(qkv);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.L = int(L); p.C = int(C); p.heads = heads;
    p.scale_log2 = float(1.4426950408889634 / sqrt(double(dh)));
    p.dev_status = dev_status;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (dh) {
        case 32: e = launch_attention<32>(p, int(Nb), st); break;
        case 48: e = launch_attention<48>(p, int(Nb), st); break;
        case 64: return launch_attention_tma<64>(p, int(Nb), st);
        case 96: e = launch_attention<96>(p, int(Nb), st); break;
        case 128: return launch_attention_tma<128>(p, int(Nb), st);
        default: return HQ_ERR_UNSUPPORTED;      // head widths the tensor-core tile shapes here cover: 32, 48, 64, 96, 128
    }
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
