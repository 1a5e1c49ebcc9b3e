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
#include "hq_common.cuh"

namespace hq {
namespace {

constexpr int kQTile = 128;      // queries per CTA (tensor-memory lanes)
constexpr int kKeyBlock = 128;   // keys per step
constexpr int kAttnTmemCols = 256;
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
template <int DH>
__device__ __forceinline__ void fetch_tile(uint4 (&reg)[DH / 8], const __nv_bfloat16* src, int64_t pitch, int rows_valid, int tid) {
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
        const int f = tid + 128 * i;
        const int rg = f / DH, within = f - rg * DH;
        const int row = rg * 8 + (within & 7), v = within >> 3;
        reg[i] = make_uint4(0u, 0u, 0u, 0u);
        if (row < rows_valid) reg[i] = __ldg(reinterpret_cast<const uint4*>(src + int64_t(row) * pitch + v * 8));
    }
}
template <int DH>
__device__ __forceinline__ void put_tile(unsigned char* dst, const uint4 (&reg)[DH / 8], int tid) {
    constexpr int group_stride = (DH / 8) * 128;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
        const int f = tid + 128 * i;
        const int rg = f / DH, within = f - rg * DH;
        *reinterpret_cast<uint4*>(dst + rg * group_stride + (within >> 3) * 128 + (within & 7) * 16) = reg[i];
    }
}
template <int DH>
__device__ __forceinline__ void stage_tile(unsigned char* dst, const __nv_bfloat16* src, int64_t pitch, int rows_valid,
                                           int tid) {
    uint4 reg[DH / 8];
    fetch_tile<DH>(reg, src, pitch, rows_valid, tid);
    put_tile<DH>(dst, reg, tid);
}

template <int DH>
__global__ void __launch_bounds__(128) attention_kernel(const AttnParams p) {
    extern __shared__ __align__(128) unsigned char smem_attn[];
    constexpr int kTileBytes = kQTile * DH * 2;
    unsigned char* sQ = smem_attn;
    unsigned char* sK = sQ + kTileBytes;
    unsigned char* sV = sK + kTileBytes;
    unsigned char* sP = sV + kTileBytes;                       // 128 x 128 bf16
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int q0 = blockIdx.x * kQTile, head = blockIdx.y, n = blockIdx.z;
    const int L = p.L, C = p.C;
    const int64_t pitch = 3 * int64_t(C);
    const __nv_bfloat16* base = p.qkv + int64_t(n) * L * pitch + head * DH;

    if (tid == 0) { mbar_init(&bar, 1); fence_barrier_init(); }
    // the allocation is a warp-wide (.sync.aligned) instruction: it runs in a warp none of whose lanes took another path
    if (warp == 1) { __syncwarp(); tmem_alloc(&tmem_slot, kAttnTmemCols); tmem_relinquish(); }
    stage_tile<DH>(sQ, base + int64_t(q0) * pitch, pitch, L - q0 < kQTile ? L - q0 : kQTile, tid);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t t_s = tmem_base + (uint32_t(warp * 32) << 16);          // this warp's lanes, S at columns 0..127
    const uint32_t t_o = t_s + uint32_t(kKeyBlock);                        // O at columns 128..128+DH

    constexpr uint32_t kGroup = (DH / 8) * 128;                            // bytes of one 8-row group of a DH-wide tile
    const uint32_t idesc_s = make_idesc_bf16(kQTile, kKeyBlock, false);
    const uint32_t idesc_o = make_idesc_bf16(kQTile, DH, true);

    float m_run = -INFINITY, l_run = 0.f;
    uint32_t phase = 0;
    bool ok = true;
    const int nblocks = (L + kKeyBlock - 1) / kKeyBlock;
    // The next key block's K and V pieces are requested into registers while the current block's softmax runs (head
    // widths up to 64: 16 registers per operand), so that their latency is not on the block's critical path.
    constexpr bool PREFETCH = DH <= 64;
    uint4 kreg[DH / 8], vreg[DH / 8];
    if (PREFETCH) {
        fetch_tile<DH>(kreg, base + C, pitch, L < kKeyBlock ? L : kKeyBlock, tid);
        fetch_tile<DH>(vreg, base + 2 * C, pitch, L < kKeyBlock ? L : kKeyBlock, tid);
    }
    for (int j = 0; j < nblocks && ok; ++j) {
        const int k0 = j * kKeyBlock;
        const int kvalid = L - k0 < kKeyBlock ? L - k0 : kKeyBlock;
        if (PREFETCH) {
            put_tile<DH>(sK, kreg, tid);
            put_tile<DH>(sV, vreg, tid);
        } else {
            stage_tile<DH>(sK, base + C + int64_t(k0) * pitch, pitch, kvalid, tid);
            stage_tile<DH>(sV, base + 2 * C + int64_t(k0) * pitch, pitch, kvalid, tid);
        }
        fence_proxy_async_smem();
        __syncthreads();
        if (PREFETCH && j + 1 < nblocks) {
            const int k1 = k0 + kKeyBlock;
            const int kv1 = L - k1 < kKeyBlock ? L - k1 : kKeyBlock;
            fetch_tile<DH>(kreg, base + C + int64_t(k1) * pitch, pitch, kv1, tid);
            fetch_tile<DH>(vreg, base + 2 * C + int64_t(k1) * pitch, pitch, kv1, tid);
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

        // ---- row maximum of this block (the next 32 columns are requested while the current ones are reduced)
        const bool full = kvalid == kKeyBlock;
        float mx = -INFINITY;
        {
            uint32_t ra[32], rb[32];
            tmem_ld_32x32(t_s, ra);
#pragma unroll
            for (int c = 0; c < kKeyBlock / 32; ++c) {
                uint32_t (&cur)[32] = (c & 1) ? rb : ra;
                uint32_t (&nxt)[32] = (c & 1) ? ra : rb;
                tmem_ld_wait_32(cur);
                if (c + 1 < kKeyBlock / 32) tmem_ld_32x32(t_s + uint32_t((c + 1) * 32), nxt);
                if (full) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(cur[e]));
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e < kvalid) mx = fmaxf(mx, __uint_as_float(cur[e]));
                }
            }
        }
        const float m_new = fmaxf(m_run, mx);
        const float mc = m_new * p.scale_log2;
        const float alpha = ex2(m_run * p.scale_log2 - mc);              // 0 on the first block (m_run = -inf)
        // ---- P = exp2(c (S - m)), row sum, bf16 into shared memory (K-major: 16 key groups of 128 bytes per row group)
        float sum = 0.f;
        unsigned char* prow = sP + (tid >> 3) * 2048 + (tid & 7) * 16;
        {
            uint32_t ra[32], rb[32];
            tmem_ld_32x32(t_s, ra);
#pragma unroll
            for (int c = 0; c < kKeyBlock / 32; ++c) {
                uint32_t (&cur)[32] = (c & 1) ? rb : ra;
                uint32_t (&nxt)[32] = (c & 1) ? ra : rb;
                tmem_ld_wait_32(cur);
                if (c + 1 < kKeyBlock / 32) tmem_ld_32x32(t_s + uint32_t((c + 1) * 32), nxt);
                float pv[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float v = ex2(fmaf(__uint_as_float(cur[e]), p.scale_log2, -mc));
                    pv[e] = (full || c * 32 + e < kvalid) ? v : 0.f;
                    sum += pv[e];
                }
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    uint4 w;
                    w.x = pack_bf16(pv[8 * g + 0], pv[8 * g + 1]); w.y = pack_bf16(pv[8 * g + 2], pv[8 * g + 3]);
                    w.z = pack_bf16(pv[8 * g + 4], pv[8 * g + 5]); w.w = pack_bf16(pv[8 * g + 6], pv[8 * g + 7]);
                    *reinterpret_cast<uint4*>(prow + (c * 4 + g) * 128) = w;
                }
            }
        }
        l_run = fmaf(l_run, alpha, sum);
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
                // P: K-major, row groups 2048 bytes apart.  V: MN-major, key groups kGroup apart (lbo), dh groups 128 (sbo).
                const uint64_t a = make_desc_noswizzle(smem_u32(sP), 128, 2048);
                const uint64_t b = make_desc_noswizzle(smem_u32(sV), kGroup, 128);
#pragma unroll
                for (int k = 0; k < kKeyBlock / 16; ++k)
                    mma_bf16(tmem_base + uint32_t(kKeyBlock), a + uint64_t(k * 16), b + uint64_t(k * 2 * (kGroup >> 4)), idesc_o,
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
    if (warp == 1) tmem_dealloc(tmem_base, kAttnTmemCols);
}

template <int DH>
cudaError_t launch_attention(const AttnParams& p, int Nb, cudaStream_t st) {
    const size_t smem = size_t(3) * kQTile * DH * 2 + size_t(kQTile) * kKeyBlock * 2 + 128;
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
    if (Nb > 65535 || heads > 65535 || L > (1 << 24)) return HQ_ERR_UNSUPPORTED;
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
        case 64: e = launch_attention<64>(p, int(Nb), st); break;
        case 96: e = launch_attention<96>(p, int(Nb), st); break;
        case 128: e = launch_attention<128>(p, int(Nb), st); break;
        default: return HQ_ERR_UNSUPPORTED;      // head widths the tensor-core tile shapes here cover: 32, 48, 64, 96, 128
    }
    return e == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
