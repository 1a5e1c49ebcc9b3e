// Building blocks of the in-register fast Walsh-Hadamard transform + quantization shared by the stand-alone
// transform+quantize kernel and the fused linear kernel: two-wide fp32 arithmetic, butterfly stages, the shared-memory
// exchange between the two register phases, and rounding + packing of the codes.
#pragma once

#include "hq_common.cuh"

namespace hq {

constexpr float kMagic = 12582912.0f;            // 1.5 * 2^23: adding it rounds to an integer in the low mantissa bits
constexpr uint32_t kMagicBits = 0x4B400000u;

// ---- two-wide fp32 arithmetic (one instruction for a pair of values held in a 64-bit register) -----------------
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk2(float lo, float hi) { f32x2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void upk2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) { f32x2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) { f32x2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }

// The largest of three values in one instruction.
__device__ __forceinline__ float max3(float a, float b, float c) { float r; asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c)); return r; }

// Butterflies over pair-index bits: element distance 2*h for h = LO .. HI (pairs stay pairs).
template <int P, int LO, int HI>
__device__ __forceinline__ void butterflies_pairs(f32x2 (&v)[P]) {
#pragma unroll
    for (int h = LO; h <= HI; h <<= 1) {
#pragma unroll
        for (int i = 0; i < P; ++i) {
            if (!(i & h)) {
                const f32x2 a = v[i], b = v[i | h];
                v[i] = add2(a, b);
                v[i | h] = sub2(a, b);
            }
        }
    }
}
// The stage between the two values of each pair.
template <int P>
__device__ __forceinline__ void butterfly_within_pairs(f32x2 (&v)[P]) {
#pragma unroll
    for (int i = 0; i < P; ++i) {
        float a, b;
        upk2(v[i], a, b);
        v[i] = pk2(a + b, a - b);
    }
}

__host__ __device__ constexpr int ilog2_c(int v) { return v <= 1 ? 0 : 1 + ilog2_c(v >> 1); }

// Rounds E values held as pairs (ties to even, optional clamp) and packs them in register order into words: 8
// four-bit codes or 4 bytes per word.  Adding kMagic + bias leaves code + bias in the low mantissa bits.  The second
// value of every pair is rounded F times larger (F = 256 for bytes, 16 for four-bit codes): scaling the multiplier and
// the magic number by a power of two scales the sum exactly, so the code is the same, and it lands F units up.  Taking
// the scaled magic number off again (exact) and adding the first value (exact: the sum stays below 2^22 units) leaves
// both biased codes side by side in the low bits of one float, on the floating-point pipe; byte permutes then gather
// the fields of a word, and one XOR turns the biased fields into two's complement.
template <int E, bool INT8_OUT, bool CLAMP>
__device__ __forceinline__ void round_pack(const f32x2 (&v)[E / 2], float inv, int bits, uint32_t (&out)[INT8_OUT ? E / 4 : E / 8]) {
    constexpr float F = INT8_OUT ? 256.0f : 16.0f;
    const float bias = INT8_OUT ? 128.0f : 8.0f;
    const float mb = kMagic + bias;
    const float lo = mb + float(-(1 << (bits - 1))), hi = mb + float((1 << (bits - 1)) - 1);
    const f32x2 inv2 = pk2(inv, F * inv), mb2 = pk2(mb, F * mb);
    uint32_t u[E / 2];                                 // per pair: kMagicBits + (c0 + bias) + F (c1 + bias)
#pragma unroll
    for (int e = 0; e < E / 2; ++e) {
        float f0, f1;
        upk2(fma2(v[e], inv2, mb2), f0, f1);
        if (CLAMP) { f0 = fminf(fmaxf(f0, lo), hi); f1 = fminf(fmaxf(f1, F * lo), F * hi); }
        u[e] = __float_as_uint(f0 + (f1 - F * kMagic));
    }
    if (INT8_OUT) {
#pragma unroll
        for (int w = 0; w < E / 4; ++w) out[w] = __byte_perm(u[2 * w], u[2 * w + 1], 0x5410) ^ 0x80808080u;
    } else {
#pragma unroll
        for (int w = 0; w < E / 8; ++w)
            out[w] = __byte_perm(__byte_perm(u[4 * w], u[4 * w + 1], 0x0040), __byte_perm(u[4 * w + 2], u[4 * w + 3], 0x0040),
                                 0x5410) ^ 0x88888888u;
    }
}

// Exchange-buffer geometry for a Hadamard block of 2^KLOG channels owned by N / E threads holding E values each.
template <int KLOG, int E>
struct FwhtShape {
    static constexpr int N = 1 << KLOG;
    static constexpr int LE = ilog2_c(E);
    static constexpr int P = E / 2;                    // two-wide registers per thread
    static constexpr int TB = N / E;                   // threads per Hadamard block
    static constexpr int R = KLOG - LE;                // index bits left for the second register phase
    static constexpr bool PAIR = R >= LE - 1;
    static constexpr bool SHUF = R == LE;
    static constexpr int J = PAIR ? E / 2 : E / 4;     // float4 slots a second-phase thread (pair) walks
    static constexpr int S = ilog2_c(J);
    static constexpr int GS = N / 4 + (N / 4) / J;     // padded float4 slots of the exchange buffer per Hadamard block
    static_assert(R <= LE, "block too large for this thread shape");
    static_assert(TB % J == 0 || J % TB == 0, "exchange layout needs TB and J to divide one another");
};

// All KLOG butterfly stages of one Hadamard block.  On entry thread tb of the block holds the float4s {tb + TB i} of the
// block (coalesced load order) as pairs; phase A covers index bits {0, 1} and the top log2(E) - 2 bits in registers, the
// values make one trip through the block's exchange buffer `grp` (float4 slot f at f + f / J, conflict-free both ways),
// and phase B covers the remaining bits in registers (KLOG = 12: one lane exchange more).  On exit thread u holds the E
// contiguous channels E u .. (or, PAIR, the channel pairs {4 j, 4 j + 1} + 2 (u & 1) of a 2E-channel group).
// CTA_SYNC: the block's threads span more than one warp (or the caller needs a CTA-wide barrier here anyway).
template <int KLOG, int E, bool CTA_SYNC>
__device__ __forceinline__ void fwht_stages(f32x2 (&v)[E / 2], float4* grp, int tb) {
    using Sh = FwhtShape<KLOG, E>;
    constexpr int P = Sh::P, TB = Sh::TB, J = Sh::J, S = Sh::S, R = Sh::R;
    butterfly_within_pairs<P>(v);                      // index bit 0
    butterflies_pairs<P, 1, P / 2>(v);                 // index bit 1 and the top LE-2 bits
    {
        // slot f = tb + TB i sits at f + f / J; with TB and J dividing one another that is a per-thread base plus a
        // compile-time offset
        ulonglong2* wr = reinterpret_cast<ulonglong2*>(grp + tb + (tb >> S));
#pragma unroll
        for (int i = 0; i < E / 4; ++i) wr[TB * i + ((TB * i) >> S)] = make_ulonglong2(v[2 * i], v[2 * i + 1]);
    }
    if (CTA_SYNC) __syncthreads(); else __syncwarp();
    if (!Sh::PAIR) {
        const ulonglong2* rd = reinterpret_cast<const ulonglong2*>(grp + (J + 1) * tb);
#pragma unroll
        for (int j = 0; j < E / 4; ++j) {
            const ulonglong2 q = rd[j];
            v[2 * j] = q.x; v[2 * j + 1] = q.y;
        }
        butterflies_pairs<P, 2, (2 << R) / 2>(v);      // index bits 2 .. R+1 are pair-index bits 1 .. R
    } else {
        const f32x2* rd = reinterpret_cast<const f32x2*>(grp + (J + 1) * (tb >> 1)) + (tb & 1);
#pragma unroll
        for (int j = 0; j < P; ++j) v[j] = rd[2 * j];
        butterflies_pairs<P, 1, P / 2>(v);             // index bits 2 .. LE are pair-index bits 0 .. LE-2
        if (Sh::SHUF) {                                // index bit LE+1 lives in lane bit 1
            const float sgn = (tb & 2) ? -1.0f : 1.0f;
            const f32x2 sgn2 = pk2(sgn, sgn);
#pragma unroll
            for (int e = 0; e < P; ++e) {
                const f32x2 other = __shfl_xor_sync(0xffffffffu, v[e], 2);
                v[e] = fma2(sgn2, v[e], other);
            }
        }
    }
}

// Rounds and packs the E values a thread holds after fwht_stages into words of codes for the E contiguous channels
// E tb .. of the block (8 four-bit codes or 4 bytes per word).  In the PAIR layout the two threads of a group first
// exchange halves: w holds the codes of channel pairs {4j, 4j+1} (+2 for the odd thread); the even thread emits the first
// half of the group's bytes, the odd thread the second half, interleaved at pair granularity (1 byte or 2 bytes).
template <int KLOG, int E, bool INT8_OUT, bool CLAMP>
__device__ __forceinline__ void pack_codes(const f32x2 (&v)[E / 2], float inv, int bits, int tb,
                                           uint32_t (&w)[INT8_OUT ? E / 4 : E / 8]) {
    constexpr int NW = INT8_OUT ? E / 4 : E / 8;
    round_pack<E, INT8_OUT, CLAMP>(v, inv, bits, w);
    if (FwhtShape<KLOG, E>::PAIR) {
        constexpr int H = NW / 2;
        const bool odd = tb & 1;
        uint32_t o[NW];
#pragma unroll
        for (int i = 0; i < H; ++i) {
            const uint32_t send = odd ? w[i] : w[i + H];
            const uint32_t keep = odd ? w[i + H] : w[i];
            const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
            const uint32_t ev = odd ? recv : keep, od = odd ? keep : recv;
            o[2 * i + 0] = __byte_perm(ev, od, INT8_OUT ? 0x5410 : 0x5140);
            o[2 * i + 1] = __byte_perm(ev, od, INT8_OUT ? 0x7632 : 0x7362);
        }
#pragma unroll
        for (int i = 0; i < NW; ++i) w[i] = o[i];
    }
}

}  // namespace hq
