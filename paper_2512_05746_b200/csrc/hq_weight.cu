// Offline weight side (host code): Eq. 3 per output channel, then one of
//   PLAIN   B = Q(W)
//   FOLDED  B = H_raw * Q(W)   -- the inner product of Eq. 12 / Eq. 14 kept in exact integers, computed with
//                                 integer butterflies over each block of input channels
//   DOUBLE  B = Q(H^T W)       -- Double-Hadamard weights (H orthonormal)
// and the byte layout the tensor-core kernels consume:
//   rows   128 output channels per group; with two limbs a group is 128 "hi" rows followed by 128 "lo" rows
//          (B = 256*hi + lo, lo in [-128,127]), so one 256-row operand tile carries both limbs of 128 channels;
//   K axis tap-major, each tap padded with zeros to a multiple of 128 channels; for the NIBBLE activation
//          container every 8 consecutive channels are stored in the order 0,2,4,6,1,3,5,7, which is the order
//          the in-kernel nibble unpack produces for the activation operand.
#include <cmath>
#include <cstring>
#include <vector>

#include "hq_common.cuh"

namespace hq {
namespace {

constexpr int kTileK = 128;
constexpr int kTileN = 128;

int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

int limbs_for(int w_bits, int had_block, hq_weight_mode mode) {
    if (mode == HQ_W_PLAIN_A2) return 2;
    if (mode != HQ_W_FOLDED || had_block <= 1) return 1;
    return (int64_t(had_block) << (w_bits - 1)) > 128 ? 2 : 1;
}

template <typename T>
void fwht_inplace(T* v, int n) {
    for (int h = 1; h < n; h <<= 1)
        for (int s = 0; s < n; s += 2 * h)
            for (int j = s; j < s + h; ++j) {
                const T a = v[j], b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
}

void quantize_channel(const double* w, int64_t count, int w_bits, int32_t* out, float* scale) {
    const int qmax = kQmax(w_bits), qmin = kQmin(w_bits);
    double amax = 0.0;
    for (int64_t i = 0; i < count; ++i) amax = std::fmax(amax, std::fabs(w[i]));
    float s = amax > 0.0 ? float(amax / double(qmax)) : 1.0f;
    if (!(s > 0.0f)) s = 1.0f;
    *scale = s;
    for (int64_t i = 0; i < count; ++i) {
        double c = std::nearbyint(w[i] / double(s));
        c = std::fmin(std::fmax(c, double(qmin)), double(qmax));
        out[i] = int32_t(c);
    }
}

}  // namespace
}  // namespace hq

extern "C" int64_t hq_weight_blob_bytes(int64_t N, int32_t RS, int64_t C, int32_t w_bits, int32_t had_block,
                                        hq_weight_mode mode) {
    if (N <= 0 || RS <= 0 || C <= 0) return 0;
    const int limbs = hq::limbs_for(w_bits, had_block, mode);
    const int64_t Ck = mode == HQ_W_PLAIN_A2 ? 2 * C : C;          // channels per tap along K
    return hq::round_up(N, hq::kTileN) * limbs * RS * hq::round_up(Ck, hq::kTileK);
}

extern "C" hq_status hq_weight_prepare(const float* w, int64_t N, int32_t RS, int64_t C, int32_t w_bits,
                                       int32_t had_block, hq_weight_mode mode, hq_container container, void* blob,
                                       int64_t blob_bytes, float* s_w, hq_weight_desc* desc) {
    using namespace hq;
    if (w == nullptr || blob == nullptr || s_w == nullptr || desc == nullptr) return HQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return HQ_ERR_INVALID_ARG;
    if (mode != HQ_W_PLAIN && mode != HQ_W_FOLDED && mode != HQ_W_DOUBLE && mode != HQ_W_PLAIN_A2) return HQ_ERR_INVALID_ARG;
    if (mode == HQ_W_PLAIN_A2 && container != HQ_CODES_INT8) return HQ_ERR_SHAPE;
    if (container != HQ_CODES_NIBBLE && container != HQ_CODES_INT8) return HQ_ERR_INVALID_ARG;
    if (N <= 0 || RS <= 0 || C <= 0) return HQ_ERR_SHAPE;
    const int n = had_block > 1 ? had_block : 1;
    if (n > 1 && (!is_pow2(n) || C % n != 0)) return HQ_ERR_SHAPE;
    if (container == HQ_CODES_NIBBLE && C % 8 != 0) return HQ_ERR_SHAPE;
    const int limbs = limbs_for(w_bits, had_block, mode);
    const bool a2 = mode == HQ_W_PLAIN_A2;
    const int64_t Ck = a2 ? 2 * C : C;                              // channels per tap along K
    const int64_t C_pad = round_up(Ck, kTileK), N_pad = round_up(N, kTileN);
    const int64_t Kp = int64_t(RS) * C_pad;
    const int64_t need = N_pad * limbs * Kp;
    if (blob_bytes < need) return HQ_ERR_WORKSPACE;

    const int64_t KK = int64_t(RS) * C;
    std::vector<double> row(KK);
    std::vector<int32_t> B(KK);
    int8_t* out = static_cast<int8_t*>(blob);
    std::memset(out, 0, size_t(need));
    int32_t max_abs = 0;

    for (int64_t o = 0; o < N; ++o) {
        for (int64_t i = 0; i < KK; ++i) row[i] = double(w[o * KK + i]);
        if (mode == HQ_W_DOUBLE && n > 1) {
            const double norm = std::exp2(-0.5 * double(ilog2(n)));
            for (int64_t b = 0; b < KK / n; ++b) {
                fwht_inplace(row.data() + b * n, n);
                for (int j = 0; j < n; ++j) row[b * n + j] *= norm;
            }
        }
        quantize_channel(row.data(), KK, w_bits, B.data(), &s_w[o]);
        if (mode == HQ_W_FOLDED && n > 1)
            for (int64_t b = 0; b < KK / n; ++b) fwht_inplace(B.data() + b * n, n);

        const int64_t grp = o / kTileN, within = o % kTileN;
        for (int t = 0; t < RS; ++t) {
            for (int64_t c = 0; c < Ck; ++c) {
                // two activation limbs: the channels of a tap are [hi(C) | lo(C)] and B = [256 Q(W) | Q(W)], whose limb
                // split below gives the "hi" rows [Q(W) | 0] and the "lo" rows [0 | Q(W)]
                const int32_t v = a2 ? (c < C ? 256 * B[t * C + c] : B[t * C + (c - C)]) : B[t * C + c];
                max_abs = std::max(max_abs, v < 0 ? -v : v);
                // position along K inside the tap
                int64_t pos = c;
                if (container == HQ_CODES_NIBBLE) {
                    // slot p of an 8-group holds channel {0,2,4,6,1,3,5,7}[p]; this is the inverse map
                    const int r = int(c & 7);
                    const int slot = (r & 1) ? 4 + (r >> 1) : (r >> 1);
                    pos = (c & ~int64_t(7)) + slot;
                }
                const int64_t k = int64_t(t) * C_pad + pos;
                if (limbs == 1) {
                    if (v < -128 || v > 127) return HQ_ERR_OVERFLOW_RISK;
                    out[(grp * kTileN + within) * Kp + k] = int8_t(v);
                } else {
                    const int32_t lo = ((v + 128) & 255) - 128;
                    const int32_t hi = (v - lo) / 256;
                    if (hi < -128 || hi > 127) return HQ_ERR_OVERFLOW_RISK;
                    out[(grp * 2 * kTileN + within) * Kp + k] = int8_t(hi);
                    out[(grp * 2 * kTileN + kTileN + within) * Kp + k] = int8_t(lo);
                }
            }
        }
    }
    desc->N = N; desc->C = Ck; desc->RS = RS; desc->w_bits = w_bits; desc->had_block = had_block;
    desc->mode = int32_t(mode); desc->limbs = limbs; desc->container = int32_t(container);
    desc->C_pad = C_pad; desc->N_pad = N_pad; desc->bytes = need; desc->max_abs_b = max_abs; desc->reserved = 0;
    return HQ_OK;
}

extern "C" float hq_alpha_for(const hq_weight_desc* desc) {
    if (desc == nullptr) return 1.0f;
    if (desc->mode == HQ_W_FOLDED && desc->had_block > 1)
        return float(std::exp2(-0.5 * double(hq::ilog2(desc->had_block))));
    return 1.0f;
}
