// Host-side packer / loader: logical bit-planes and coefficients <-> device blob.
// The blob stores Eq. 1's B_i (as 32-bit words along the input dimension, grouped in 16-byte
// units per 128-column block, plane and row) and C_i (binary16), see bpdq.h for the layout.
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "bpdq_internal.h"

namespace bpdq {

static thread_local char g_err[512] = "";

int set_error(int code, const char* fmt, ...) {
    if (code == BPDQ_OK) return code;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

bool shape_supported(int out, int in, int K, int group) {
    if (out <= 0 || in <= 0) return false;
    if (K < 1 || K > 4) return false;
    if (group != 64 && group != 128 && group != 256) return false;
    if (in % kBlockCols) return false;                // whole 128-column blocks; with g = 256 the last group may hold 128 columns
    if (out % 16) return false;
    return true;
}

}  // namespace bpdq

using namespace bpdq;

extern "C" const char* bpdq_last_error(void) { return g_err; }

extern "C" size_t bpdq_packed_bytes(int out, int in, int K, int group) {
    if (!shape_supported(out, in, K, group)) return 0;
    return planes_bytes(out, in, K) + coefs_bytes(out, in, K, group);
}

extern "C" int bpdq_pack(const uint8_t* bits, const uint16_t* coef, int out, int in, int K,
                         int group, void* blob) {
    if (!bits || !coef || !blob) return set_error(BPDQ_ERR_INVALID, "bpdq_pack: null pointer");
    if (!shape_supported(out, in, K, group))
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_pack: unsupported shape out=%d in=%d K=%d g=%d",
                         out, in, K, group);
    uint8_t* dst = static_cast<uint8_t*>(blob);
    const int64_t nblocks = in / kBlockCols, ngroups = (in + group - 1) / group;
    for (int i = 0; i < K; ++i) {
        for (int64_t r = 0; r < out; ++r) {
            const uint8_t* row = bits + ((int64_t)i * out + r) * in;
            for (int64_t b = 0; b < nblocks; ++b) {
                uint8_t* unit = dst + plane_unit_offset(b, i, r, K, out);
                uint8_t logical[16] = {0};                // logical byte L = 4*word + byte-in-word
                for (int c = 0; c < kBlockCols; ++c) {
                    const unsigned v = row[b * kBlockCols + c];
                    if (v > 1u)
                        return set_error(BPDQ_ERR_INVALID, "bpdq_pack: bit value %u at plane %d row %lld col %lld",
                                         v, i, (long long)r, (long long)(b * kBlockCols + c));
                    const int k = c >> 5, u = (c >> 3) & 3, j = c & 7;
                    const int bit = 4 * j + u;            // position inside word k
                    logical[4 * k + (bit >> 3)] |= (uint8_t)(v << (bit & 7));
                }
                for (int L = 0; L < 16; ++L) unit[(L - (int)(r & 15)) & 15] = logical[L];   // physical byte p holds logical byte (p + r) mod 16
            }
        }
    }
    uint8_t* cdst = dst + planes_bytes(out, in, K);
    for (int i = 0; i <= K; ++i)
        for (int64_t r = 0; r < out; ++r)
            for (int64_t G = 0; G < ngroups; ++G) {
                const uint16_t v = coef[((int64_t)i * out + r) * ngroups + G];
                std::memcpy(cdst + coef_offset(G, i, r, K, out), &v, 2);
            }
    return BPDQ_OK;
}

extern "C" int bpdq_unpack(const void* blob, int out, int in, int K, int group, uint8_t* bits,
                           uint16_t* coef) {
    if (!bits || !coef || !blob) return set_error(BPDQ_ERR_INVALID, "bpdq_unpack: null pointer");
    if (!shape_supported(out, in, K, group))
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_unpack: unsupported shape out=%d in=%d K=%d g=%d",
                         out, in, K, group);
    const uint8_t* src = static_cast<const uint8_t*>(blob);
    const int64_t nblocks = in / kBlockCols, ngroups = (in + group - 1) / group;
    for (int i = 0; i < K; ++i)
        for (int64_t r = 0; r < out; ++r) {
            uint8_t* row = bits + ((int64_t)i * out + r) * in;
            for (int64_t b = 0; b < nblocks; ++b) {
                const uint8_t* unit = src + plane_unit_offset(b, i, r, K, out);
                for (int c = 0; c < kBlockCols; ++c) {
                    const int k = c >> 5, u = (c >> 3) & 3, j = c & 7;
                    const int bit = 4 * j + u;
                    const int L = 4 * k + (bit >> 3);
                    row[b * kBlockCols + c] = (unit[(L - (int)(r & 15)) & 15] >> (bit & 7)) & 1u;
                }
            }
        }
    const uint8_t* csrc = src + planes_bytes(out, in, K);
    for (int i = 0; i <= K; ++i)
        for (int64_t r = 0; r < out; ++r)
            for (int64_t G = 0; G < ngroups; ++G) {
                uint16_t v;
                std::memcpy(&v, csrc + coef_offset(G, i, r, K, out), 2);
                coef[((int64_t)i * out + r) * ngroups + G] = v;
            }
    return BPDQ_OK;
}
