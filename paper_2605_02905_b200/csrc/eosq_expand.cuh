// Expansion of packed 2- and 3-bit codes to fp16 centroids with byte permutes, shared by the kernels
// that feed codes to the tensor cores.  lo_tab / hi_tab hold the low / high bytes of the fp16
// centroids (level k in byte k; eight levels take two words).
#pragma once

#include <cstdint>

namespace eosq {

__device__ __forceinline__ uint32_t code_prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Sixteen 2-bit codes (one word, coordinate j in bits 2j, 2j + 1) -> eight words of fp16 pairs in
// coordinate order.
__device__ __forceinline__ void expand16_2bit(uint32_t w, uint32_t lo_tab, uint32_t hi_tab, uint32_t *out) {
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        uint32_t t = (w >> (16 * part)) & 0xFFFFu;
        t = (t | (t << 8)) & 0x00FF00FFu;
        t = (t | (t << 4)) & 0x0F0F0F0Fu;
        t = (t | (t << 2)) & 0x33333333u;   // one nibble per code
#pragma unroll
        for (int quad = 0; quad < 2; ++quad) {
            const uint32_t sel = t >> (16 * quad);
            const uint32_t lows = code_prmt(lo_tab, 0u, sel), highs = code_prmt(hi_tab, 0u, sel);
            out[4 * part + 2 * quad] = code_prmt(lows, highs, 0x5140u);
            out[4 * part + 2 * quad + 1] = code_prmt(lows, highs, 0x7362u);
        }
    }
}

// Eight 3-bit codes (24 bits) -> one nibble per code.
__device__ __forceinline__ uint32_t spread3to4(uint32_t x) {
    uint32_t s = (x & 0x00000FFFu) | ((x & 0x00FFF000u) << 4);
    s = (s & 0x003F003Fu) | ((s & 0x0FC00FC0u) << 2);
    return (s & 0x07070707u) | ((s & 0x38383838u) << 1);
}

// Eight 3-bit codes (bits 0..23 of `field`) -> four words of fp16 pairs in coordinate order.
__device__ __forceinline__ void expand8_3bit(uint32_t field, uint32_t lo0, uint32_t lo1, uint32_t hi0, uint32_t hi1, uint32_t *out) {
    const uint32_t t = spread3to4(field);
#pragma unroll
    for (int quad = 0; quad < 2; ++quad) {
        const uint32_t sel = t >> (16 * quad);
        const uint32_t lows = code_prmt(lo0, lo1, sel), highs = code_prmt(hi0, hi1, sel);
        out[2 * quad] = code_prmt(lows, highs, 0x5140u);
        out[2 * quad + 1] = code_prmt(lows, highs, 0x7362u);
    }
}

// Sixteen codes of width BITS (2 or 3), the q-th group of sixteen in the packed words `cw` of a run
// of 64 codes -> eight words of fp16 pairs.  lo / hi: the centroid byte tables.
template <int BITS>
__device__ __forceinline__ void expand16_codes(const uint32_t *cw, int q, const uint32_t (&lo)[2], const uint32_t (&hi)[2], uint32_t *out) {
    if (BITS == 2) {
        expand16_2bit(cw[q], lo[0], hi[0], out);
    } else {
        // bits [48 q, 48 q + 48) of the stream: two fields of 24 bits
        uint32_t f0, f1;
        if ((q & 1) == 0) {
            const uint32_t w0 = cw[3 * (q >> 1)], w1 = cw[3 * (q >> 1) + 1];
            f0 = w0 & 0x00FFFFFFu;
            f1 = (w0 >> 24) | ((w1 & 0x0000FFFFu) << 8);
        } else {
            const uint32_t w1 = cw[3 * (q >> 1) + 1], w2 = cw[3 * (q >> 1) + 2];
            f0 = (w1 >> 16) | ((w2 & 0x000000FFu) << 16);
            f1 = w2 >> 8;
        }
        expand8_3bit(f0, lo[0], lo[1], hi[0], hi[1], out);
        expand8_3bit(f1, lo[0], lo[1], hi[0], hi[1], out + 4);
    }
}

}  // namespace eosq
