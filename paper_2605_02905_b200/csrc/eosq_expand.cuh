// Expansion of packed 1- to 4-bit codes to fp16 centroids with byte permutes, shared by the kernels
// that feed codes to the tensor cores.  lo_tab / hi_tab hold the low / high bytes of the fp16
// centroids (level k in byte k & 3 of word k >> 2).
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

// Eight 1-bit codes (bits 0..7) -> one nibble per code.
__device__ __forceinline__ uint32_t spread1to4(uint32_t x) {
    uint32_t s = (x | (x << 12)) & 0x000F000Fu;
    s = (s | (s << 6)) & 0x03030303u;
    return (s | (s << 3)) & 0x11111111u;
}

// Eight codes, one per nibble of `sel` (levels 0..7) -> four words of fp16 pairs in coordinate order.
__device__ __forceinline__ void expand8_nibbles(uint32_t sel, uint32_t lo0, uint32_t lo1, uint32_t hi0, uint32_t hi1, uint32_t *out) {
#pragma unroll
    for (int quad = 0; quad < 2; ++quad) {
        const uint32_t s4 = sel >> (16 * quad);
        const uint32_t lows = code_prmt(lo0, lo1, s4), highs = code_prmt(hi0, hi1, s4);
        out[2 * quad] = code_prmt(lows, highs, 0x5140u);
        out[2 * quad + 1] = code_prmt(lows, highs, 0x7362u);
    }
}

// Eight 4-bit codes (one word) -> four words of fp16 pairs: a byte permute selects among eight bytes, so
// levels 0-7 and 8-15 are looked up separately and a third permute, steered by bit 3 of every code, picks.
__device__ __forceinline__ void expand8_4bit(uint32_t w, const uint32_t (&lo)[4], const uint32_t (&hi)[4], uint32_t *out) {
#pragma unroll
    for (int quad = 0; quad < 2; ++quad) {
        const uint32_t s4 = (w >> (16 * quad)) & 0xFFFFu;
        const uint32_t idx = s4 & 0x7777u, pick = 0x3210u | ((s4 & 0x8888u) >> 1);   // byte i from the first (i) or the second (4 + i) lookup
        const uint32_t lows = code_prmt(code_prmt(lo[0], lo[1], idx), code_prmt(lo[2], lo[3], idx), pick);
        const uint32_t highs = code_prmt(code_prmt(hi[0], hi[1], idx), code_prmt(hi[2], hi[3], idx), pick);
        out[2 * quad] = code_prmt(lows, highs, 0x5140u);
        out[2 * quad + 1] = code_prmt(lows, highs, 0x7362u);
    }
}

// Sixteen codes of width BITS, the q-th group of sixteen in the packed words `cw` of a run of 64 codes
// -> eight words of fp16 pairs.  lo / hi: the centroid byte tables (level k in byte k & 3 of word k >> 2).
template <int BITS>
__device__ __forceinline__ void expand16_codes(const uint32_t *cw, int q, const uint32_t (&lo)[4], const uint32_t (&hi)[4], uint32_t *out) {
    if (BITS == 1) {
        const uint32_t f = cw[q >> 1] >> (16 * (q & 1));
        expand8_nibbles(spread1to4(f & 0xFFu), lo[0], lo[1], hi[0], hi[1], out);
        expand8_nibbles(spread1to4((f >> 8) & 0xFFu), lo[0], lo[1], hi[0], hi[1], out + 4);
    } else if (BITS == 2) {
        expand16_2bit(cw[q], lo[0], hi[0], out);
    } else if (BITS == 3) {
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
        expand8_nibbles(spread3to4(f0), lo[0], lo[1], hi[0], hi[1], out);
        expand8_nibbles(spread3to4(f1), lo[0], lo[1], hi[0], hi[1], out + 4);
    } else {
        expand8_4bit(cw[2 * q], lo, hi, out);
        expand8_4bit(cw[2 * q + 1], lo, hi, out + 4);
    }
}

}  // namespace eosq
