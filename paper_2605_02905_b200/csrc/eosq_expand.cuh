// Expansion of packed 2-bit codes to fp16 centroids with byte permutes, shared by the kernels that
// feed codes to the tensor cores.  lo_tab / hi_tab hold the low / high bytes of the four fp16
// centroids (level k in byte k).
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

}  // namespace eosq
