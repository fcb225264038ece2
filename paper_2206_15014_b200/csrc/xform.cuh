// Shared-memory operand construction for weights that are not already in the tensor core's form:
// widening of packed 4-bit codes to int8, placement of 1:4 / 2:8 / 1:8 codes into the 2-of-4 slots
// (with explicit zeros) that tcgen05.mma.sp reads, and scatter of 4:8 codes into a dense tile.
//
// Everything works on one weight row and one 128-wide k-block at a time (one thread = one row):
// the thread reads the row's packed codes and canonical metadata for the k-block from global
// memory, builds the 64 (sparse target) or 128 (dense target) operand bytes in registers and
// writes them into the swizzled K-major tile the MMA descriptors expect.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace nm {
namespace xf {

// Patterns handled here.  Sparse target (2-of-4 slots + hardware metadata): 0..6.  Dense target: 7..9.
enum Pattern : int {
    P24_4 = 0, P14_8 = 1, P14_4 = 2, P28_8 = 3, P28_4 = 4, P18_8 = 5, P18_4 = 6,
    PDENSE_4 = 7, P48_8 = 8, P48_4 = 9, PNONE = -1
};

__host__ __device__ inline int pattern_of(int n, int m, int bits) {
    if (n == m) return bits == 4 ? PDENSE_4 : PNONE;
    if (m == 4 && n == 2) return bits == 4 ? P24_4 : PNONE;
    if (m == 4 && n == 1) return bits == 8 ? P14_8 : P14_4;
    if (m == 8 && n == 2) return bits == 8 ? P28_8 : P28_4;
    if (m == 8 && n == 1) return bits == 8 ? P18_8 : P18_4;
    if (m == 8 && n == 4) return bits == 8 ? P48_8 : P48_4;
    return PNONE;
}
__host__ __device__ inline bool sparse_target(int pat) { return pat >= P24_4 && pat <= P18_4; }
// bytes of packed codes / canonical metadata of one row per 128-wide k-block
__host__ __device__ inline int code_bytes(int pat) {
    switch (pat) { case P24_4: case P14_8: case P28_8: return 32; case P14_4: case P28_4: case P18_8: return 16;
                   case P18_4: return 8; case PDENSE_4: case P48_8: return 64; case P48_4: return 32; default: return 0; }
}
__host__ __device__ inline int meta_bytes(int pat) {
    switch (pat) { case P24_4: case P28_8: case P28_4: return 16; case P14_8: case P14_4: case P18_8: case P18_4: return 8;
                   case P48_8: case P48_4: return 32; default: return 0; }
}

// ---- slot tables ------------------------------------------------------------------------------------
// One "unit" is 8 consecutive logical positions = two hardware chunks of four = one 32-bit word of
// four slot bytes.  Entry = byte-permute selector (low 16 bits; nibble 0/1 = first/second code of the
// unit, 4 = zero) | hardware metadata byte << 16 (low nibble = first chunk).
// A chunk that keeps a single code at position p stores it as (code, 0) with positions (p, 3), or as
// (0, code) with positions (0, 3) when p == 3; an empty chunk stores (0, 0) with positions (0, 1).
constexpr int kLut14 = 0, kLut18 = 16, kLut28 = 32, kLutWords = 288;

__device__ inline void single_chunk(unsigned code, unsigned pl, unsigned& s0, unsigned& s1, unsigned& nib) {
    if (pl == 3) { s0 = 4; s1 = code; nib = 0xC; } else { s0 = code; s1 = 4; nib = pl | 0xC; }
}
__device__ inline uint32_t lut_entry(int table, unsigned idx) {
    unsigned s[4] = {4, 4, 4, 4}, nib[2] = {0x4, 0x4};
    if (table == kLut14) {            // idx = p_a | p_b << 2 : one code per chunk
        single_chunk(0, idx & 3, s[0], s[1], nib[0]);
        single_chunk(1, (idx >> 2) & 3, s[2], s[3], nib[1]);
    } else if (table == kLut18) {     // idx = p (0..7): one code in the group of eight
        unsigned c = (idx >> 2) & 1;
        single_chunk(0, idx & 3, s[2 * c], s[2 * c + 1], nib[c]);
    } else {                          // idx = p0 | p1 << 4, p0 < p1: two codes in the group of eight
        unsigned p0 = idx & 7, p1 = (idx >> 4) & 7, c0 = p0 >> 2, c1 = p1 >> 2;
        if (c0 == c1) { s[2 * c0] = 0; s[2 * c0 + 1] = 1; nib[c0] = (p0 & 3) | ((p1 & 3) << 2); }
        else { single_chunk(0, p0 & 3, s[0], s[1], nib[0]); single_chunk(1, p1 & 3, s[2], s[3], nib[1]); }
    }
    return (s[0] | (s[1] << 4) | (s[2] << 8) | (s[3] << 12)) | ((nib[0] | (nib[1] << 4)) << 16);
}
__device__ inline void build_lut(uint32_t* lut, int tid, int nthreads) {
    for (int i = tid; i < kLutWords; i += nthreads)
        lut[i] = i < kLut18 ? lut_entry(kLut14, i) : (i < kLut28 ? lut_entry(kLut18, i - kLut18) : lut_entry(kLut28, i - kLut28));
}

// ---- 4-bit -> 8-bit -----------------------------------------------------------------------------------
// Eight two's-complement nibbles (element 2j in bits 3:0 of byte j, element 2j+1 in bits 7:4) to
// eight int8 in element order.
__device__ __forceinline__ void widen8(uint32_t w, uint32_t& lo, uint32_t& hi) {
    uint32_t e = w & 0x0F0F0F0Fu, o = (w >> 4) & 0x0F0F0F0Fu;
    e |= (e & 0x08080808u) * 0x1Eu;   // sign bit of the nibble copied into bits 7:4 (no carries between bytes)
    o |= (o & 0x08080808u) * 0x1Eu;
    lo = __byte_perm(e, o, 0x5140);   // e0 o0 e1 o1
    hi = __byte_perm(e, o, 0x7362);   // e2 o2 e3 o3
}

// Packed codes and canonical metadata of one row for one k-block, as loaded from global memory.
struct Raw {
    uint4 v[4];  // up to 64 bytes of codes
    uint4 m[2];  // up to 32 bytes of metadata
};

__device__ __forceinline__ uint4 ldg16(const uint8_t* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ uint2 ldg8(const uint8_t* p) { return __ldg(reinterpret_cast<const uint2*>(p)); }

__device__ __forceinline__ Raw load_raw(int pat, const uint8_t* vsrc, const uint8_t* msrc, bool ok) {
    Raw r;
#pragma unroll
    for (int i = 0; i < 4; ++i) r.v[i] = make_uint4(0, 0, 0, 0);
    r.m[0] = r.m[1] = make_uint4(0, 0, 0, 0);
    if (!ok) return r;
    const int cb = code_bytes(pat), mb = meta_bytes(pat);
    if (cb == 8) { uint2 t = ldg8(vsrc); r.v[0].x = t.x; r.v[0].y = t.y; }
    else {
        r.v[0] = ldg16(vsrc);
        if (cb >= 32) r.v[1] = ldg16(vsrc + 16);
        if (cb >= 64) { r.v[2] = ldg16(vsrc + 32); r.v[3] = ldg16(vsrc + 48); }
    }
    if (pat != P24_4 && mb) {
        if (mb == 8) { uint2 t = ldg8(msrc); r.m[0].x = t.x; r.m[0].y = t.y; }
        else { r.m[0] = ldg16(msrc); if (mb >= 32) r.m[1] = ldg16(msrc + 16); }
    }
    return r;
}

__device__ __forceinline__ uint32_t word_of(const uint4* a, int i) {
    const uint4 q = a[i >> 2];
    return (i & 3) == 0 ? q.x : ((i & 3) == 1 ? q.y : ((i & 3) == 2 ? q.z : q.w));
}

// Builds the operand words of one row: 16 words (sparse target) or 32 words (dense target).
template <bool SPARSE>
__device__ __forceinline__ void build_row(int pat, const Raw& r, const uint32_t* lut, uint32_t (&out)[SPARSE ? 16 : 32]) {
    if constexpr (SPARSE) {
        uint32_t cw[8];  // widened codes: 32 (1:4, 2:8) or 16 (1:8) int8
        const bool four_bit = pat == P24_4 || pat == P14_4 || pat == P28_4 || pat == P18_4;
        if (pat == P24_4) {       // 64 codes -> the 64 slot bytes, already in slot order
#pragma unroll
            for (int i = 0; i < 8; ++i) widen8(word_of(r.v, i), out[2 * i], out[2 * i + 1]);
            return;
        }
        if (four_bit) {
#pragma unroll
            for (int i = 0; i < 4; ++i) widen8(word_of(r.v, i), cw[2 * i], cw[2 * i + 1]);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) cw[i] = word_of(r.v, i);
        }
        if (pat == P18_8 || pat == P18_4) {   // one code (byte u) and one 4-bit field per unit
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const uint32_t idx = (word_of(r.m, u >> 3) >> ((u & 7) * 4)) & 0x7u;
                const uint32_t code = cw[u >> 2] >> ((u & 3) * 8);
                out[u] = __byte_perm(code, 0u, lut[kLut18 + idx] & 0xFFFFu);
            }
        } else if (pat == P14_8 || pat == P14_4) {  // two codes (halfword u) and two 2-bit fields per unit
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const uint32_t idx = (word_of(r.m, u >> 3) >> ((u & 7) * 4)) & 0xFu;
                const uint32_t code = cw[u >> 1] >> ((u & 1) * 16);
                out[u] = __byte_perm(code, 0u, lut[kLut14 + idx] & 0xFFFFu);
            }
        } else {                                // 2:8: two codes (halfword u) and two 4-bit fields per unit
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const uint32_t idx = (word_of(r.m, u >> 2) >> ((u & 3) * 8)) & 0x77u;
                const uint32_t code = cw[u >> 1] >> ((u & 1) * 16);
                out[u] = __byte_perm(code, 0u, lut[kLut28 + idx] & 0xFFFFu);
            }
        }
    } else {
        if (pat == PDENSE_4) {
#pragma unroll
            for (int i = 0; i < 16; ++i) widen8(word_of(r.v, i), out[2 * i], out[2 * i + 1]);
            return;
        }
        uint32_t cw[16];  // 64 codes: four per group of eight
        if (pat == P48_4) {
#pragma unroll
            for (int i = 0; i < 8; ++i) widen8(word_of(r.v, i), cw[2 * i], cw[2 * i + 1]);
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) cw[i] = word_of(r.v, i);
        }
#pragma unroll
        for (int g = 0; g < 16; ++g) {
            // selector nibble d of the 8-byte group = index of the code stored at position d, 4 = zero
            const uint32_t f = (word_of(r.m, g >> 1) >> ((g & 1) * 16)) & 0x7777u;
            uint32_t sel = 0x44444444u;
#pragma unroll
            for (int i = 0; i < 4; ++i) sel ^= (uint32_t)(4 ^ i) << (4 * ((f >> (4 * i)) & 7u));
            out[2 * g] = __byte_perm(cw[g], 0u, sel & 0xFFFFu);
            out[2 * g + 1] = __byte_perm(cw[g], 0u, sel >> 16);
        }
    }
}

// Writes one row of operand bytes into a K-major tile with 64-byte (sparse) or 128-byte (dense) rows and
// the matching hardware swizzle: 16-byte chunk c of row r lands at chunk c ^ ((r >> 1) & 3), resp. c ^ (r & 7).
template <bool SPARSE>
__device__ __forceinline__ void store_row(uint8_t* tile, int row, const uint32_t (&w)[SPARSE ? 16 : 32]) {
    constexpr int CH = SPARSE ? 4 : 8;
    uint8_t* base = tile + row * (CH * 16);
    const int x = SPARSE ? ((row >> 1) & 3) : (row & 7);
#pragma unroll
    for (int c = 0; c < CH; ++c)
        *reinterpret_cast<uint4*>(base + ((c ^ x) << 4)) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
}

// The 64 operand bytes of one row and one 128-wide k-block into a tile whose rows are 128 bytes wide (two k-blocks side by
// side: `half` says which) with the 128-byte swizzle: 16-byte chunk c of row r lands at chunk c ^ (r & 7).
__device__ __forceinline__ void store_half_row128(uint8_t* tile, int row, int half, const uint32_t (&w)[16]) {
    uint8_t* base = tile + row * 128;
    const int x = row & 7;
#pragma unroll
    for (int c = 0; c < 4; ++c)
        *reinterpret_cast<uint4*>(base + (((half * 4 + c) ^ x) << 4)) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
}

// Hardware metadata words (4 per k-block) of one row from its canonical metadata.
__device__ __forceinline__ uint4 hw_meta(int pat, const uint8_t* msrc, const uint32_t* lut) {
    if (pat == P24_4) return ldg16(msrc);
    uint32_t h[4] = {0, 0, 0, 0};
    if (pat == P28_8 || pat == P28_4) {
        const uint4 m = ldg16(msrc);
        const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
        for (int u = 0; u < 16; ++u) h[u >> 2] |= (lut[kLut28 + ((mw[u >> 2] >> ((u & 3) * 8)) & 0x77u)] >> 16) << ((u & 3) * 8);
    } else {
        const uint2 m = ldg8(msrc);
        const uint32_t mw[2] = {m.x, m.y};
        const int base = (pat == P14_8 || pat == P14_4) ? kLut14 : kLut18;
        const uint32_t mask = base == kLut14 ? 0xFu : 0x7u;
#pragma unroll
        for (int u = 0; u < 16; ++u) h[u >> 2] |= (lut[base + ((mw[u >> 3] >> ((u & 7) * 4)) & mask)] >> 16) << ((u & 3) * 8);
    }
    return make_uint4(h[0], h[1], h[2], h[3]);
}

}  // namespace xf
}  // namespace nm
