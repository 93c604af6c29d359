// Index maps of the packed ternary layouts.  Every layout stores a code t as the
// 2-bit field e = t + 1, sixteen fields per 32-bit word, field f at bits 2f..2f+1.
// Each map answers: which (n, k) of W[N,K] does field f of destination word widx hold?
#pragma once
#include <stdint.h>

// Canonical layout: row-major [N][K4] bytes, byte j of row n holds k = 4j..4j+3.
__host__ __device__ __forceinline__ int a48_l0_code(const uint8_t* l0, int K4, int n, int k) {
    unsigned byte = l0[(size_t)n * K4 + (k >> 2)];
    return (int)((byte >> (2 * (k & 3))) & 3u) - 1;
}

// Tile-major layout for the tcgen05 prefill kernel.  A tile is 128 rows (n) by
// 128 channels (k) = 4 KB, tiles ordered [n-tile][k-block].  Inside a tile the
// 16-byte vector of (half h, lane r) sits at byte h*2048 + r*16, so that one
// warp-wide 128-bit load is contiguous.  Lane r is row n = 128*nt + r and also
// the TMEM lane the expanded row is written to.  Word wq = 4h + (word in vector)
// expands to TMEM columns c = 4*wq + q, q = 0..3, taken from bit offsets
// s_q = {0, 2, 16, 18}; byte j of that column (k = 128*kb + 4c + j) is the field
// at bit s_q + 4j.  (Two fields share a nibble, which is what a byte-permute
// lookup consumes: see expand_word in gemm_tcgen05.cu.)
struct GemmLayout {
    int Kp;
    __host__ __device__ void field_to_nk(size_t widx, int f, int& n, int& k) const {
        int kblocks = Kp / 128;
        size_t tile = widx / 1024;
        int wi = (int)(widx % 1024);
        int nt = (int)(tile / kblocks), kb = (int)(tile % kblocks);
        int h = wi / 512, r = (wi % 512) / 4, w4 = wi % 4;
        int wq = 4 * h + w4;
        int q = ((f >> 3) & 1) * 2 + (f & 1);
        int j = (f & 7) >> 1;
        int c = 4 * wq + q;
        n = nt * 128 + r;
        k = kb * 128 + 4 * c + j;
    }
};

// Fragment-major layout for the decode kernel (mma.sync m16n8k32 with the weights
// as the A operand).  A unit is 16 rows by 128 channels = 512 B, units ordered
// [n16-tile][k-chunk]; lane l of the warp owns the 16-byte vector at l*16.  With
// g = l/4 and tig = l%4, word j of the vector becomes A-fragment register a_j of
// four MMAs, one per 2-bit position i of every byte: masking with 0x03030303<<2i
// leaves, in byte b, the field of
//   n = 16*nt + g + 8*(j&1),   k = 128*kc + 32*i + 16*(j>>1) + 4*tig + b
// scaled by 4^i, which is the operand layout the MMA expects for rows g / g+8 and
// k positions 4*tig+b / 16+4*tig+b of a 32-wide k slice.
struct DecodeLayout {
    int Kp;
    __host__ __device__ void field_to_nk(size_t widx, int f, int& n, int& k) const {
        int kchunks = Kp / 128;
        int j = (int)(widx % 4);
        int lane = (int)((widx / 4) % 32);
        size_t unit = widx / 128;
        int nt = (int)(unit / kchunks), kc = (int)(unit % kchunks);
        int g = lane >> 2, tig = lane & 3;
        int b = f >> 2, i = f & 3;
        n = nt * 16 + g + 8 * (j & 1);
        k = kc * 128 + 32 * i + 16 * (j >> 1) + 4 * tig + b;
    }
};

// Channel-major layout for the zero-skipping batch-1 decode kernel: row k holds
// the codes of every output feature for input channel k, Np/16 words per row,
// field f of word j is n = 16j + f.
struct SparseLayout {
    int Np;
    __host__ __device__ void field_to_nk(size_t widx, int f, int& n, int& k) const {
        int wpr = Np / 16;
        k = (int)(widx / wpr);
        n = (int)(widx % wpr) * 16 + f;
    }
};
