// Helpers of the token-wise quantizers: the rank of a sink position, and the walk over the fields of one 32-bit word
// of a packed tile in memory order (the layout kvsink.h documents under kvsink_cache).
#pragma once
#include "common.cuh"

namespace kvsink {

// Slot of position `pos` in the ascending list sink_pos[0..count), or -1.
__device__ __forceinline__ int find_slot(const int32_t *__restrict__ sink_pos, int count, int pos)
{
    int lo = 0, hi = count - 1;
    while (lo <= hi) {
        int mid = (lo + hi) >> 1;
        int v = sink_pos[mid];
        if (v == pos) return mid;
        if (v < pos) lo = mid + 1;
        else hi = mid - 1;
    }
    return -1;
}

// Matrix element (m, row, col) held in pair slot s, half e of `lane`.
__device__ __forceinline__ void slot_to_elem(int lane, int s, int e, int *m, int *row, int *col)
{
    const int g = lane >> 2, t = lane & 3, r = s & 3;
    *m = s >> 2;
    *row = g + 8 * (r & 1);
    *col = 2 * t + e + 8 * (r >> 1);
}

// Assemble one physical word of a tile; get(m,row,col) supplies the code of a matrix element and `word`
// indexes the tile's 32-bit words in memory order.
template <typename Get>
__device__ __forceinline__ uint32_t assemble_word(int bits, int D, int word, Get get)
{
    uint32_t out = 0;
    int lane, i, m, row, col;
    if (bits == 2 || bits == 4) {
        const int n = D * bits / 64, fields = 16 / bits;   // fields per half word: 8 or 4
        section_word_owner(n, word, &lane, &i);
        for (int k = 0; k < fields; ++k)
            for (int e = 0; e < 2; ++e) {
                slot_to_elem(lane, fields * i + k, e, &m, &row, &col);
                out |= (get(m, row, col) & ((1u << bits) - 1u)) << (16 * e + bits * k);
            }
    } else {
        const int nlo = D / 32, nhi = D / 64;
        if (word < 32 * nlo) {
            section_word_owner(nlo, word, &lane, &i);
            for (int k = 0; k < 8; ++k)
                for (int e = 0; e < 2; ++e) {
                    slot_to_elem(lane, 8 * i + k, e, &m, &row, &col);
                    out |= (get(m, row, col) & 3u) << (16 * e + 2 * k);
                }
        } else {
            int j;
            section_word_owner(nhi, word - 32 * nlo, &lane, &j);
            for (int w = 0; w < 2; ++w)
                for (int k = 0; k < 8; ++k)
                    for (int e = 0; e < 2; ++e) {
                        slot_to_elem(lane, 8 * (2 * j + w) + k, e, &m, &row, &col);
                        out |= ((get(m, row, col) >> 2) & 1u) << (16 * e + 4 * (k >> 1) + 2 * (1 - w) + (k & 1));
                    }
        }
    }
    return out;
}

// The same walk over a word's fields, for the insert path: get(m,row,col) returns the code, or a value >= 0x100 for an
// element that is not being written; *fieldmask receives the bits of the fields that are.
template <typename Get>
__device__ __forceinline__ uint32_t assemble_word_masked(int bits, int D, int word, Get get, uint32_t *fieldmask)
{
    uint32_t out = 0, msk = 0;
    int lane, i, m, row, col;
    auto put = [&](uint32_t v, uint32_t width_mask, int shift) {
        const bool on = v < 0x100u;
        out |= on ? (v & width_mask) << shift : 0u;
        msk |= on ? width_mask << shift : 0u;
    };
    if (bits == 2 || bits == 4) {
        const int n = D * bits / 64, fields = 16 / bits;
        section_word_owner(n, word, &lane, &i);
        for (int k = 0; k < fields; ++k)
            for (int e = 0; e < 2; ++e) {
                slot_to_elem(lane, fields * i + k, e, &m, &row, &col);
                put(get(m, row, col), (1u << bits) - 1u, 16 * e + bits * k);
            }
    } else {
        const int nlo = D / 32, nhi = D / 64;
        if (word < 32 * nlo) {
            section_word_owner(nlo, word, &lane, &i);
            for (int k = 0; k < 8; ++k)
                for (int e = 0; e < 2; ++e) {
                    slot_to_elem(lane, 8 * i + k, e, &m, &row, &col);
                    put(get(m, row, col), 3u, 16 * e + 2 * k);
                }
        } else {
            int j;
            section_word_owner(nhi, word - 32 * nlo, &lane, &j);
            for (int w = 0; w < 2; ++w)
                for (int k = 0; k < 8; ++k)
                    for (int e = 0; e < 2; ++e) {
                        slot_to_elem(lane, 8 * (2 * j + w) + k, e, &m, &row, &col);
                        const uint32_t v = get(m, row, col);
                        put(v < 0x100u ? v >> 2 : v, 1u, 16 * e + 4 * (k >> 1) + 2 * (1 - w) + (k & 1));
                    }
        }
    }
    *fieldmask = msk;
    return out;
}

}  // namespace kvsink
