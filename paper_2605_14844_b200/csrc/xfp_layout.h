// Device layout of a packed XFP blob.  Everything is a function of the descriptor, so a blob
// carries no header and can be copied freely.
//
// Rows are cut into row-blocks of 32 (one warp lane per output channel) and K into super-chunks
// of 128 weights (= one V2a group).  Sections, each 256-byte aligned:
//
//   idx     for (row-block rb, super-chunk sc, vector v < N, lane l): one uint4.
//           The 128 indices of channel rb*32+l in super-chunk sc form a dense little-endian bit
//           stream of 128*N bits (index j at bits [j*N, j*N+N)); vector v holds bits
//           [128 v, 128 v + 128).  A warp-wide load of vector v is one contiguous 512-byte read.
//   cb      V2: fp16 [rows_pad][2^N] (padding rows zero);  V2a: fp16 [L][2^N]
//   gid     V2a: u8  [RB][SC][32]      library id of (channel rb*32+l, group sc)
//   gsm     V2a: half2 [RB][SC][32]    (scale, mid) of the same group
//   rowptr  int32 [rows_pad + 1]       clamped to [0, nnz]
//   oent    u32 [nnz]                  column | fp16 value << 16, CSR order
//   ellptr  int32 [RB + 1]             start of each row-block's transposed outlier slab, in entries
//   ell     u32 [ell_cap]              slab of row-block b: slot j of channel b*32+l at ellptr[b] + j*32 + l,
//                                      width W_b = min(longest row of the block, 2*ceil(nnz_b/32) + 8) slots,
//                                      unused slots hold column 0 / value +0.  Rows longer than W_b keep their
//                                      remaining entries in the CSR arrays only (the "spill").
#pragma once
#include <cstddef>
#include <cstdint>

namespace xfp {

constexpr int kRowsPerBlock = 32;
constexpr int kSuper = 128;

struct Layout {
    int mode, rows, cols, bits, L, E;
    int RB, SC, rows_pad;
    long long nnz;
    size_t off_idx, off_cb, off_gid, off_gsm, off_rowptr, off_oent, off_ellptr, off_ell, total;
    long long ell_cap;  // entries reserved for the transposed slabs (an upper bound from nnz and RB)
};

inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

inline Layout make_layout(int mode, int rows, int cols, int bits, int lib_size, long long nnz) {
    Layout l{};
    l.mode = mode; l.rows = rows; l.cols = cols; l.bits = bits; l.L = mode ? lib_size : 0; l.E = 1 << bits;
    l.RB = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
    l.SC = cols / kSuper;
    l.rows_pad = l.RB * kRowsPerBlock;
    l.nnz = nnz;
    size_t o = 0;
    l.off_idx = o;    o = align256(o + (size_t)l.RB * l.SC * bits * 512);
    l.off_cb = o;     o = align256(o + (size_t)(mode ? l.L : l.rows_pad) * l.E * 2);
    l.off_gid = o;    o = align256(o + (mode ? (size_t)l.RB * l.SC * 32 : 0));
    l.off_gsm = o;    o = align256(o + (mode ? (size_t)l.RB * l.SC * 32 * 4 : 0));
    l.off_rowptr = o; o = align256(o + (size_t)(l.rows_pad + 1) * 4);
    l.off_oent = o;   o = align256(o + (size_t)nnz * 4);
    l.ell_cap = nnz ? 2 * nnz + 320LL * l.RB : 0;
    l.off_ellptr = o; o = align256(o + (size_t)(l.RB + 1) * 4);
    l.off_ell = o;    o = align256(o + (size_t)l.ell_cap * 4);
    l.total = o;
    return l;
}

}  // namespace xfp
