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
//   gid     V2a: u8  [RB][SC][GH][32]  library id of channel rb*32+l for part h of super-chunk sc
//   gsm     V2a: half2 [RB][SC][GH][32] (scale, mid) of the same part
//           The format's group size G is 64, 128 or 256 weights.  A super-chunk holds GH = 2 groups at G = 64 and
//           one otherwise; a group of 256 spans two super-chunks and its metadata is stored with both (the
//           decode kernels then see one (id, scale, mid) per 128 weights, whatever G is above 64).
//   rowptr  int32 [rows_pad + 1]       clamped to [0, nnz]
//   hdr     256 bytes                  {int32 ell_slots, int32 0, int64 off_ell}: the two values of this layout that
//                                      depend on nnz, for launches over several blobs of one shape whose outlier
//                                      counts differ (everything before hdr is independent of nnz)
//   oent    u32 [nnz]                  column | fp16 value << 16, CSR order
//   ell     u32 [RB][C + 1][32]        transposed outlier slab of every row-block, C = ell_slots(nnz, rows) slots:
//                                      word [b][0][l]   = number of slots channel b*32+l uses (min(row length, C)),
//                                      word [b][1+j][l] = j-th outlier of that channel, or column 0 / value +0.
//                                      C comes from the descriptor alone (mean row length + 4 sigma + 8), so a slab's
//                                      address needs no pointer load.  Rows longer than C keep their remaining
//                                      entries in the CSR arrays only (the "spill").
#pragma once
#include <cstddef>
#include <cstdint>

namespace xfp {

constexpr int kRowsPerBlock = 32;
constexpr int kSuper = 128;

struct Layout {
    int mode, rows, cols, bits, L, E;
    int G, GH;   // group size of the format (64, 128, 256); groups per super-chunk (2 at G = 64, else 1)
    int RB, SC, rows_pad;
    long long nnz;
    size_t off_idx, off_cb, off_gid, off_gsm, off_rowptr, off_hdr, off_oent, off_ell, total;
    int ell_slots;  // C: slots per channel in the transposed outlier slabs (0 when nnz == 0)
};

inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

// Slots per channel of the transposed outlier slabs: mean row length m plus four binomial standard
// deviations plus 8; rows beyond it spill to the CSR arrays.
inline int ell_slots(long long nnz, int rows) {
    if (nnz <= 0) return 0;
    const long long m = (nnz + rows - 1) / rows;
    long long r = 1;
    while (r * r < m) ++r;  // ceil(sqrt(m))
    const long long c = m + 4 * r + 8;
    return (int)(c > 65535 ? 65535 : c);
}

inline Layout make_layout(int mode, int rows, int cols, int bits, int lib_size, long long nnz, int group_size = 128) {
    Layout l{};
    l.mode = mode; l.rows = rows; l.cols = cols; l.bits = bits; l.L = mode ? lib_size : 0; l.E = 1 << bits;
    l.G = group_size; l.GH = (mode && group_size == 64) ? 2 : 1;
    l.RB = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
    l.SC = cols / kSuper;
    l.rows_pad = l.RB * kRowsPerBlock;
    l.nnz = nnz;
    size_t o = 0;
    l.off_idx = o;    o = align256(o + (size_t)l.RB * l.SC * bits * 512);
    l.off_cb = o;     o = align256(o + (size_t)(mode ? l.L : l.rows_pad) * l.E * 2);
    l.off_gid = o;    o = align256(o + (mode ? (size_t)l.RB * l.SC * l.GH * 32 : 0));
    l.off_gsm = o;    o = align256(o + (mode ? (size_t)l.RB * l.SC * l.GH * 32 * 4 : 0));
    l.off_rowptr = o; o = align256(o + (size_t)(l.rows_pad + 1) * 4);
    l.off_hdr = o;    o = align256(o + 256);
    l.off_oent = o;   o = align256(o + (size_t)nnz * 4);
    l.ell_slots = ell_slots(nnz, rows);
    l.off_ell = o;    o = align256(o + (l.ell_slots ? (size_t)l.RB * (l.ell_slots + 1) * 32 * 4 : 0));
    l.total = o;
    return l;
}

}  // namespace xfp
