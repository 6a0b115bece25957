// Host-side representation of an encoded matrix (internal to the library).
//
// Layout ("lane-stream" IE-BME, H_L = 16, R_A = 2, C_A = 1, paper Sec. V-A with the in-tile
// order chosen for the sm_100a kernel):
//   * rows are cut into strips of 16 (after an optional row order); columns into segments of
//     K_L; one (strip, segment) pair is a tile ("item"), tile index = strip * n_segs + segment.
//   * a tile is decoded by one warp; lane l = 4*g + t owns, for every 32-column k-block kb of
//     the tile, the 8 columns 32*kb + 8*t + j (j = 0..7) of strip rows g and g+8 -- exactly
//     the A-fragment slots of that lane in an m16n8k32 integer MMA.
//   * union mask: bit j of the lane's mask byte for k-block kb is set iff W[g][k] or W[g+8][k]
//     is nonzero (one bit covers Q = 2 values, area 0 = strip rows 0..7, area 1 = rows 8..15).
//   * payload: one byte per set bit, in (kb, j) order: high nibble = W[g+8][k] (two's
//     complement), low nibble = W[g][k] + 8 (excess-8). A cleared bit stands for the byte 0x08.
//   * tile blob = mask matrix [K_L/128 rows][32 lanes] u32 (byte i of word w = k-block 4w+i)
//                 followed by the payload matrix [J rows][32 lanes] u32, J = the longest lane
//                 stream in words; shorter streams are zero padded. Word (j, l) of either
//                 matrix sits in shared-memory bank l: every decode load is conflict free.
//   * per-tile offsets: item_off[t] in units of 16 bytes, n_items + 1 entries.
//
// Folded variant (H_L = 16, R_A = 2, C_A = 2, Q = 4; K_L a multiple of 256): the tile's columns form two
// areas of K_L/2; a mask bit covers rows g, g+8 at column k of BOTH areas, i.e. the same slot of k-blocks kb
// and kb + K_L/64. The mask matrix has K_L/256 rows; a set bit owns one payload byte per area, at the same
// position of two streams whose 128-byte rows alternate in the payload matrix ([2J rows][32 lanes]).
// INT2 weights (w2, folded variant only): one stream; the byte of a set bit packs the bit's four 2-bit values,
// each + 2 -- bits 1:0 = W[g][k], 3:2 = W[g+8][k] of area 0, bits 5:4 and 7:6 the same of area 1; a cleared
// bit stands for 0xAA.
//
// Any other valid IE-BME format (other H_L, R_A, C_A, narrow tiles) is encoded on the host in the
// paper's own array layout (GenericArrays) for us_get_stats / us_decode; no kernel reads it.
#pragma once
#include <cstdint>
#include <vector>

#include "../../include/unionsparse.h"

namespace us {

// The paper's three arrays for an arbitrary (H_L, K_L, R_A, C_A) (Sec. V-A "Storage Arrays"): what
// a format without a kernel is encoded into, for us_get_stats / us_decode.
struct GenericArrays {
    int64_t n_lt = 0, words_per_lt = 0;
    std::vector<uint64_t> bitmaps;   // Union Bitmaps: row-major, leftmost column = LSB, 64-bit words
    std::vector<uint32_t> offsets;   // Union Value Offsets, in INT4 values, n_lt + 1 entries
    std::vector<uint8_t> values;     // Compressed Values: two per byte, even index in the low nibble
};

struct HostMatrix {
    int64_t M = 0, K = 0, Mp = 0, Kp = 0;
    us_format fmt{16, 1024, 2, 1};
    bool kernel_layout = true;   // false: generic arrays only (host-only formats)
    bool w2 = false;             // INT2 weights: one payload byte per union-mask bit of the (16, K_L, 2, 2) format
    GenericArrays gen;
    int32_t nkb = 0;        // k-blocks (32 columns) per tile
    int32_t mask_rows = 0;  // mask words per lane and tile: nkb / (4 * C_A)
    int64_t n_strips = 0, n_segs = 0, n_items = 0;
    std::vector<int32_t> row_order;   // Mp entries: original row at padded position, -1 = padding
    std::vector<uint32_t> item_off;   // n_items + 1, units of 16 bytes
    std::vector<uint8_t> blob;        // all tile blobs back to back
    std::vector<uint16_t> w_scale;    // M fp16 bit patterns (empty if none)
    int64_t nnz = 0, sum_P = 0, bytes_payload_padded = 0;
    uint32_t max_item_bytes = 0;
};

// Returns US_OK or an error; `out` is filled on success. `threads` <= 0 picks the core count.
us_status encode_host(const int8_t* W, int64_t M, int64_t K, const uint16_t* w_scale,
                      const us_format& fmt, uint32_t flags, int threads, HostMatrix* out);
void decode_host(const HostMatrix& h, int8_t* W_out);
void fill_stats(const HostMatrix& h, us_stats* st);

// Byte-balanced split of the processing order (K range of G segments, strip, segment) over
// `n_cta` persistent CTAs: CTA c processes positions [begin[c], begin[c+1]) (n_cta + 1 entries).
// max_local_strips = the most strips any CTA touches within one K range.
void make_schedule(const HostMatrix& h, int n_cta, int G, std::vector<uint32_t>* begin,
                   int* max_local_strips);

// Default K_L for a shape when the caller passes no format.
int32_t default_K_L(int64_t M, int64_t K, int n_sm);

}  // namespace us
