// Where a logical code lives inside a packed atom (16 rows x 128 k of one bit-width).
//
// The layout is "fragment native" for mma.sync m16n8k16 with the weights as the A operand: lane
// (gid = lane/4, tid4 = lane%4) of a warp owns rows gid and gid+8 of the atom and, in MMA step
// s (k in [16s, 16s+16)), the four consecutive k = 16s + 4*tid4 + {0,1,2,3}.  Its 64 codes are
// contiguous per lane so that one or two 16-byte shared-memory loads fetch them, and the fields
// of a 32-bit word are ordered so that ((w >> shift) & mask) | 0x64006400 is directly the fp16
// pair (1024 + code_even, 1024 + code_odd) of one A-fragment register:
//
//   A register ri = rowhalf + 2*h  holds (row gid + 8*rowhalf, k = 16s + 4*tid4 + 2*h + {0,1}).
//
//   4-bit: atom = 2 planes x [32 lanes x 16 B]; plane s/4, word s%4; nibble ri (even k) and
//          nibble ri+4 (odd k).
//   2-bit: atom = [32 lanes x 16 B]; word s/2; 2-bit field (s%2)*4 + ri (even k), +8 (odd k).
//   8-bit: atom = 4 planes x [32 lanes x 16 B]; plane s/2, word 2*(s%2) + h; byte 2*rowhalf + odd.
//   3-bit: the low two bits exactly as a 2-bit atom (512 B), followed by a 1-bit plane
//          [32 lanes x 8 B]: word s/4, bit R (even k) and R+16 (odd k), R = ((s/2)%2)*8 + (s%2)*4 + ri.
#pragma once
#include <stdint.h>

namespace dyn {

struct CodeLoc {
    int byte_off;  // byte offset of the 32-bit word inside the atom
    int shift;     // bit position of the field inside that word
    int width;     // field width
};

// r: row in atom (0..15), kk: k in chunk (0..127).  For 3-bit, part 0 = low two bits, part 1 = high bit.
__host__ __device__ inline CodeLoc code_loc(int bits, int r, int kk, int part) {
    const int gid = r & 7, rowhalf = r >> 3;
    const int s = kk >> 4, kq = kk & 15;
    const int tid4 = kq >> 2, h = (kq >> 1) & 1, odd = kq & 1;
    const int lane = gid * 4 + tid4;
    const int ri = rowhalf + 2 * h;
    CodeLoc L;
    if (bits == 4) {
        L.byte_off = (s >> 2) * 512 + lane * 16 + (s & 3) * 4;
        L.shift = 4 * (ri + 4 * odd);
        L.width = 4;
    } else if (bits == 8) {
        L.byte_off = (s >> 1) * 512 + lane * 16 + (2 * (s & 1) + h) * 4;
        L.shift = 8 * (2 * rowhalf + odd);
        L.width = 8;
    } else if (bits == 2 || (bits == 3 && part == 0)) {
        L.byte_off = lane * 16 + (s >> 1) * 4;
        L.shift = 2 * ((s & 1) * 4 + ri + 8 * odd);
        L.width = 2;
    } else {  // 3-bit, high bit plane
        L.byte_off = 512 + lane * 8 + (s >> 2) * 4;
        L.shift = ((s >> 1) & 1) * 8 + (s & 1) * 4 + ri + 16 * odd;
        L.width = 1;
    }
    return L;
}

}  // namespace dyn
