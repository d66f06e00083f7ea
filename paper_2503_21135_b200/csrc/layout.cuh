// Where a logical code lives inside a packed atom (16 rows x 128 k of one bit-width), and the
// power-of-two scale the activations carry so that codes can be used where they lie.
//
// The layout is "fragment native" for mma.sync m16n8k16 with the weights as the A operand: lane
// (gid = lane/4, tid4 = lane%4) of a warp owns rows gid and gid+8 of the atom and, in MMA step
// s (k in [16s, 16s+16)), the four consecutive k = 16s + 4*tid4 + {0,1,2,3}.  A-fragment register
// ri = rowhalf + 2*h holds (row gid + 8*rowhalf, k = 16s + 4*tid4 + 2*h + {0,1}) as an fp16 pair.
//
// A code is NOT shifted down to bit 0 before use.  A field of width b at bit offset o (o + b <= 10)
// of a 16-bit half, masked in place, is the fp16 SUBNORMAL q * 2^(o-24); the matching activation is
// stored pre-multiplied by 2^(bias - o), so the product is q * x * 2^(bias-24) whatever o is, and one
// AND per register pair (plus one shift per 32-bit word to bring the upper fields below bit 10)
// replaces shift + mask + or.  The offset o of a k must not depend on the row (the B fragment is
// shared by all rows), so the two row halves live in different words:
//
//   2-bit: atom = [32 lanes x 16 B]; word jh*2 + rowhalf (jh = s/4, the 64-k half chunk);
//          field phi = 2*(s%4) + h at bits [2phi, 2phi+2) (even k) and +16 (odd k);
//          phi <= 4 used in place (o = 2phi), phi >= 5 after >> 10 (o = 2phi - 10).
//   3-bit: low two bits stored exactly as a 2-bit atom but used as phi <= 3 in place (o = 2phi),
//          phi >= 4 after >> 8 (o = 2phi - 8); then a 1-bit plane [32 lanes x 8 B], word = rowhalf:
//          the high bit of field (jh, phi) must land on bit o+2 (even k) / o+18 (odd k) after a
//          rotation by rot = {0, 1, 8, 9}[2*jh + phi/4], i.e. it is stored at bit (o + 2 + 16*odd + rot) % 32.
//   4-bit: atom = 2 planes (= half chunks) x [32 lanes x 16 B]; word rowhalf*2 + (s%4)/2;
//          nibble phi = 2*(s%2) + h at bits [4phi, 4phi+4) (even k) and +16 (odd k);
//          phi <= 1 in place (o = 4phi), phi >= 2 after >> 8 (o = 4phi - 8): o = 4h.
//   8-bit: atom = 4 planes x [32 lanes x 16 B]; plane s/2, word 2*(s%2) + h; byte 2*rowhalf + odd
//          (expanded with one byte permute per pair; o = 0).
//   6-bit: low four bits stored exactly as a 4-bit atom (1024 B, o = 4h), then a 2-bit plane [32 lanes x 16 B] with
//          the high two bits, word jh*2 + rowhalf as in a 2-bit atom.  The high bits of step s4 = s%4, pair h must
//          land on bits [o+4, o+6) = 4 + 4h (even k; +16 odd k) of a copy of that word: the copies are the word
//          itself (s4 = 0), the word >> 2 (s4 = 1), the word with the bytes of each half swapped (s4 = 2) and that
//          one >> 2 (s4 = 3), so the field is stored at bit (4 + 4h + {0, 2, 8, 10}[s4]) % 16 of its half.  The
//          eight fields of a half tile its sixteen bits exactly.
#pragma once
#include <stdint.h>

namespace dyn {

struct CodeLoc {
    int byte_off;  // byte offset of the 32-bit word inside the atom
    int shift;     // bit position of the field inside that word
    int width;     // field width
};

// r: row in atom (0..15), kk: k in chunk (0..127).  For 3-bit, part 0 = low two bits, part 1 = high bit; for
// 6-bit, part 0 = low four bits, part 1 = high two bits.
__host__ __device__ inline CodeLoc code_loc(int bits, int r, int kk, int part) {
    const int gid = r & 7, rowhalf = r >> 3;
    const int s = kk >> 4, kq = kk & 15;
    const int tid4 = kq >> 2, h = (kq >> 1) & 1, odd = kq & 1;
    const int lane = gid * 4 + tid4;
    const int jh = s >> 2, s4 = s & 3;
    CodeLoc L;
    if (bits == 6 && part == 1) {  // 6-bit, high two bits
        const int rot = (s4 & 1) * 2 + (s4 >> 1) * 8;
        L.byte_off = 1024 + lane * 16 + (jh * 2 + rowhalf) * 4;
        L.shift = ((4 + 4 * h + rot) & 15) + 16 * odd;
        L.width = 2;
    } else if (bits == 4 || bits == 6) {
        const int phi = 2 * (s4 & 1) + h;
        L.byte_off = jh * 512 + lane * 16 + (rowhalf * 2 + (s4 >> 1)) * 4;
        L.shift = 4 * phi + 16 * odd;
        L.width = 4;
    } else if (bits == 8) {
        L.byte_off = (s >> 1) * 512 + lane * 16 + (2 * (s & 1) + h) * 4;
        L.shift = 8 * (2 * rowhalf + odd);
        L.width = 8;
    } else if (bits == 2 || (bits == 3 && part == 0)) {
        const int phi = 2 * s4 + h;
        L.byte_off = lane * 16 + (jh * 2 + rowhalf) * 4;
        L.shift = 2 * phi + 16 * odd;
        L.width = 2;
    } else {  // 3-bit, high bit plane
        const int phi = 2 * s4 + h;
        const int o = 2 * (phi & 3);
        const int st = 2 * jh + (phi >> 2);
        const int rot = (st & 1) + 8 * (st >> 1);
        L.byte_off = 512 + lane * 8 + rowhalf * 4;
        L.shift = (o + 2 + 16 * odd + rot) & 31;
        L.width = 1;
    }
    return L;
}

// Activations feeding a matrix packed at `bits` are stored multiplied by 2^x_scale_exp(bits, k):
// bias - o(k), with o the in-place bit offset of the code of input index k (periodic in k mod 64).
__host__ __device__ inline int x_scale_bias(int bits) {
    return bits == 2 ? 4 : (bits == 3 ? 3 : ((bits == 4 || bits == 6) ? 2 : 0));
}
__host__ __device__ inline int x_scale_exp(int bits, int k) {
    const int s4 = (k >> 4) & 3, h = (k >> 1) & 1;
    const int phi = 2 * s4 + h;
    int o = 0;
    if (bits == 2) o = phi <= 4 ? 2 * phi : 2 * phi - 10;
    else if (bits == 3) o = 2 * (phi & 3);
    else if (bits == 4 || bits == 6) o = 4 * h;
    return x_scale_bias(bits) - o;
}

}  // namespace dyn
