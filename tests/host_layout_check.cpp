// Host-side check of the packed-code position functions (csrc/innerq_layout.h), compiled and run by
// tests/test_layout_host.py with the system C++ compiler; no GPU.  Two properties:
//   1. every position function is a bijection between (token, channel) and the bit fields of a row / chunk;
//   2. the mask arithmetic with which the integer-MMA decode kernel takes operand bytes out of a byte-ordered row or
//      chunk yields code * weight for the channel / token the layout's comments promise.
// Prints one line per failed property and returns the number of failures.
#include <cstdint>
#include <cstdio>
#include <vector>

#include "innerq_layout.h"

using namespace iq;

namespace {

int failures = 0;
void fail(const char* what, int a, int b) {
  if (failures < 20) std::printf("FAIL %s (%d, %d)\n", what, a, b);
  ++failures;
}

struct Bits {
  std::vector<int> hit;
  explicit Bits(int words) : hit(words * 32, 0) {}
  void mark(const BitPos& p, int n) {
    for (int b = 0; b < n; ++b) ++hit[p.word * 32 + p.bit + b];
  }
  bool exact_cover() const {
    for (int h : hit)
      if (h != 1) return false;
    return true;
  }
};

int test_code(int a, int b, int bits) { return (a * 7 + b * 3 + (a >> 3) + 5 * (b >> 2)) & ((1 << bits) - 1); }

void check_bijections() {
  for (int bits = 2; bits <= 4; ++bits) {
    for (int perm = 0; perm < 2; ++perm) {
      Bits row(4 * bits), chunk(128 * bits);
      for (int c = 0; c < kD; ++c) {
        if (bits == 3 && perm == 1) {
          const BitPos3 p = row_pos_i8_3(c);
          row.mark(p.lo, 2);
          row.mark(p.hi, 1);
        } else if (bits == 3) {
          BitPos lo = row_pos_plane(c, 2), hi = row_pos_plane(c, 1);
          hi.word += row_hi_plane_word();
          row.mark(lo, 2);
          row.mark(hi, 1);
        } else {
          row.mark(perm ? row_pos_i8(c, bits) : row_pos_plane(c, bits), bits);
        }
        for (int t = 0; t < kChunk; ++t) {
          if (bits == 3 && perm == 1) {
            const BitPos3 p = block_pos_i8_3(t, c);
            chunk.mark(p.lo, 2);
            chunk.mark(p.hi, 1);
          } else if (bits == 3) {
            BitPos lo = block_pos_plane(t, c, 2), hi = block_pos_plane(t, c, 1);
            hi.word += chunk_hi_plane_word();
            chunk.mark(lo, 2);
            chunk.mark(hi, 1);
          } else {
            chunk.mark(perm ? block_pos_i8(t, c, bits) : block_pos_plane(t, c, bits), bits);
          }
        }
      }
      if (!row.exact_cover()) fail("row positions are not a bijection", bits, perm);
      if (!chunk.exact_cover()) fail("chunk positions are not a bijection", bits, perm);
    }
  }
}

// operand byte b of a 32-bit fragment register
int byte_of(uint32_t w, int b) { return (w >> (8 * b)) & 0xff; }

// Keys: lane (gid, j) of the warp takes, for channel run p, the bytes k = 4 j + b (register half h = 0) and
// k = 16 + 4 j + b (h = 1) of its row: channel 32 p + k.
void check_row_extraction() {
  for (int bits = 2; bits <= 4; ++bits) {
    uint32_t row[16] = {0};
    int code[kD];
    for (int c = 0; c < kD; ++c) {
      code[c] = test_code(c, bits, bits);
      if (bits == 3) {
        const BitPos3 p = row_pos_i8_3(c);
        row[p.lo.word] |= code3_lo(code[c], p.odd) << p.lo.bit;
        row[p.hi.word] |= code3_hi(code[c], p.odd) << p.hi.bit;
      } else {
        const BitPos p = row_pos_i8(c, bits);
        row[p.word] |= (uint32_t)code[c] << p.bit;
      }
    }
    for (int j = 0; j < 4; ++j)
      for (int h = 0; h < 2; ++h)
        for (int p = 0; p < 4; ++p) {
          uint32_t a;
          int weight;
          if (bits == 2) {
            a = row[2 * j + h] & (0x03030303u << (2 * p));
            weight = 1 << (2 * p);
          } else if (bits == 4) {
            a = row[4 * j + 2 * (p >> 1) + h] & ((p & 1) ? 0xF0F0F0F0u : 0x0F0F0F0Fu);
            weight = (p & 1) ? 16 : 1;
          } else {
            const uint32_t lo = row[2 * j + h], hi = row[8 + j];
            const uint32_t ze = h ? hi >> 1 : hi, zo = h ? hi << 1 : hi;
            const uint32_t we = (lo & 0x33333333u) | (ze & 0xCCCCCCCCu), wo = (lo & 0xCCCCCCCCu) | (zo & 0x33333333u);
            a = (p & 1) ? (wo & (0x0E0E0E0Eu << (4 * (p >> 1)))) : (we & (0x07070707u << (4 * (p >> 1))));
            weight = field_weight_i8_3(p);
          }
          for (int b = 0; b < 4; ++b)
            if (byte_of(a, b) != code[32 * p + 16 * h + 4 * j + b] * weight) fail("row operand byte", bits, 32 * p + 16 * h + 4 * j + b);
        }
  }
}

// Values: lane (gid, j) takes, for m-tile m, register role 2 * half + rh, the bytes k = 16 half + 4 j + b of
// fragment row gid + 8 rh: token tau with 4 (tau % 8) + tau / 8 = k, channel block_row_channel(m, rh, gid).
void check_chunk_extraction() {
  for (int bits = 2; bits <= 4; ++bits) {
    std::vector<uint32_t> chunk(128 * bits, 0u);
    auto code_of = [&](int t, int c) { return test_code(c, t, bits); };
    for (int t = 0; t < kChunk; ++t)
      for (int c = 0; c < kD; ++c) {
        const uint32_t code = code_of(t, c);
        if (bits == 3) {
          const BitPos3 p = block_pos_i8_3(t, c);
          chunk[p.lo.word] |= code3_lo(code, p.odd) << p.lo.bit;
          chunk[p.hi.word] |= code3_hi(code, p.odd) << p.hi.bit;
        } else {
          const BitPos p = block_pos_i8(t, c, bits);
          chunk[p.word] |= code << p.bit;
        }
      }
    for (int lane = 0; lane < 32; ++lane) {
      const int gid = lane >> 2, j = lane & 3;
      for (int m = 0; m < 8; ++m)
        for (int role = 0; role < 4; ++role) {
          const int half = role >> 1, rh = role & 1;
          uint32_t a;
          int weight;
          if (bits == 2) {
            a = chunk[(m >> 2) * 128 + lane * 4 + role] & (0x03030303u << (2 * (m & 3)));
            weight = 1 << (2 * (m & 3));
          } else if (bits == 4) {
            a = chunk[(m >> 1) * 128 + lane * 4 + role] & ((m & 1) ? 0xF0F0F0F0u : 0x0F0F0F0Fu);
            weight = (m & 1) ? 16 : 1;
          } else {
            const int W = m >> 2, p = m & 3;
            const uint32_t lo = chunk[W * 128 + lane * 4 + role], hi = chunk[256 + lane * 4 + role];
            const uint32_t ze = W ? hi >> 1 : hi, zo = W ? hi << 1 : hi;
            const uint32_t we = (lo & 0x33333333u) | (ze & 0xCCCCCCCCu), wo = (lo & 0xCCCCCCCCu) | (zo & 0x33333333u);
            a = (p & 1) ? (wo & (0x0E0E0E0Eu << (4 * (p >> 1)))) : (we & (0x07070707u << (4 * (p >> 1))));
            weight = field_weight_i8_3(p);
          }
          for (int b = 0; b < 4; ++b) {
            const int k = 16 * half + 4 * j + b, tau = 8 * (k & 3) + (k >> 2);
            if (byte_of(a, b) != code_of(tau, block_row_channel(m, rh, gid)) * weight) fail("chunk operand byte", bits, lane * 64 + m * 4 + role);
          }
        }
    }
  }
}

// metadata order of a BLOCK-store group: index and channel are inverse to each other
void check_block_meta() {
  for (int c = 0; c < kD; ++c)
    if (block_meta_channel(block_meta_index(c)) != c) fail("block metadata order", c, block_meta_index(c));
}

}  // namespace

int main() {
  check_bijections();
  check_row_extraction();
  check_chunk_extraction();
  check_block_meta();
  std::printf("%d failure(s)\n", failures);
  return failures > 255 ? 255 : failures;
}
