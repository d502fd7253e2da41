// Host-side re-tiling of a matrix's canonical k-bit index stream into the layout the kernels read.
//
// Canonical (upload) order: index i = row * kc + col at stream bits [i*k, i*k+k).
// A *quantum* is 128 consecutive indexes held by one lane = k 16-byte planes:
//   kc >= 128 : quantum (row r, chunk j) = columns [128 j, 128 j + 128) of row r
//   kc == 64  : quantum (group g, lane l) = row 64 g + l followed by row 64 g + 32 + l
// Device order: for each row group (32 rows, or 64 rows when kc == 64) and chunk j, plane p of
// the 32 lanes' quanta is one contiguous 512-byte line:
//   byte address = (((g * J + j) * k + p) * 32 + lane) * 16,   J = max(kc / 128, 1).
// The size stays k bits per weight.
#pragma once
#include <stdint.h>
#include <string.h>

namespace sti {

inline void retile_matrix(const uint8_t* src, uint8_t* dst, uint32_t rows, uint32_t kc, uint32_t k) {
  if (kc >= 128) {
    const uint32_t J = kc / 128;
    for (uint32_t r = 0; r < rows; ++r) {
      const uint32_t g = r / 32, l = r % 32;
      for (uint32_t j = 0; j < J; ++j) {
        const uint8_t* q = src + (static_cast<size_t>(r) * J + j) * 16 * k;
        for (uint32_t p = 0; p < k; ++p)
          memcpy(dst + ((static_cast<size_t>(g) * J + j) * k + p) * 512 + l * 16, q + p * 16, 16);
      }
    }
  } else {   // kc == 64: a row is 8k bytes
    for (uint32_t r = 0; r < rows; ++r) {
      const uint32_t g = r / 64, l = r % 32, half = (r % 64) / 32;
      const uint8_t* row = src + static_cast<size_t>(r) * 8 * k;
      for (uint32_t u = 0; u < k; ++u) {
        const uint32_t qb = half * 8 * k + 8 * u;     // byte position inside the lane's quantum
        memcpy(dst + ((static_cast<size_t>(g) * k + qb / 16) * 32 + l) * 16 + qb % 16, row + 8 * u, 8);
      }
    }
  }
}

}  // namespace sti
