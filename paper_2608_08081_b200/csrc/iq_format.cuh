// The packed layouts of a run of entries (a K row, or a V record) for the three bit widths (Section 3.2, Step 4 fixes
// the size only): where entry e keeps its code, as plain arithmetic. The tuned 3-bit kernels and the decode kernel's
// byte-permute lookups use the same layouts through their own word-level code.
#pragma once
#include <stdint.h>

namespace iq {

template <int BITS>
struct PackedFormat {
  static constexpr int WORDS_PER_32 = BITS;            // 32 entries take BITS words
  static constexpr int V_RECORD_BYTES = 16 * BITS;     // 128 entries
  static __host__ __device__ constexpr int row_bytes(int d) { return BITS * d / 8; }
};

// Code of entry e of the run that starts at w.
template <int BITS>
__device__ __forceinline__ uint32_t packed_code(const uint32_t* w, int e) {
  if constexpr (BITS == 4) {
    return (w[e >> 3] >> (4 * (e & 7))) & 15u;
  } else if constexpr (BITS == 2) {
    const int j = e & 15;
    return (w[e >> 4] >> (j < 8 ? 4 * j : 4 * (j - 8) + 2)) & 3u;
  } else {
    const uint32_t* u = w + 3 * (e >> 5);  // groups of 32 entries in 3 words
    const int c = e & 31;
    if (c < 24) return (u[c >> 3] >> (4 * (c & 7))) & 7u;
    const int sh = 4 * (c - 24) + 3;
    return ((u[0] >> sh) & 1u) | (((u[1] >> sh) & 1u) << 1) | (((u[2] >> sh) & 1u) << 2);
  }
}

// b = 2 and b = 4 keep a code in contiguous bits of one word: which word of the run, and the shift.
template <int BITS>
__device__ __forceinline__ void packed_place(int e, int& word, int& shift) {
  static_assert(BITS == 2 || BITS == 4, "the 3-bit layout slices a quarter of its codes over three words");
  if constexpr (BITS == 4) {
    word = e >> 3;
    shift = 4 * (e & 7);
  } else {
    const int j = e & 15;
    word = e >> 4;
    shift = j < 8 ? 4 * j : 4 * (j - 8) + 2;
  }
}

}  // namespace iq
