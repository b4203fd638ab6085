// Host-side construction of the constant tables of the dynamic-tree 8-bit data type, and the
// table-driven encoder shared by the kernels and the host self-check.
//
// Decode table: the 256 ascending code-book values (Section IV-B, Fig. dynamic_tree).
//
// Encode table: Eq. quant2 asks for the table entry nearest to a normalised value v.  In the
// magnitude domain that is p = #{ i : t_i < a }, a = |v|, where t_i is the mid-point between
// magnitude i and i+1 of the code book.  For a binary32 `a` the test t_i < a is the integer test
// bits(floor32(t_i)) < bits(a), so the count can be read from a table indexed by the top bits of
// `a`: every bucket of 2^shift consecutive bit patterns stores how many thresholds lie below the
// bucket and the low bits of the single threshold (if any) inside it.  The buckets are narrower
// than the smallest gap between thresholds, so one compare finishes the search exactly.
//
// Exact ties: the paper's argmin is read as "lowest index wins".  For positive v the lower index
// is the smaller magnitude (a == t_i stays below), for negative v it is the larger magnitude
// (a == t_i goes up); thresholds that are themselves binary32 numbers carry a flag for that.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define DT8_HD __host__ __device__ __forceinline__
#else
#define DT8_HD inline
#endif

namespace dt8 {

constexpr int kSignedShift = 16;    // 7 mantissa bits per bucket: width <= 2^-7 of the value
constexpr int kUnsignedShift = 15;  // 8 mantissa bits per bucket
constexpr uint32_t kNoThreshold = 0x7FFFFFu;
constexpr int kMaxEncEntries = 6656;

// entry = count_below | tie_flag << 8 | threshold_low_bits << 9
struct EncTable {
  int shift;            // bucket = bits(a) >> shift
  uint32_t first_key;   // bucket key of the first regular bucket
  int num_entries;      // entry 0: everything below; last entry: a >= 1
  uint32_t entries[kMaxEncEntries];
};

struct Tables {
  float dec_signed[256];
  float dec_unsigned[256];
  EncTable enc_signed;    // magnitude patterns 0..127
  EncTable enc_unsigned;  // magnitude patterns 0..255
};

// Fills the 256 ascending values.  Signed: out[127-p] = -value(p), out[128+p] = value(p).
void build_codebook(bool is_signed, float out[256]);

// Builds all tables; returns false if an internal consistency check fails (two thresholds in one
// bucket, more than 23 low bits, table overflow).
bool build_tables(Tables* t);

// The process-wide tables, built on first use (thread-safe).  nullptr if the build failed.
const Tables* host_tables();

// Magnitude pattern of `a_bits` (bits of a non-negative binary32); tie_up = 1 sends exact ties to
// the larger magnitude.
DT8_HD uint32_t encode_magnitude(const uint32_t* entries, int shift, uint32_t first_key,
                                 int num_entries, uint32_t a_bits, uint32_t tie_up) {
  int idx = (int)(a_bits >> shift) - (int)first_key + 1;
  idx = idx < 0 ? 0 : idx;
  idx = idx > num_entries - 1 ? num_entries - 1 : idx;
  const uint32_t e = entries[idx];
  const uint32_t low = (a_bits & ((1u << shift) - 1u)) + ((e >> 8) & tie_up);
  return (e & 0xFFu) + (low > (e >> 9) ? 1u : 0u);
}

// Code (index into the ascending signed table) of a normalised value given as raw bits.
DT8_HD uint32_t encode_signed(const uint32_t* entries, uint32_t first_key, int num_entries,
                              uint32_t v_bits) {
  const uint32_t neg = v_bits >> 31;
  const uint32_t p = encode_magnitude(entries, kSignedShift, first_key, num_entries,
                                      v_bits & 0x7FFFFFFFu, neg);
  const uint32_t c = neg ? 127u - p : 128u + p;
  return p == 0u ? 127u : c;   // both zeros are stored as the first one
}

// Code of a normalised value for the unsigned table; negative values map to the value 0.
DT8_HD uint32_t encode_unsigned(const uint32_t* entries, uint32_t first_key, int num_entries,
                                uint32_t v_bits) {
  const int32_t s = (int32_t)v_bits;
  const uint32_t a_bits = s < 0 ? 0u : (uint32_t)s;
  return encode_magnitude(entries, kUnsignedShift, first_key, num_entries, a_bits, 0u);
}

}  // namespace dt8
