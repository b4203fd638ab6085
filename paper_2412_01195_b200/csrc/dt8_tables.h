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
constexpr int kMaxEncEntries = 6656;

// Entry layouts.  The low bits hold one more than the number of thresholds below the bucket (the
// magnitude pattern at the bucket's lower edge, plus one), the top bits the threshold field:
//   signed   : T2 << 15 | 0x7F00 | (count + 1),  T2 = 2*threshold_low16 + (tie flag ? 0 : 1), 17 bits
//   unsigned : thr << 17 | (count + 1),           thr = threshold_low15, count + 1 in 9 bits
// A query word x carries its own threshold field in the same place, and the look-up returns
// entry - (x < entry ? 1 : 0): the pattern is count when the query's field does not exceed the
// stored one and count + 1 when it does.  The bits of an entry below its threshold field are never
// smaller than a query's (signed: ones down to the byte, above every bucket key up to 1.0;
// unsigned: the query has zeros there and count + 1 >= 1), so equal fields compare as "not above".
// A bucket without a threshold stores the all-ones field, which no query exceeds.
struct EncTable {
  int shift;            // bucket key = bits(a) >> shift
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
// bucket, table overflow).
bool build_tables(Tables* t);

// The process-wide tables, built on first use (thread-safe).  nullptr if the build failed.
const Tables* host_tables();

// Byte permute with the semantics of the PTX prmt.b32 default mode: output byte i is byte
// (nibble_i & 7) of the pair {y, x}; if bit 3 of the nibble is set the byte's sign bit is
// replicated instead.
DT8_HD uint32_t byte_perm(uint32_t x, uint32_t y, uint32_t sel) {
#if defined(__CUDA_ARCH__)
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(x), "r"(y), "r"(sel));
  return d;
#else
  const uint64_t src = (static_cast<uint64_t>(y) << 32) | x;
  uint32_t d = 0;
  for (int i = 0; i < 4; ++i) {
    const uint32_t nib = (sel >> (4 * i)) & 0xFu;
    uint32_t b = static_cast<uint32_t>(src >> (8 * (nib & 7u))) & 0xFFu;
    if (nib & 8u) b = (b & 0x80u) ? 0xFFu : 0u;
    d |= b << (8 * i);
  }
  return d;
#endif
}

// entry - (x < entry ? 1 : 0).  On the device the borrow of x - entry is taken off the entry
// (sub.cc / subc): two instructions, no predicate and no select.
DT8_HD uint32_t below_by_borrow(uint32_t entry, uint32_t x) {
#if defined(__CUDA_ARCH__)
  uint32_t r;
  asm("{\n\t.reg .b32 diff;\n\tsub.cc.u32 diff, %2, %1;\n\tsubc.u32 %0, %1, 0;\n\t}" : "=r"(r) : "r"(entry), "r"(x));
  return r;
#else
  return entry - (x < entry ? 1u : 0u);
#endif
}

// Bounds of one encode table in "byte address" form: bucket key k is looked up at byte offset
// 4*k.  lo4 = 4*(first_key - 1) is the entry "everything below", hi4 the entry "a >= 1".  In the
// kernels the table is placed in shared memory so that 4*k IS the shared-memory address of the
// entry of key k (no base to add); on the host HostFetch maps the offset back to the array.
struct EncBounds {
  uint32_t lo4, hi4;
};

DT8_HD EncBounds make_bounds(uint32_t first_key, int num_entries) {
  EncBounds b;
  b.lo4 = 4u * (first_key - 1u);
  b.hi4 = b.lo4 + 4u * (static_cast<uint32_t>(num_entries) - 1u);
  return b;
}

struct HostFetch {
  const uint32_t* entries;
  uint32_t lo4;
  DT8_HD uint32_t operator()(uint32_t k4) const { return entries[(k4 - lo4) >> 2]; }
};

// Signed table.  Returns a word whose low byte is the magnitude pattern p of |v| (exact ties go
// down for v > 0 and up for v < 0, i.e. to the lower index of the ascending table).
// x = v rotated by 16 bits: [mantissa_low16 | sign | exponent+mantissa_high7]; its top 17 bits are
// 2*low16 + sign, which is compared with T2; its low 15 bits are the bucket key.
// CLAMP_HI = false may be used only when |v| <= 1 is known (the key then never exceeds hi4).
template <bool CLAMP_HI, class Fetch>
DT8_HD uint32_t lookup_signed(const Fetch& fetch, const EncBounds& t, uint32_t v_bits) {
  const uint32_t x = byte_perm(v_bits, 0u, 0x1032u);
  uint32_t k4 = (x << 2) & 0x1FFFCu;
  k4 = k4 < t.lo4 ? t.lo4 : k4;
  if (CLAMP_HI) k4 = k4 > t.hi4 ? t.hi4 : k4;
  const uint32_t e = fetch(k4);
  return below_by_borrow(e, x);
}

// Unsigned table; negative values (and -0) count as 0.  lo4 << 13 is the bit pattern of the
// lower edge of the lowest bucket (4 * key << 13 == key << kUnsignedShift).
template <bool CLAMP_HI, class Fetch>
DT8_HD uint32_t lookup_unsigned(const Fetch& fetch, const EncBounds& t, uint32_t v_bits) {
  static_assert(kUnsignedShift == 15, "offset arithmetic below assumes a 15-bit bucket");
  const int32_t lo_bits = static_cast<int32_t>(t.lo4 << 13);
  int32_t s = static_cast<int32_t>(v_bits);
  s = s < lo_bits ? lo_bits : s;                      // also maps negatives to the lowest bucket
  const uint32_t a = static_cast<uint32_t>(s);
  uint32_t k4 = (a >> 13) & 0x7FFFCu;
  if (CLAMP_HI) k4 = k4 > t.hi4 ? t.hi4 : k4;
  const uint32_t e = fetch(k4);
  return below_by_borrow(e, a << 17);
}

// Gathers the low bytes of four words into one word (word 0 in byte 0).
DT8_HD uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return byte_perm(byte_perm(a, b, 0x0040u), byte_perm(c, d, 0x0040u), 0x5410u);
}

// Four signed codes from four looked-up words and the four normalised values they came from:
// code = 128 + p for v > 0, 127 - p for v < 0, and 127 whenever p == 0 (both zeros of the table
// are stored as the first one).  127 - p == p ^ 0x7F and 128 + p == p ^ 0x80 for p <= 127.
DT8_HD uint32_t finish_signed4(uint32_t e0, uint32_t e1, uint32_t e2, uint32_t e3, uint32_t v0,
                               uint32_t v1, uint32_t v2, uint32_t v3) {
  const uint32_t P = pack_low_bytes(e0, e1, e2, e3);
  const uint32_t top = byte_perm(byte_perm(v0, v1, 0x0073u), byte_perm(v2, v3, 0x0073u), 0x5410u);
  const uint32_t nonzero = P + 0x7F7F7F7Fu;                 // bit 7 of a byte set iff p >= 1
  const uint32_t flip = byte_perm(top | ~nonzero, 0u, 0xBA98u);  // 0xFF where v < 0 or p == 0
  return P ^ 0x80808080u ^ flip;
}

DT8_HD uint32_t finish_unsigned4(uint32_t e0, uint32_t e1, uint32_t e2, uint32_t e3) {
  return pack_low_bytes(e0, e1, e2, e3);
}

}  // namespace dt8
