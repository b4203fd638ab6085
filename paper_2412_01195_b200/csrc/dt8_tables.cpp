// Host-side builders for the dt8 constant tables (see dt8_tables.h).
#include "dt8_tables.h"

#include <cmath>
#include <cstring>
#include <mutex>

namespace dt8 {

namespace {

uint32_t bits_of(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return u;
}

// Positive magnitudes of the data type, indexed by the magnitude bit pattern (Section IV-B):
// decade E = length of the zero run holds 2^F values, F = W-1-E, spaced evenly over
// (10^-(E+1), 10^-E]; the pattern of the k-th of them is 2^F + k.
void build_magnitudes(int W, float* mag) {
  mag[0] = 0.0f;
  double decade_scale = 10.0;  // 10^(E+1)
  for (int E = 0; E < W; ++E, decade_scale *= 10.0) {
    const int levels = 1 << (W - 1 - E);
    const double den = decade_scale * levels;  // an exact integer
    for (int k = 0; k < levels; ++k) {
      const double num = levels + 9.0 * (k + 1);
      mag[levels + k] = static_cast<float>(num / den);
    }
  }
}

bool build_enc(int W, int shift, EncTable* t) {
  const int P = (1 << W) - 1;  // largest magnitude pattern
  float mag[256];
  build_magnitudes(W, mag);
  uint32_t thr_bits[256];
  bool thr_exact[256];
  for (int i = 0; i < P; ++i) {
    const double mid = (static_cast<double>(mag[i]) + static_cast<double>(mag[i + 1])) * 0.5;
    float f = static_cast<float>(mid);
    if (static_cast<double>(f) > mid) f = std::nextafterf(f, 0.0f);  // round toward zero
    thr_bits[i] = bits_of(f);
    thr_exact[i] = static_cast<double>(f) == mid;
    if (i > 0 && thr_bits[i] <= thr_bits[i - 1]) return false;
  }
  const uint32_t one_bits = 0x3F800000u;
  if (thr_bits[P - 1] >= one_bits) return false;
  t->shift = shift;
  t->first_key = (thr_bits[0] >> 23) << (23 - shift);
  const uint32_t top_key = one_bits >> shift;
  const int n = static_cast<int>(top_key - t->first_key) + 2;
  if (n > kMaxEncEntries) return false;
  const bool is_signed = (W == 7);
  if (is_signed ? shift != 16 : shift != 15) return false;
  // field layouts, see dt8_tables.h
  const uint32_t ones = is_signed ? 0x7F00u : 0u;   // the bits between the count and the field
  const int field_shift = is_signed ? 15 : 17;
  const uint32_t none = (is_signed ? 0x1FFFFu : 0x7FFFu) << field_shift;
  t->num_entries = n;
  t->entries[0] = 1u | ones | none;   // the count is stored plus one
  int next = 0;  // first threshold not yet below the current bucket
  for (int idx = 1; idx <= n - 2; ++idx) {
    const uint32_t start = (t->first_key + static_cast<uint32_t>(idx - 1)) << shift;
    const uint32_t end = start + (1u << shift);
    while (next < P && thr_bits[next] < start) ++next;
    uint32_t entry = static_cast<uint32_t>(next + 1) | ones | none;
    if (next < P && thr_bits[next] < end) {
      if (next + 1 < P && thr_bits[next + 1] < end) return false;  // two thresholds in a bucket
      const uint32_t low = thr_bits[next] - start;
      const uint32_t field = is_signed ? 2u * low + (thr_exact[next] ? 0u : 1u) : low;
      entry = static_cast<uint32_t>(next + 1) | ones | (field << field_shift);
    }
    t->entries[idx] = entry;
  }
  t->entries[n - 1] = static_cast<uint32_t>(P + 1) | ones | none;
  return true;
}

}  // namespace

void build_codebook(bool is_signed, float out[256]) {
  float mag[256];
  if (is_signed) {
    build_magnitudes(7, mag);
    for (int p = 0; p < 128; ++p) {
      out[128 + p] = mag[p];
      out[127 - p] = -mag[p];
    }
  } else {
    build_magnitudes(8, mag);
    for (int p = 0; p < 256; ++p) out[p] = mag[p];
  }
}

bool build_tables(Tables* t) {
  build_codebook(true, t->dec_signed);
  build_codebook(false, t->dec_unsigned);
  return build_enc(7, kSignedShift, &t->enc_signed) && build_enc(8, kUnsignedShift, &t->enc_unsigned);
}

const Tables* host_tables() {
  static Tables tables;
  static bool ok = false;
  static std::once_flag once;
  std::call_once(once, [] { ok = build_tables(&tables); });
  return ok ? &tables : nullptr;
}

}  // namespace dt8
