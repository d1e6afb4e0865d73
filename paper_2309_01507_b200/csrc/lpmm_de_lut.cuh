// Lookup table of the table-driven nearest-entry search for the signed 4-bit dynamic-exponent map.
//
// For a normalized value n with |n| in [2^-9, 2) the key is the top 11 bits of |n| below the sign
// (8 exponent bits, 3 mantissa bits), minus the key of 2^-9: 80 bins, each holding at most one of the
// decision thresholds of the nearest-entry rule. An entry is {threshold bits, code if |n| <= threshold};
// the code if |n| > threshold is one more. Bins without a threshold carry FLT_MAX.
//   non-negative n: thresholds are the largest binary32 values not above the exact midpoints of adjacent
//                   table entries (a tie stays at the lower entry); codes 7 .. 15.
//   negative n    : a tie must go to the lower index, i.e. to the larger magnitude, so a threshold that is
//                   an exact midpoint is lowered by one ulp; codes are stored as 15 - code (8 .. 15) so that
//                   the same "+1 above the threshold" rule applies; the caller flips them back with ^ 15.
// Values below 2^-9 are clamped into bin 0 (nearest entry 0, code 7).
#pragma once
#include <stdint.h>

namespace lpmm {

constexpr int kDeLutBins = 80;
constexpr float kDeLutMinAbs = 0.001953125f;             // 2^-9
constexpr uint32_t kDeLutKeyBias = 118u * 64u;           // byte offset of the key of 2^-9: (exponent 118 * 8 + 0) * 8

__device__ __constant__ uint2 kDeLut[2 * kDeLutBins] = {
    // non-negative side
    {0x7f7fffffu, 7u}, {0x7f7fffffu, 7u}, {0x7f7fffffu, 7u}, {0x3b343958u, 7u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x3c9ba5e3u, 8u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x3d6147aeu, 9u}, {0x7f7fffffu, 10u},
    {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u},
    {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u},
    {0x7f7fffffu, 10u}, {0x3e147ae1u, 10u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u},
    {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u},
    {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x3ea66666u, 11u}, {0x7f7fffffu, 12u},
    {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u},
    {0x3f0ccccdu, 12u}, {0x7f7fffffu, 13u}, {0x7f7fffffu, 13u}, {0x7f7fffffu, 13u},
    {0x3f466666u, 13u}, {0x7f7fffffu, 14u}, {0x7f7fffffu, 14u}, {0x3f719999u, 14u},
    {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u},
    {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u},
    // negative (codes stored as 15 - code) side
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x3b343957u, 8u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x3c9ba5e2u, 9u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u},
    {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u},
    {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u},
    {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x3d6147adu, 10u}, {0x7f7fffffu, 11u},
    {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u},
    {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u},
    {0x7f7fffffu, 11u}, {0x3e147ae1u, 11u}, {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u},
    {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u},
    {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u}, {0x3ea66666u, 12u}, {0x7f7fffffu, 13u},
    {0x7f7fffffu, 13u}, {0x7f7fffffu, 13u}, {0x7f7fffffu, 13u}, {0x7f7fffffu, 13u},
    {0x3f0cccccu, 13u}, {0x7f7fffffu, 14u}, {0x7f7fffffu, 14u}, {0x7f7fffffu, 14u},
    {0x3f466666u, 14u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u},
    {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u},
    {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u},
};

}  // namespace lpmm
