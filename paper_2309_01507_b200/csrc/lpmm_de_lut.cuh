// Lookup table of the table-driven nearest-entry search for the signed 4-bit dynamic-exponent map.
//
// The key of a normalized value n is its top 11 bits (sign, 8 exponent bits, 2 mantissa bits: the binade
// [0.5, 1) holds three thresholds, in three different quarters). For |n| in [2^-9, 2) that leaves 40 bins per
// sign, each holding at most one decision threshold of the nearest-entry rule. An entry is {threshold, code for n <= threshold}; the code for n > threshold is one
// more ("n > threshold" is an ordinary signed fp32 comparison). Bins without a threshold carry FLT_MAX.
//   n >= 0: a threshold is the largest binary32 value not above the exact midpoint of two adjacent table
//           entries, so a value exactly on a midpoint keeps the lower code (ties go to the lower index).
//   n <  0: the code must go DOWN as |n| passes a midpoint, and a tie must take the lower index, i.e. the
//           larger magnitude. With t the largest binary32 magnitude that still keeps the upper code, the
//           entry stores the next value below -t and the lower code, so that n >= -t adds one.
// Outside the 40 bins the end codes repeat: entry 0 (code 7) below 2^-9, the extreme entries from 2.0 upwards.
#pragma once
#include <stdint.h>

namespace lpmm {

constexpr int kDeLutBins = 40;
constexpr uint32_t kDeLutFirstKey = 118u * 4u;           // key of 2^-9: exponent field 118, mantissa bits 00

__device__ __constant__ uint2 kDeLut[2 * kDeLutBins] = {
    // n >= 0
    {0x7f7fffffu, 7u}, {0x3b343958u, 7u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u}, {0x7f7fffffu, 8u},
    {0x3c9ba5e3u, 8u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u},
    {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x7f7fffffu, 9u}, {0x3d6147aeu, 9u},
    {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u}, {0x7f7fffffu, 10u},
    {0x3e147ae1u, 10u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u}, {0x7f7fffffu, 11u},
    {0x7f7fffffu, 11u}, {0x3ea66666u, 11u}, {0x7f7fffffu, 12u}, {0x7f7fffffu, 12u},
    {0x3f0ccccdu, 12u}, {0x7f7fffffu, 13u}, {0x3f466666u, 13u}, {0x3f719999u, 14u},
    {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u}, {0x7f7fffffu, 15u},
    // n < 0
    {0x7f7fffffu, 7u}, {0xbb343958u, 6u}, {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u},
    {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u},
    {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u}, {0x7f7fffffu, 6u},
    {0xbc9ba5e3u, 5u}, {0x7f7fffffu, 5u}, {0x7f7fffffu, 5u}, {0x7f7fffffu, 5u},
    {0x7f7fffffu, 5u}, {0x7f7fffffu, 5u}, {0x7f7fffffu, 5u}, {0xbd6147aeu, 4u},
    {0x7f7fffffu, 4u}, {0x7f7fffffu, 4u}, {0x7f7fffffu, 4u}, {0x7f7fffffu, 4u},
    {0xbe147ae2u, 3u}, {0x7f7fffffu, 3u}, {0x7f7fffffu, 3u}, {0x7f7fffffu, 3u},
    {0x7f7fffffu, 3u}, {0xbea66667u, 2u}, {0x7f7fffffu, 2u}, {0x7f7fffffu, 2u},
    {0xbf0ccccdu, 1u}, {0x7f7fffffu, 1u}, {0xbf466667u, 0u}, {0x7f7fffffu, 0u},
    {0x7f7fffffu, 0u}, {0x7f7fffffu, 0u}, {0x7f7fffffu, 0u}, {0x7f7fffffu, 0u},
};

}  // namespace lpmm
