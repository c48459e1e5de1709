#pragma once
#include "swaa_internal.cuh"
namespace swaa {
constexpr int kPrefillBM = 128;
constexpr int kPrefillBN = 128;
}
extern "C" int swaa_prefill(const void*, const void*, const void*, void*, const int32_t*, int, int, int, int, int, int, int, int, int, float, float*, void*) { return SWAA_ERR_UNSUPPORTED; }
