// Optional in-kernel clock stamps for role timelines.  Off in the product build: without -DRTN_TIMELINE every
// macro below expands to nothing.  `python -m paper_1912_02057_b200.build --timeline` builds
// librtn_b200_timeline.so with the stamps compiled in; `python -m paper_1912_02057_b200.timeline` runs a
// workload on it and prints, per recorded CTA, when each role began and ended each tile.
//
// A translation unit that wants stamps says RTN_TL_DEFINE(tag) once at file scope (its own stamp array and an
// extern "C" reader rtn_timeline_read_<tag>) and RTN_TL(tag, slot) where a role passes a point; one thread of
// the role calls it.  Stamps are raw SM cycle counters (clock64): consistent within a CTA, so the tool reports
// them relative to the CTA's slot 0.  Four CTAs are recorded: blockIdx.x = 0, g/4, 2g/4, 3g/4 of a grid of g.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace rtn {
namespace tl {
constexpr int kCtas = 4;
constexpr int kSlots = 96;
}  // namespace tl
}  // namespace rtn

#ifdef RTN_TIMELINE
#define RTN_TL_DEFINE(tag)                                                                              \
    namespace rtn { namespace tl { __device__ long long g_stamps_##tag[kCtas][kSlots]; } }              \
    extern "C" int rtn_timeline_read_##tag(long long* host, int clear)                                  \
    {                                                                                                   \
        if (clear) {                                                                                    \
            static long long zeros[rtn::tl::kCtas * rtn::tl::kSlots];                                   \
            return (int)cudaMemcpyToSymbol(rtn::tl::g_stamps_##tag, zeros, sizeof(zeros));              \
        }                                                                                               \
        return (int)cudaMemcpyFromSymbol(host, rtn::tl::g_stamps_##tag,                                 \
                                         sizeof(long long) * rtn::tl::kCtas * rtn::tl::kSlots);         \
    }
// RTN_TL_INIT(tag) once per thread near the kernel's entry (works out whether this CTA is recorded, and where);
// RTN_TL(tag, slot) is then a clock read and one store.
#define RTN_TL_INIT(tag)                                                                                \
    long long* tl_base_ = nullptr;                                                                      \
    {                                                                                                   \
        const unsigned tl_stride_ = gridDim.x >= rtn::tl::kCtas ? gridDim.x / rtn::tl::kCtas : 1u;      \
        if (blockIdx.x % tl_stride_ == 0 && blockIdx.x / tl_stride_ < (unsigned)rtn::tl::kCtas)         \
            tl_base_ = rtn::tl::g_stamps_##tag[blockIdx.x / tl_stride_];                                \
    }
#define RTN_TL(tag, slot)                                                                               \
    do {                                                                                                \
        const int tl_slot_ = (slot);                                                                    \
        if (tl_base_ != nullptr && tl_slot_ >= 0 && tl_slot_ < rtn::tl::kSlots) tl_base_[tl_slot_] = clock64(); \
    } while (0)
#else
#define RTN_TL_DEFINE(tag)
#define RTN_TL_INIT(tag)
#define RTN_TL(tag, slot) do {} while (0)
#endif
