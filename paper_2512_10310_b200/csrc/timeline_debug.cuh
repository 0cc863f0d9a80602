// Clock stamps for debug builds of the attention kernel (-DEVLN_TIMELINE): each CTA records up to
// 64 values of clock64() in a caller-provided buffer.  Regular builds compile the stamps away and
// carry no trace of them in the kernel arguments.
#pragma once

#ifdef EVLN_TIMELINE
namespace evln {
__device__ long long* g_timeline_dev = nullptr;   // [grid][64]; set through evlnDebugSetTimeline
}
#define EVLN_STAMP(slot)                                                                    \
    do {                                                                                    \
        long long* tl__ = evln::g_timeline_dev;                                             \
        if (tl__ && (slot) < 64) tl__[(long)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 64 + (slot)] = clock64(); \
    } while (0)
#else
#define EVLN_STAMP(slot) do { } while (0)
#endif
