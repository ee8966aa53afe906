// Range checks of the bounds-checked build, shared by every kernel file.
#pragma once
#include "h1b_layout.cuh"

namespace h1b {

// Bounds-checked build (-DH1B_DEBUG_BOUNDS; compute-sanitizer's stand-in for the small test cases): every address a
// kernel derives from its parameters for a global-memory access (cache chunks, split-K partials, query sketches) and
// every carve of its shared memory is range-checked first. A check that fails records kStatusBounds + its number
// in the status word (the first failure stays) and the access is NOT made: nothing traps or faults; the host reads
// it with h1b_poll_status(). In the ordinary build the checks are the constant `true` and cost nothing.
enum BoundsSite { kSiteKeyWord = 1, kSiteValueRow = 2, kSiteQueryStore = 3, kSitePrefillValues = 4, kSitePrefillKeys = 5,
                  kSiteChunkCopy = 6, kSiteRing = 7, kSitePartialStore = 8, kSiteQueryLoad = 9, kSitePartialLoad = 10,
                  kSitePrefillSmem = 11, kSiteProbe = 12, kSitePromptChunk = 13, kSitePromptQuery = 14,
                  kSitePromptOut = 15 };
#ifdef H1B_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(bool ok, int32_t *status, int site) {
    if (!ok) atomicCAS(status, kStatusOk, kStatusBounds + site);
    return ok;
}
#define H1B_IN_BOUNDS(cond, status, site) bounds_ok((cond), (status), (site))
#else
#define H1B_IN_BOUNDS(cond, status, site) true
#endif
// [ptr, ptr + bytes) lies inside the cache region
__device__ __forceinline__ bool in_cache(const CacheAddr &ca, const void *ptr, size_t bytes) {
    const unsigned char *q = static_cast<const unsigned char *>(ptr);
    return q >= ca.base && q + bytes <= ca.base + ca.cache_bytes;
}

}  // namespace h1b
