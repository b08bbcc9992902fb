// NVTX ranges around the C entry points (host side), compiled in only with -DCLADA_NVTX: a timeline tool then shows
// which library call enqueued which launches.  Header-only NVTX 3; nothing is linked.
#pragma once

#ifdef CLADA_NVTX
#include <nvtx3/nvToolsExt.h>

namespace clada {
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};
}  // namespace clada
#define CLADA_RANGE(name) ::clada::NvtxRange clada_nvtx_range__(name)
#else
#define CLADA_RANGE(name) \
    do {                  \
    } while (0)
#endif
