// Registry of signature-specialised kernels.  Entries are appended by the generated
// translation units listed in fast/registry_entries.inc (a build with overlay signatures, see build.py,
// points E3J_REGISTRY_INC at its own list).
#include "fast_registry.hpp"

#include <cstring>

namespace e3j {

#ifndef E3J_REGISTRY_INC
#define E3J_REGISTRY_INC "fast/registry_entries.inc"
#endif

#define E3J_FAST_ENTRY(name) extern const FastKernels name;
#include E3J_REGISTRY_INC
#undef E3J_FAST_ENTRY

static const FastKernels* const kEntries[] = {
#define E3J_FAST_ENTRY(name) &name,
#include E3J_REGISTRY_INC
#undef E3J_FAST_ENTRY
    nullptr};

int fast_find(const char* signature) {
    for (int i = 0; kEntries[i]; ++i)
        if (std::strcmp(kEntries[i]->signature, signature) == 0) return i;
    return -1;
}

const FastKernels* fast_lookup(const e3j_plan* plan) {
    return (plan && plan->fast_id >= 0) ? kEntries[plan->fast_id] : nullptr;
}

}  // namespace e3j
