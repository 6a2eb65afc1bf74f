// placeholder: the tcgen05 kernel is added next
#include "dm_internal.h"
namespace dm {
struct FusedState { int unused; };
bool fused_supported(const HeadDesc&, int) { return false; }
int fused_create(FusedState** out, const HeadDesc&, int, int, size_t* bytes) { *out = nullptr; *bytes = 0; return DM_OK; }
void fused_destroy(FusedState*) {}
int fused_launch(FusedState*, const HeadDesc&, const void*, int, int, const RowMap&, const MaskKey&, int*,
                 unsigned long long*, float*, uint32_t*, cudaStream_t, int*) { return DM_EUNSUPPORTED; }
}
