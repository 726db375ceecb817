// Prefill kernel placeholder: dispatches to the generic prefill-order kernel until the tiled
// kernel lands.
#include "internal.h"
namespace detlin {
cudaError_t launch_prefill(const LaunchArgs& a) { return launch_generic(a, 1); }
}
