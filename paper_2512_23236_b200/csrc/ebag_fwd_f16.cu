// Forward kernel instantiation for one storage type (its own translation unit so that the
// four types compile in parallel).
#include "ebag_fwd.cuh"

namespace ebag {
EBAG_DEFINE_LAUNCHERS(f16, DT_F16)
}  // namespace ebag
