// Forward kernel instantiation for one storage type (its own translation unit so that the
// four types compile in parallel).
#include "ebag_fwd.cuh"

namespace ebag {
EBAG_DEFINE_LAUNCHERS(int8, DT_INT8)
}  // namespace ebag
