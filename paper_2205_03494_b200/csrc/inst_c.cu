// Kernel instantiations for one group of formats (split so the groups compile in parallel).
#include "kernels.cuh"
namespace omc {
OMC_DEFINE_FORMAT(4, 14)
OMC_DEFINE_FORMAT(3, 7)
OMC_DEFINE_FORMAT(2, 3)
}  // namespace omc
