// Kernel instantiations for one group of formats (split so the groups compile in parallel).
#include "kernels.cuh"
namespace omc {
OMC_DEFINE_FORMAT(3, 9)
OMC_DEFINE_FORMAT(4, 8)
OMC_DEFINE_FORMAT(5, 7)
}  // namespace omc
