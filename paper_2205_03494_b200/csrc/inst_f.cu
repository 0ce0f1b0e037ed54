// Kernel instantiations for one group of formats (split so the groups compile in parallel).
#include "kernels.cuh"
namespace omc {
OMC_DEFINE_FIXED_FORMAT(0, 7)
OMC_DEFINE_FIXED_FORMAT(0, 11)
OMC_DEFINE_FIXED_FORMAT(0, 15)
}  // namespace omc
