// Kernel instantiations for one group of formats (split so the groups compile in parallel).
#include "kernels.cuh"
namespace omc {
OMC_DEFINE_FORMAT(8, 7)
OMC_DEFINE_FORMAT(8, 23)
}  // namespace omc
