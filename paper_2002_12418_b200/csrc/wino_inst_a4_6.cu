// Instantiations of the Winograd transform kernels (see wino_transforms.cuh).
#include "wino_transforms.cuh"

MNNB_DEFINE_INPUT(4)
MNNB_DEFINE_INPUT(6)
MNNB_DEFINE_OUTPUT(4, 2)
MNNB_DEFINE_OUTPUT(6, 4)
MNNB_DEFINE_OUTPUT(6, 2)
