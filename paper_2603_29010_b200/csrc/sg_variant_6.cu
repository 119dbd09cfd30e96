// Kernel variant 6 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 6
#include "sg_variant.inc"
