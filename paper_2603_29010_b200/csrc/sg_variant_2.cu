// Kernel variant 2 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 2
#include "sg_variant.inc"
