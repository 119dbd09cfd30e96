// Kernel variant 9 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 9
#include "sg_variant.inc"
