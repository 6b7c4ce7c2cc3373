// Per-centre kernel instantiations for l_max = 12.
#define SOAP_L 12
#include "center_inst.inc"
