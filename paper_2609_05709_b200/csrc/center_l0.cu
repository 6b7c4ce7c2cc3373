// Per-centre kernel instantiations for l_max = 0.
#define SOAP_L 0
#include "center_inst.inc"
