// Per-centre kernel instantiations for l_max = 11.
#define SOAP_L 11
#include "center_inst.inc"
