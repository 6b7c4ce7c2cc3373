// Per-centre kernel instantiations for l_max = 8.
#define SOAP_L 8
#include "center_inst.inc"
