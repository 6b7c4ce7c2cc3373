// Per-centre kernel instantiations for l_max = 3.
#define SOAP_L 3
#include "center_inst.inc"
