// Per-centre kernel instantiations for l_max = 6.
#define SOAP_L 6
#include "center_inst.inc"
