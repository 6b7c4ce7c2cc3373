// Per-centre kernel instantiations for l_max = 10.
#define SOAP_L 10
#include "center_inst.inc"
