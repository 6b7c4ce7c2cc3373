// Per-centre kernel instantiations for l_max = 5.
#define SOAP_L 5
#include "center_inst.inc"
