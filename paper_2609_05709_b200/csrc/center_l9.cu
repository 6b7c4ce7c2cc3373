// Per-centre kernel instantiations for l_max = 9.
#define SOAP_L 9
#include "center_inst.inc"
