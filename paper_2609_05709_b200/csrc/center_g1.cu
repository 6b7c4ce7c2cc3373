// Per-centre kernel instantiations for l_max in [6, 7, 8].
#define SOAP_GROUP 1
#define SOAP_L_LIST X(6) X(7) X(8)
#include "center_inst.inc"
