// Per-centre kernel instantiations for l_max in [11, 12].
#define SOAP_GROUP 3
#define SOAP_L_LIST X(11) X(12)
#include "center_inst.inc"
