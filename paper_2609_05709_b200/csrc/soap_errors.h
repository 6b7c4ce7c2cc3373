// Error codes of the C ABI, for the internal translation units.
#pragma once
#include "soap.h"
