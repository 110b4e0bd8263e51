#include "kvp_host.h"
