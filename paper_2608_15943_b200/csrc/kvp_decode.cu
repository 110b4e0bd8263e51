#include "kvp_host.h"
namespace kvp {
int decode_read_status() { return 0; }
}  // namespace kvp
