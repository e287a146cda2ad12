// placeholder, replaced below
#include "lq_internal.h"
extern "C" lq_status lq_calibrate(const lq_config*, const uint16_t*, const uint16_t*, lq_layer**, double*) {
  return LQ_ERR_UNSUPPORTED;
}
