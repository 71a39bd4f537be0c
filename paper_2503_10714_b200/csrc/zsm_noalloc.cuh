// Set-up hook of the static-scratch prompt pass (zsm_prefill_compress_static).
#pragma once

namespace zsm {

// Looks up, for the current device, the device address of the library's fixed scratch array (the
// module that holds it is loaded, and its bytes reserved, at that moment).  Returns 0 on success.
// Idempotent and cheap after the first call on a device.
int static_scratch_setup();

}  // namespace zsm
