// Shared by the translation units of the library; not part of the C ABI.
#pragma once

namespace sidco_internal {

// Count one kernel launch towards sidco_launch_count().
void note_launch();

}  // namespace sidco_internal
