// Host-side state shared by the translation units of the library.
#pragma once

namespace gaf {

// Sets what gaf_last_launch_count() reports for the calling thread.
void set_last_launch_count(int launches);

}  // namespace gaf
