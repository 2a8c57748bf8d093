// Test hooks of libmars: integer switches that force launch shapes which the library would not
// pick by itself for a given size (row splits, the single-block MMA kernel, cluster sizes of the
// stochastic tail, the top-k kernel's two batch shapes), so that tests can reach those code paths with small inputs.  They are set
// only through mars_test_hook() of the C ABI -- never from the environment -- so in a process
// that does not call it the library's behaviour is a function of the call's arguments alone.
#pragma once

namespace mars {

enum Hook { kHookForceSplit = 0, kHookLmheadSingleBlock = 1, kHookStochTailCluster = 2, kHookNoOverlap = 3,
            kHookTopkVariant = 4, kHookCount = 5 };

// Current value of a hook; 0 means "not set" (the library chooses).
int hook(int which);

}  // namespace mars
