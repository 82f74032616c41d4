"""Properties of the kernel sources that other code relies on and that no GPU run would show when broken."""
import glob
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2506_06295_b200", "csrc")


def _events(path):
    out = []
    for n, line in enumerate(open(path).read().split("\n"), 1):
        code = line.split("//")[0]
        if "pdl_wait()" in code or "pdl_trigger()" in code:
            if re.search(r"__device__.*void\s+pdl_(wait|trigger)\s*\(", code):
                continue                                    # the definitions themselves
            out.append((n, "wait" if "pdl_wait()" in code else "trigger"))
    return out


def test_every_kernel_releases_its_dependents_only_after_its_own_dependency_wait():
    """The row-wise kernels that follow a projection fetch, BEFORE their dependency wait, data written two or more
    launches earlier.  That is only sound while every kernel calls griddepcontrol.launch_dependents after its own
    griddepcontrol.wait: then a launch can become resident only once the launch before it has passed its wait, i.e.
    once everything older has completed."""
    files = sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cuh")))
    assert files
    triggers = 0
    for f in files:
        ev = _events(f)
        for k, (n, what) in enumerate(ev):
            if what != "trigger":
                continue
            triggers += 1
            assert k > 0 and ev[k - 1][1] == "wait" and n - ev[k - 1][0] <= 3, \
                f"{os.path.basename(f)}:{n}: launch_dependents is not directly behind the kernel's dependency wait"
    assert triggers >= 30                                    # the scan sees the kernels
