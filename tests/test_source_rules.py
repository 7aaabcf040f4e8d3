"""Rules the CUDA sources must keep, checked on the text (no GPU needed)."""
import glob
import os
import re

CSRC = os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", "paper_2609_16648_b200", "csrc")


def _kernels(text):
    for m in re.finditer(r"__global__[^{;]*?(\w+)\s*\(([^)]*)\)\s*\{", text, re.S):
        i, depth = m.end(), 1
        while depth and i < len(text):
            depth += {"{": 1, "}": -1}.get(text[i], 0)
            i += 1
        yield m.group(1), text[m.end():i]


def test_every_kernel_launched_with_the_dependent_launch_attribute_waits_for_its_predecessor():
    """Kernels go out through launch_k, which allows programmatic dependent launch: the next kernel of the stream may start
    as soon as this one has signalled, so a kernel that never executes the wait can read its predecessor's output before it
    is written - and breaks the chain of completion for its successors too.  Every kernel calls pdl_prologue() (signal +
    wait) before touching global memory; the only exceptions are kernels launched with the plain <<< >>> syntax."""
    missing = []
    for path in sorted(glob.glob(os.path.join(CSRC, "*.cu"))):
        text = open(path).read()
        plain = set(re.findall(r"(\w+)\s*<<<", text))
        for name, body in _kernels(text):
            if "pdl_prologue" not in body and "griddepcontrol.wait" not in body and name not in plain:
                missing.append((os.path.basename(path), name))
    assert not missing, missing


def test_no_closed_cuda_calls_and_no_cluster_multicast_loads():
    banned = ["MemcpyBatch" + "Async", "Memcpy3DBatch" + "Async", ".multicast" + "::cluster"]
    for path in sorted(glob.glob(os.path.join(CSRC, "*"))):
        if not path.endswith((".cu", ".cuh", ".h")):
            continue
        text = open(path).read()
        for b in banned:
            if b == banned[2]:
                # the commit form that signals an mbarrier in the peer CTA is allowed; bulk / tensor loads are not
                for line in text.splitlines():
                    assert not (b in line and "cp.async.bulk" in line), (path, line)
            else:
                assert b not in text, (path, b)
