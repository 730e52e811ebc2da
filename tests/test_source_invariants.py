"""Invariants of the CUDA sources that no run on a single shape would catch.

A kernel launched with the stream-serialization attribute may start before its predecessor has
finished; it is only ordered after it by its own `dep_wait()`.  A kernel that is launched through
`dep_launch` and never waits would silently race with the previous kernel of the stream, and so
would every later kernel that relies on it for transitive ordering.
"""
import os
import re

CSRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                    "paper_1412_7580_b200", "csrc")


def kernels_of(text):
    """(name, body) of every __global__ kernel: the body runs to the next kernel or launcher."""
    parts = re.split(r"\n__global__ ", text)
    out = []
    for chunk in parts[1:]:
        m = re.search(r"([A-Za-z_0-9]*_kernel)\s*\(", chunk)
        end = chunk.find("\nstatic ")
        out.append((m.group(1), chunk if end < 0 else chunk[:end]))
    return out


def test_every_kernel_launched_as_a_dependent_waits_for_its_predecessor():
    checked = 0
    for name in sorted(os.listdir(CSRC)):
        if not name.endswith((".cu", ".cuh")) or name == "dep_launch.cuh":
            continue
        text = open(os.path.join(CSRC, name)).read()
        if "dep_launch(" not in text:
            assert "dep_wait()" not in text
            continue
        for kern, body in kernels_of(text):
            assert "dep_wait();" in body, f"{name}: {kern} is launched through dep_launch but never waits"
            assert "dep_trigger();" in body, f"{name}: {kern} never lets its dependents start"
            first_wait = body.index("dep_wait();")
            # no global-memory traffic before the wait: none of the access helpers may appear above it
            head = body[:first_wait]
            for token in ("__ldg(", "tma_load", "tma_store", "fk_tma_", "fk_cp16(", "cp.async", "atomic"):
                if token in head:
                    # lambdas defined above the wait may name these; they must not be *called* there:
                    # a call outside a lambda body sits at brace depth 1 of the kernel
                    depth, i, offending = 0, 0, False
                    while i < len(head):
                        c = head[i]
                        if c == "{":
                            depth += 1
                        elif c == "}":
                            depth -= 1
                        elif head.startswith(token, i) and depth <= 1:
                            offending = True
                            break
                        i += 1
                    assert not offending, f"{name}: {kern} touches global memory ({token}) before dep_wait()"
            checked += 1
    assert checked >= 6      # forward, inverse, two-pass forward and inverse, both contractions


def test_plain_launch_syntax_is_not_mixed_into_files_with_dependent_launches():
    for name in sorted(os.listdir(CSRC)):
        text = open(os.path.join(CSRC, name)).read()
        if "dep_launch(" in text and name != "dep_launch.cuh":
            assert "<<<" not in text, f"{name}: a kernel here bypasses dep_launch"
