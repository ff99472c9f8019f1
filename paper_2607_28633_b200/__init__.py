"""TopKV data plane for one B200: per-layer pack / unpack of a paged KV cache to and from a
contiguous wire buffer, plus the pinned-host PCIe leg (§3.4, §5.2 of the paper).

``paper_2607_28633_b200.binding`` wraps the C-ABI library built from ``csrc/``;
``paper_2607_28633_b200.workloads`` draws the seeded synthetic inputs. Importing this
package does not load the CUDA library; the first binding call does, and raises if the
library has not been built.
"""
__all__ = ["binding", "workloads"]
