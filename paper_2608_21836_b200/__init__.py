"""B200-native causal attention hot path: prefill, decode and KV-cache append.

``paper_2608_21836_b200.binding`` is the thin ctypes layer over the C-ABI library
(``libl4l.so``, built from ``csrc/``); ``paper_2608_21836_b200.workloads`` draws the
seeded synthetic inputs. Importing the package loads nothing heavy; the library is
opened on first use and its absence is an error, never a fallback.
"""
__all__ = ["binding", "workloads"]
