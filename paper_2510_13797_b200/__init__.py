"""Breadcrumbs Reasoning decode hot path for B200 (sm_100a).

The compute lives in a C-ABI shared library (csrc/ -> libbreadcrumbs.so);
`binding` marshals arguments to it.  Importing this package loads nothing
heavy; the library is opened on first use and its absence is an error.
"""
__all__ = ["binding", "workloads"]
