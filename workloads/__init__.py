"""Expression descriptions and seeded synthetic inputs (data only, no arithmetic of the method)."""
from .expr import Access, Builder, Expr, Node, OPS, unit  # noqa: F401
from . import configs  # noqa: F401
