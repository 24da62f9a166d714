"""CPU oracle of the DEF / DEF-A / EF step (test infrastructure, never the product path)."""
from .def_oracle import *  # noqa: F401,F403
