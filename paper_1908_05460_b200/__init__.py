from . import layers, inputs  # noqa: F401
