"""CPU oracle for GLIDE hybrid attention: test infrastructure only.

Nothing under the product package may import this; the product path never
falls back to it.
"""
